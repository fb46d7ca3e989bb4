"""GPU parity of PAPA's EMA (Eq. 1), the final average, PAPA-all and the consensus
distance against the oracle.  The kernels use the oracle's operation order with
explicitly rounded binary32 operations, so results are expected to be bit-identical;
the stated bar is 2 ulp (max relative error 2.4e-7)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_17517_b200 import binding as B
from paper_2405_17517_b200 import workloads as W
from gpu_util import Case, bits, to_device, to_host_bits, ulp_distance_f32

pytestmark = pytest.mark.gpu

RAGGED = [1000, 33, 7, 1, 4, 8, 5003, 2048]
MAX_ULP = 2


def _assert_close_f32(got_bits, want_bits, what):
    d = ulp_distance_f32(got_bits, want_bits)
    assert d.max() <= MAX_ULP, "%s: %d ulp" % (what, d.max())
    return int(d.max())


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N", [2, 3, 5, 7, 8, 10, 16, 32, 33, 64])
def test_ema_average_papa_all_fp32(N, layout):
    c = Case(N, RAGGED, layout, seed=N + 40)
    worst = 0
    for alpha in (0.99, 0.001, 0.5):
        B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, alpha)
        oracle.papa_ema(c.ora, c.host, alpha)
        torch.cuda.synchronize()
        worst = max(worst, _assert_close_f32(to_host_bits(c.dev), bits(c.host), "ema"))
        # keep both sides on the same state so errors cannot build up across calls
        c.dev.copy_(torch.from_numpy(c.host.reshape(-1).copy()))
    out = torch.full((c.P,), float("nan"), dtype=torch.float32, device="cuda")
    B.population_average(c.gpu.ctx, B.WASH_STACK_PARAMS, out, B.WASH_F32)
    want = np.full(c.P, np.nan, dtype=np.float32)
    oracle.population_average(c.ora, c.host, want)
    worst = max(worst, _assert_close_f32(to_host_bits(out), want.view(np.uint32), "average"))
    outb = torch.zeros(c.P, dtype=torch.bfloat16, device="cuda")
    B.population_average(c.gpu.ctx, B.WASH_STACK_PARAMS, outb, B.WASH_BF16)
    wantb = np.zeros(c.P, dtype=np.uint16)
    oracle.population_average(c.ora, c.host, wantb)
    assert (to_host_bits(outb) == wantb).all()
    B.papa_all(c.gpu.ctx, B.WASH_STACK_PARAMS)
    oracle.papa_all(c.ora, c.host)
    torch.cuda.synchronize()
    worst = max(worst, _assert_close_f32(to_host_bits(c.dev), bits(c.host), "papa_all"))
    assert worst == 0          # same operations in the same order: no difference at all
    B.wash_check(c.gpu.ctx)
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N", [2, 8, 9])
def test_bf16_stacks(N, layout):
    c = Case(N, RAGGED, layout, "bf16", seed=N + 60)
    B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, 0.999)
    oracle.papa_ema(c.ora, c.host, 0.999)
    c.assert_equal("bf16 ema")
    for code, np_dtype, t_dtype in ((B.WASH_F32, np.float32, torch.float32), (B.WASH_BF16, np.uint16, torch.bfloat16)):
        out = torch.zeros(c.P, dtype=t_dtype, device="cuda")
        B.population_average(c.gpu.ctx, B.WASH_STACK_PARAMS, out, code)
        want = np.zeros(c.P, dtype=np_dtype)
        oracle.population_average(c.ora, c.host, want)
        assert (to_host_bits(out) == bits(want)).all()
    B.papa_all(c.gpu.ctx, B.WASH_STACK_PARAMS)
    oracle.papa_all(c.ora, c.host)
    c.assert_equal("bf16 papa_all")
    c.close()


def test_special_values_follow_ieee():
    N, d = 4, 64
    dense = W.flat_population(N, d, seed=1)
    dense[0, 0] = np.inf; dense[1, 1] = -np.inf; dense[2, 2] = np.nan
    dense[0, 3] = np.inf; dense[1, 3] = -np.inf                     # inf - inf -> NaN
    dense[:, 4] = np.float32(1e-45)                                 # denormals are kept, not flushed
    dense[:, 5] = np.array([3e38, 3e38, -3e38, -3e38], np.float32)  # overflow in the running sum
    c = Case(N, [d], 0, dense=dense)
    B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, 0.9)
    oracle.papa_ema(c.ora, c.host, 0.9)
    torch.cuda.synchronize()
    assert ulp_distance_f32(to_host_bits(c.dev), bits(c.host)).max() == 0     # NaN == NaN by class
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
def test_bf16_rounding_cases_follow_the_oracle(layout):
    """Results that land on ties, overflow to infinity, stay denormal or are NaN, in whole
    groups (the paired conversion) and in a ragged tail (the element-wise one)."""
    N, d = 2, 4096 + 3
    rng = np.random.default_rng(5)
    dense = np.zeros((N, d), dtype=np.float32)
    # model 0 = a bf16 value, model 1 = the next bf16 value away from zero: their mean lies
    # halfway between two bf16 values, so the average is a tie for the rounding
    b = W.to_bf16_bits(rng.standard_normal(d).astype(np.float32)).astype(np.uint32)
    dense[0] = (b << 16).view(np.float32); dense[1] = ((b + 1) << 16).view(np.float32)
    dense[:, 8:16] = np.float32(3.38e38)                    # sum overflows
    dense[0, 16:24] = np.nan; dense[1, 24:32] = -np.inf
    dense[0, 32:40] = np.inf; dense[1, 32:40] = -np.inf      # inf - inf
    dense[:, 40:48] = np.float32(2e-40)                      # denormal results
    dense[0, d - 2] = np.nan                                 # in the ragged tail
    c = Case(N, [d], layout, "bf16", dense=dense)

    def same(got16, want16, what):
        dist = ulp_distance_f32(got16.astype(np.uint32) << 16, want16.astype(np.uint32) << 16)   # NaN == NaN by class
        assert dist.max() == 0, what

    for alpha in (0.5, 0.999):
        B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, alpha)
        oracle.papa_ema(c.ora, c.host, alpha)
        torch.cuda.synchronize()
        same(to_host_bits(c.dev), bits(c.host), "ema %g" % alpha)
        c.dev.copy_(to_device(c.host))
    out = torch.zeros(c.P, dtype=torch.bfloat16, device="cuda")
    B.population_average(c.gpu.ctx, B.WASH_STACK_PARAMS, out, B.WASH_BF16)
    want = np.zeros(c.P, dtype=np.uint16)
    oracle.population_average(c.ora, c.host, want)
    same(to_host_bits(out), want, "average")
    B.wash_check(c.gpu.ctx)
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N,dtype", [(5, "f32"), (8, "bf16"), (13, "f32")])
def test_consensus_distance(N, dtype, layout):
    c = Case(N, RAGGED, layout, dtype, seed=N)
    out = torch.zeros(N, dtype=torch.float64, device="cuda")
    B.wash_consensus_sq(c.gpu.ctx, B.WASH_STACK_PARAMS, 0, len(RAGGED), out)
    want = oracle.consensus_sq(c.ora, c.host)
    assert np.allclose(out.cpu().numpy(), want, rtol=1e-12, atol=0)
    part = torch.zeros(N, dtype=torch.float64, device="cuda")
    B.wash_consensus_sq(c.gpu.ctx, B.WASH_STACK_PARAMS, 2, 7, part)
    assert np.allclose(part.cpu().numpy(), oracle.consensus_sq(c.ora, c.host, 2, 7), rtol=1e-12, atol=0)
    # Eq. 5: a shuffle leaves the summed squared distance where it was; Eq. 2: the EMA scales it by alpha^2
    if dtype == "f32":
        B.wash_shuffle(c.gpu.ctx, 0, 0.5, None, seed=1)
        after = torch.zeros(N, dtype=torch.float64, device="cuda")
        B.wash_consensus_sq(c.gpu.ctx, B.WASH_STACK_PARAMS, 0, len(RAGGED), after)
        assert abs(after.sum().item() / want.sum() - 1) < 1e-12
        B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, 0.9)
        ema = torch.zeros(N, dtype=torch.float64, device="cuda")
        B.wash_consensus_sq(c.gpu.ctx, B.WASH_STACK_PARAMS, 0, len(RAGGED), ema)
        assert abs(ema.sum().item() / after.sum().item() - float(np.float32(0.9)) ** 2) < 1e-5
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N,dtype,opt_dtype,stacks", [(5, "f32", "f32", 2), (8, "bf16", "f32", 2), (13, "f32", None, 0),
                                                     (3, "f32", "bf16", 1), (40, "f32", None, 0), (2, "bf16", None, 0)])
def test_consensus_distance_inside_the_streaming_shuffle(N, dtype, opt_dtype, stacks, layout):
    """wash_shuffle_consensus: the stacks end as after the plain shuffle (bit-exact against the
    oracle), and the per-model, per-range sums equal the oracle's on the stack as it was before
    the step (1e-12 relative: binary64 sums in another order) and the standalone kernel's."""
    numel = [70001, 33, 7, 1, 4, 8, 5003, 2048, 30000]
    p_layer = [0.3, 1.0, 0.5, 1.0, 0.0, 0.9, 0.05, 0.01, 0.002]
    c = Case(N, numel, layout, dtype, opt_dtype, seed=N)
    measured = c.host_opt if stacks == 1 else c.host          # the first stack of the launch
    measured_code = B.WASH_STACK_OPT if stacks == 1 else B.WASH_STACK_PARAMS
    bounds = [1, 3, 3, 7, 9]                                      # four ranges, one empty, tensor 0 in none
    for step in (0, 1):
        want = np.stack([oracle.consensus_sq(c.ora, measured, lo, hi) for lo, hi in zip(bounds[:-1], bounds[1:])])
        alone = torch.zeros(len(bounds) - 1, N, dtype=torch.float64, device="cuda")
        for r, (lo, hi) in enumerate(zip(bounds[:-1], bounds[1:])):
            B.wash_consensus_sq(c.gpu.ctx, measured_code, lo, hi, alone[r])
        out = torch.zeros(len(bounds) - 1, N, dtype=torch.float64, device="cuda")
        B.wash_shuffle_consensus(c.gpu.ctx, stacks, step, 0.0, p_layer, seed=5, stats=c.stats_dev, tensor_bounds=bounds, dev_sq_out=out)
        st = oracle.shuffle(c.ora, c.host_opt if stacks == 1 else c.host, p_layer, seed=5, step=step,
                            stack2=c.host_opt if stacks == 2 else None)
        c.assert_equal("step %d" % step)
        got = out.cpu().numpy()
        assert np.allclose(got, want, rtol=1e-12, atol=0), (got, want)
        assert np.allclose(got, alone.cpu().numpy(), rtol=1e-12, atol=0)
        assert (got[1] == 0).all() and (got[0] > 0).all()
    # the whole model as one range, accumulated on top of what the array holds
    whole = torch.full((1, N), 1.0, dtype=torch.float64, device="cuda")
    want = oracle.consensus_sq(c.ora, measured)
    B.wash_shuffle_consensus(c.gpu.ctx, stacks, 2, 0.0, p_layer, seed=5, tensor_bounds=[0, len(numel)], dev_sq_out=whole)
    oracle.shuffle(c.ora, c.host_opt if stacks == 1 else c.host, p_layer, seed=5, step=2, stack2=c.host_opt if stacks == 2 else None)
    c.assert_equal("whole model")
    assert np.allclose(whole.cpu().numpy()[0] - 1.0, want, rtol=1e-11, atol=0)
    for bad in ([0], [3, 2], [0, len(numel) + 1], list(range(10))):
        with pytest.raises(B.WashError) as e:
            B.wash_shuffle_consensus(c.gpu.ctx, stacks, 3, 0.1, None, tensor_bounds=bad, dev_sq_out=whole)
        assert e.value.code == B.WASH_ERR_ARG
    c.close()


def test_consensus_inside_the_shuffle_at_config2_size():
    """ResNet-18 population of config 2: per quarter of the tensor table (Fig. 4) from one pass."""
    cfg = W.CONFIGS["cfg2_resnet18_n5"]
    table = W.table_from_spec(cfg["table"])
    N, T = cfg["N"], len(table)
    c = Case(N, W.numels(table), 0, "f32", "f32", dense=W.init_population(table, N, seed=0), dense_opt=W.init_momentum(table, N, seed=1))
    oracle.set_threads(oracle.max_threads())
    bounds = [0, T // 4, T // 2, 3 * T // 4, T]
    want = np.stack([oracle.consensus_sq(c.ora, c.host, lo, hi) for lo, hi in zip(bounds[:-1], bounds[1:])])
    out = torch.zeros(4, N, dtype=torch.float64, device="cuda")
    B.wash_shuffle_consensus(c.gpu.ctx, B.WASH_STACK_BOTH, 0, cfg["p"], None, seed=0, stats=c.stats_dev, tensor_bounds=bounds, dev_sq_out=out)
    st = oracle.shuffle(c.ora, c.host, cfg["p"], seed=0, step=0, stack2=c.host_opt)
    c.assert_equal("cfg2")
    assert c.gpu_stats() == st
    # The oracle adds a range's d terms one after the other in binary64 (a priori error d u,
    # u = 2^-53, of a sum of positive terms); the kernel adds them in another order.  Hence
    # the bar d u per range (2e-10 for the largest quarter), not the 1e-12 of the small cases.
    got = out.cpu().numpy()
    cum = np.concatenate([[0], np.cumsum(c.numel)])
    for r, (lo, hi) in enumerate(zip(bounds[:-1], bounds[1:])):
        d = float(cum[hi] - cum[lo])
        assert np.allclose(got[r], want[r], rtol=max(1e-12, d * 2.0 ** -53), atol=0), (r, got[r], want[r])
    oracle.set_threads(1)
    c.close()


def test_step_over_host_buffers():
    N, numel = 5, [3000, 17, 64]
    c = Case(N, numel, 0, "f32", "f32", seed=12)
    hp = torch.from_numpy(c.host.reshape(-1).copy()).pin_memory()
    ho = torch.from_numpy(c.host_opt.reshape(-1).copy()).pin_memory()
    havg = torch.zeros(c.P, dtype=torch.float32).pin_memory()
    ops = B.WASH_OP_SHUFFLE | B.WASH_OP_EMA | B.WASH_OP_AVERAGE
    st = B.wash_step_host(c.gpu.ctx, ops, hp, ho, havg, 3, 0.25, None, seed=4, alpha=0.99)
    want_st = oracle.shuffle(c.ora, c.host, 0.25, seed=4, step=3, stack2=c.host_opt)
    oracle.papa_ema(c.ora, c.host, 0.99)
    want_avg = np.zeros(c.P, dtype=np.float32)
    oracle.population_average(c.ora, c.host, want_avg)
    assert st == want_st
    assert (hp.numpy().view(np.uint32) == bits(c.host)).all()
    assert (ho.numpy().view(np.uint32) == bits(c.host_opt)).all()
    assert (havg.numpy().view(np.uint32) == want_avg.view(np.uint32)).all()
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_step_over_host_buffers_pipelined(dtype, layout):
    """A population large enough for wash_step_host to cut it into coordinate ranges whose
    copies and kernels overlap: the result must not depend on that."""
    N, numel = 3, [700001, 9, 400000, 77]
    c = Case(N, numel, layout, dtype, "f32", seed=14)
    assert c.P // 4 >= 1 << 18
    def pinned(a):
        t = torch.from_numpy(a.reshape(-1).view(np.int16).copy() if a.dtype == np.uint16 else a.reshape(-1).copy())
        return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).pin_memory()
    hp, ho = pinned(c.host), pinned(c.host_opt)
    havg = torch.zeros(c.P, dtype=hp.dtype).pin_memory()
    ops = B.WASH_OP_SHUFFLE | B.WASH_OP_EMA | B.WASH_OP_AVERAGE
    pl = [0.02, 1.0, 0.3, 0.0]
    for step in (5, 6):
        st = B.wash_step_host(c.gpu.ctx, ops, hp, ho, havg, step, 0.0, pl, seed=4, alpha=0.99)
        want_st = oracle.shuffle(c.ora, c.host, pl, seed=4, step=step, stack2=c.host_opt)
        oracle.papa_ema(c.ora, c.host, 0.99)
        want_avg = np.zeros(c.P, dtype=c.host.dtype)
        oracle.population_average(c.ora, c.host, want_avg)
        assert st == want_st
        assert (to_host_bits(hp) == bits(c.host)).all()
        assert (to_host_bits(ho) == bits(c.host_opt)).all()
        assert (to_host_bits(havg) == bits(want_avg)).all()
    B.wash_check(c.gpu.ctx)
    c.close()


def test_host_step_average_requested_on_a_later_call():
    """The pipeline's copy streams are set up by the first call; a later call that asks for
    the average for the first time must leave them usable."""
    N, numel = 2, [1 << 20, 12]
    c = Case(N, numel, 0, "f32", None, seed=15)
    hp = torch.from_numpy(c.host.reshape(-1).copy()).pin_memory()
    havg = torch.zeros(c.P, dtype=torch.float32).pin_memory()
    st = B.wash_step_host(c.gpu.ctx, B.WASH_OP_SHUFFLE, hp, None, None, 0, 0.01, None, seed=9, alpha=0.5)
    assert st == oracle.shuffle(c.ora, c.host, 0.01, seed=9, step=0)
    for step in (1, 2):
        st = B.wash_step_host(c.gpu.ctx, B.WASH_OP_SHUFFLE | B.WASH_OP_AVERAGE, hp, None, havg, step, 0.01, None, seed=9, alpha=0.5)
        assert st == oracle.shuffle(c.ora, c.host, 0.01, seed=9, step=step)
        want_avg = np.zeros(c.P, dtype=np.float32)
        oracle.population_average(c.ora, c.host, want_avg)
        assert (hp.numpy().view(np.uint32) == bits(c.host)).all()
        assert (havg.numpy().view(np.uint32) == want_avg.view(np.uint32)).all()
    B.wash_check(c.gpu.ctx)
    c.close()
