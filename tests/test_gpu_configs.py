"""GPU parity at the benchmark's full sizes: the ResNet populations of configs 2-4 in the
launch configurations bench.py times (streaming, sparse and automatic mode, default launch
shape), compared with the oracle bit for bit; config 5's parity grid (2^20 coordinates, every
N, p and layout of the sweep, host-generated values); and multi-gigabyte flat populations of
config 5 checked on sampled coordinate ranges that the oracle recomputes on its own."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_17517_b200 import binding as B
from paper_2405_17517_b200 import workloads as W
from gpu_util import Case, bits, to_host_bits

pytestmark = pytest.mark.gpu


def _resnet_case(name):
    cfg = W.CONFIGS[name]
    table = W.table_from_spec(cfg["table"])
    N = cfg["N"]
    dense = W.init_population(table, N, seed=0)
    mom = W.init_momentum(table, N, seed=1)
    c = Case(N, W.numels(table), 0, cfg["dtype"], "f32", dense=dense, dense_opt=mom)
    return cfg, c, len(table)


MODES = [B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE, B.WASH_MODE_AUTO]
MODE_IDS = ["stream", "sparse", "auto"]


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_config2_resnet18_n5_full_size(mode):
    cfg, c, T = _resnet_case("cfg2_resnet18_n5")
    B.wash_set_mode(c.gpu.ctx, mode)
    oracle.set_threads(oracle.max_threads())
    tot = [0, 0]
    for step in range(4):
        B.wash_shuffle_both(c.gpu.ctx, step, cfg["p"], None, seed=0, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, cfg["p"], seed=0, step=step, stack2=c.host_opt)
        tot[0] += s[0]; tot[1] += s[1]
    c.assert_equal("cfg2 shuffle")
    assert c.gpu_stats() == tuple(tot)
    B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, 0.99)
    oracle.papa_ema(c.ora, c.host, 0.99)
    c.assert_equal("cfg2 ema")
    out = torch.zeros(c.P, dtype=torch.float32, device="cuda")
    B.population_average(c.gpu.ctx, B.WASH_STACK_PARAMS, out, B.WASH_F32)
    want = np.zeros(c.P, dtype=np.float32)
    oracle.population_average(c.ora, c.host, want)
    assert (to_host_bits(out) == want.view(np.uint32)).all()
    oracle.set_threads(1)
    c.close()


@pytest.mark.parametrize("mode,steps", [(B.WASH_MODE_STREAM, 1000), (B.WASH_MODE_SPARSE, 50), (B.WASH_MODE_AUTO, 50)], ids=MODE_IDS)
def test_config3_resnet50_n10_per_layer_p_many_steps(mode, steps):
    """N = 10, 161 tensors, p_t = 0.01 (1 - t/160), momentum shuffled along, 1000 steps in the
    streaming mode (50 in the others); compared at steps 0, 1, 10, 100 (where reached) and the
    last, counters at the end."""
    cfg, c, T = _resnet_case("cfg3_resnet50_n10")
    B.wash_set_mode(c.gpu.ctx, mode)
    oracle.set_threads(oracle.max_threads())
    pl = B.wash_layer_probs(T, cfg["p"], B.WASH_SCHEDULE_DECREASING)
    assert np.array_equal(pl, oracle.layer_probs(T, cfg["p"]))
    tot = [0, 0]
    for step in range(steps):
        B.wash_shuffle_both(c.gpu.ctx, step, cfg["p"], pl, seed=3, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, pl, seed=3, step=step, stack2=c.host_opt)
        tot[0] += s[0]; tot[1] += s[1]
        if step in (0, 1, 10, 100, steps - 1):
            c.assert_equal("cfg3 step %d" % step)
    assert c.gpu_stats() == tuple(tot)
    # the paper's communicated fraction for this schedule, measured: sum_t q_t d_t / P per step
    numel = np.asarray(c.numel, dtype=np.float64)
    expect = (np.floor(pl * 2.0 ** 32) / 2.0 ** 32 * numel).sum() * steps
    assert abs(tot[0] - expect) < 5 * np.sqrt(expect)
    oracle.set_threads(1)
    c.close()


@pytest.mark.parametrize("mode", MODES, ids=MODE_IDS)
def test_config4_resnet50_bf16_weights_fp32_momentum(mode):
    cfg, c, T = _resnet_case("cfg4_resnet50_bf16_n8")
    B.wash_set_mode(c.gpu.ctx, mode)
    oracle.set_threads(oracle.max_threads())
    tot = [0, 0]
    for step in range(3):
        B.wash_shuffle_both(c.gpu.ctx, step, cfg["p"], None, seed=5, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, cfg["p"], seed=5, step=step, stack2=c.host_opt)
        tot[0] += s[0]; tot[1] += s[1]
    c.assert_equal("cfg4 shuffle")
    assert c.gpu_stats() == tuple(tot)
    for alpha in (0.999, 0.001):
        B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, alpha)
        oracle.papa_ema(c.ora, c.host, alpha)
        c.assert_equal("cfg4 ema %g" % alpha)
    for code, np_dtype, t_dtype in ((B.WASH_F32, np.float32, torch.float32), (B.WASH_BF16, np.uint16, torch.bfloat16)):
        out = torch.zeros(c.P, dtype=t_dtype, device="cuda")
        B.population_average(c.gpu.ctx, B.WASH_STACK_PARAMS, out, code)
        want = np.zeros(c.P, dtype=np_dtype)
        oracle.population_average(c.ora, c.host, want)
        assert (to_host_bits(out) == bits(want)).all()
    oracle.set_threads(1)
    c.close()


@pytest.mark.parametrize("mode", [B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE], ids=["stream", "sparse"])
@pytest.mark.parametrize("layout", [0, 1], ids=["NP", "PN"])
@pytest.mark.parametrize("p", [1e-4, 1e-3, 1e-2, 0.1, 1.0])
@pytest.mark.parametrize("N", [2, 4, 8, 16, 32])
def test_config5_parity_grid(N, p, layout, mode):
    """Config 5's parity cells: one flat fp32 tensor of 2^20 coordinates per model, values
    0.05 randn generated on the host, every N, p and layout of the sweep in both kernels;
    the whole stack and the counters compared with the oracle after two steps."""
    P = 1 << 20
    c = Case(N, [P], layout, dense=W.flat_population(N, P, seed=100 + N, std=0.05))
    B.wash_set_mode(c.gpu.ctx, mode)
    oracle.set_threads(oracle.max_threads())
    tot = [0, 0]
    for step in (0, 1):
        B.wash_shuffle(c.gpu.ctx, step, p, None, seed=55, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, p, seed=55, step=step)
        tot[0] += s[0]; tot[1] += s[1]
    c.assert_equal("N=%d p=%g layout=%d mode=%d" % (N, p, layout, mode))
    assert c.gpu_stats() == tuple(tot)
    oracle.set_threads(1)
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N,logP,p", [(8, 27, 0.01), (32, 24, 0.1), (2, 27, 1.0)])
def test_config5_large_flat_population_on_sampled_ranges(N, logP, p, layout):
    """A flat fp32 population far larger than L2 (up to 4.3 GB), generated on the device.
    64 random coordinate ranges are copied out before and after the shuffle; the oracle
    shuffles each range on its own (segment of tensor 0 starting at that coordinate) and
    must reproduce it.  The counters are checked against the binomial law."""
    P = 1 << logP
    pop = B.Population(N, [P], layout, 0)
    gen = torch.Generator(device="cuda").manual_seed(1234 + N)
    stack = torch.randn(N * pop.padded_P, generator=gen, device="cuda", dtype=torch.float32) * 0.05
    pop.bind(B.WASH_STACK_PARAMS, stack)
    view = stack.view(N, P) if layout == 0 else stack.view(P, N).t()
    rng = np.random.default_rng(7)
    starts = (rng.integers(0, (P - 4096) // 4, 62) * 4).tolist() + [0, P - 4096]
    before = [view[:, s:s + 4096].contiguous().cpu().numpy() for s in starts]
    stats = torch.zeros(2, dtype=torch.int64, device="cuda")
    B.wash_shuffle(pop.ctx, 17, p, None, seed=99, stats=stats)
    torch.cuda.synchronize()
    B.wash_check(pop.ctx)
    for s, b in zip(starts, before):
        seg = oracle.Population(N, [4096], tensor_id=[0], coord_begin=[s])
        want = np.ascontiguousarray(b)
        oracle.shuffle(seg, want, p, seed=99, step=17)
        got = view[:, s:s + 4096].contiguous().cpu().numpy()
        assert (got.view(np.uint32) == want.view(np.uint32)).all(), s
    sel = int(stats[0])
    q = oracle.threshold(p) / 2.0 ** 32
    assert abs(sel - P * q) <= 5 * np.sqrt(P * q * (1 - q)) + 1e-9
    pop.close()


def test_row_of_more_than_two_to_the_31_coordinates():
    """Largest rows: one tensor of 2^31 + 24 coordinates per model (N = 2, 17 GB).  Byte
    offsets exceed 2^32 and coordinate indices 2^31; sampled ranges, among them the last
    coordinates of the row, must match the oracle."""
    free, _ = torch.cuda.mem_get_info()
    P, N = (1 << 31) + 24, 2
    if free < N * P * 4 + (2 << 30):
        pytest.skip("not enough free device memory for a 17 GB stack")
    pop = B.Population(N, [P], B.WASH_LAYOUT_NP, 0)
    gen = torch.Generator(device="cuda").manual_seed(5)
    stack = torch.empty(N * pop.padded_P, device="cuda", dtype=torch.float32)
    for n in range(N):     # fill in pieces: randn of 2^31 elements at once needs a second buffer of that size
        for lo in range(0, pop.padded_P, 1 << 28):
            hi = min(pop.padded_P, lo + (1 << 28))
            stack[n * pop.padded_P + lo:n * pop.padded_P + hi].normal_(0.0, 0.05, generator=gen)
    pop.bind(B.WASH_STACK_PARAMS, stack)
    view = stack.view(N, pop.padded_P)
    rng = np.random.default_rng(3)
    starts = (rng.integers(0, (P - 4096) // 4, 20) * 4).tolist() + [0, (1 << 31) - 2048, P - 4096, P - 24 - 4072]
    before = [view[:, s:s + 4096].contiguous().cpu().numpy() for s in starts]
    stats = torch.zeros(2, dtype=torch.int64, device="cuda")
    for mode in (B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE):
        B.wash_set_mode(pop.ctx, mode)
        B.wash_shuffle(pop.ctx, 1 + mode, 0.01, None, seed=21, stats=stats)
    torch.cuda.synchronize()
    B.wash_check(pop.ctx)
    for s, b in zip(starts, before):
        width = min(4096, P - s)
        seg = oracle.Population(N, [width], tensor_id=[0], coord_begin=[s])
        want = np.ascontiguousarray(b[:, :width])
        for mode in (B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE):
            oracle.shuffle(seg, want, 0.01, seed=21, step=1 + mode)
        got = view[:, s:s + width].contiguous().cpu().numpy()
        assert (got.view(np.uint32) == want.view(np.uint32)).all(), s
    q = oracle.threshold(0.01) / 2.0 ** 32
    assert abs(int(stats[0]) - 2 * P * q) <= 5 * np.sqrt(2 * P * q)
    pop.close()


def test_segment_at_the_top_of_the_coordinate_and_tensor_ranges():
    """Counters near their limits: a shard holding the last 4096 coordinates of a tensor of
    2^32 coordinates whose index is 2^32 - 1, at a step just below 2^56."""
    N = 6
    c = Case(N, [4096, 100], 0, "f32", "f32", seed=2, tensor_id=[0xFFFFFFFF, 7], coord_begin=[(1 << 32) - 4096, 8])
    step = (1 << 56) - 1
    B.wash_shuffle_both(c.gpu.ctx, step, 0.5, None, seed=0xFFFFFFFFFFFFFFFF, stats=c.stats_dev)
    st = oracle.shuffle(c.ora, c.host, 0.5, seed=0xFFFFFFFFFFFFFFFF, step=step, stack2=c.host_opt)
    c.assert_equal("top of ranges")
    assert c.gpu_stats() == st
    c.close()
