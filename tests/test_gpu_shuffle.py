"""GPU parity of the shuffling step: libwash.so (through its C ABI) against the oracle,
bit for bit, on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_17517_b200 import binding as B
from paper_2405_17517_b200 import workloads as W
from gpu_util import Case, bits, to_host_bits

pytestmark = pytest.mark.gpu

RAGGED = [1000, 33, 7, 1, 4, 8, 5003, 2048]       # several tiles, ragged tails, tiny tensors


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N", [2, 3, 4, 5, 6, 7, 8, 9, 10, 12, 16, 20, 24, 32, 33, 64])
def test_shuffle_fp32_matches_oracle(N, layout):
    c = Case(N, RAGGED, layout, seed=N)
    p_layer = [0.3, 1.0, 0.5, 1.0, 0.0, 0.9, 0.05, 0.01]
    for step in (0, 1, (7 << 32) | 5):
        B.wash_shuffle(c.gpu.ctx, step, 0.0, p_layer, seed=0xABCDEF0123456789, stats=c.stats_dev)
        sel, moved = oracle.shuffle(c.ora, c.host, p_layer, seed=0xABCDEF0123456789, step=step)
        c.assert_equal("N=%d layout=%d step=%d" % (N, layout, step))
    # counters accumulate over the three calls
    st = c.gpu_stats()
    c2 = Case(N, RAGGED, layout, seed=N)
    tot = [0, 0]
    for step in (0, 1, (7 << 32) | 5):
        s = oracle.shuffle(c2.ora, c2.host, p_layer, seed=0xABCDEF0123456789, step=step)
        tot[0] += s[0]; tot[1] += s[1]
    assert st == tuple(tot)
    c.close(); c2.close()


@pytest.mark.parametrize("mode", [B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE])
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N", [2, 3, 5, 7, 8, 9, 10, 16, 17, 32, 33, 64])
def test_both_kernels_on_many_tiles_match_oracle(N, layout, mode):
    """Both kernels (run-time N) on many tiles with a ragged last tile, both stacks,
    per-layer probabilities from never to always."""
    numel = [70001, 33, 7, 1, 4, 8, 5003, 2048, 300000 if N <= 16 else 30000]
    c = Case(N, numel, layout, "f32", "f32", seed=N)
    B.wash_set_mode(c.gpu.ctx, mode)
    p_layer = [0.3, 1.0, 0.5, 1.0, 0.0, 0.9, 0.05, 0.01, 0.002]
    tot = [0, 0]
    for step in (0, 1, (7 << 32) | 5):
        B.wash_shuffle_both(c.gpu.ctx, step, 0.0, p_layer, seed=0xABCDEF0123456789, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, p_layer, seed=0xABCDEF0123456789, step=step, stack2=c.host_opt)
        tot[0] += s[0]; tot[1] += s[1]
        c.assert_equal("N=%d layout=%d step=%d" % (N, layout, step))
    assert c.gpu_stats() == tuple(tot)
    c.close()


@pytest.mark.parametrize("mode", [B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE, B.WASH_MODE_AUTO])
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("dtype,opt_dtype", [("f32", "f32"), ("bf16", "f32"), ("bf16", "bf16"), ("f32", "bf16"), ("bf16", None)])
def test_shuffle_both_stacks_and_dtypes(dtype, opt_dtype, layout, mode):
    N = 5
    c = Case(N, RAGGED, layout, dtype, opt_dtype, seed=3)
    B.wash_set_mode(c.gpu.ctx, mode)
    for step in range(3):
        if opt_dtype is None:
            B.wash_shuffle(c.gpu.ctx, step, 0.2, None, seed=9, stats=c.stats_dev)
        else:
            B.wash_shuffle_both(c.gpu.ctx, step, 0.2, None, seed=9, stats=c.stats_dev)
        oracle.shuffle(c.ora, c.host, 0.2, seed=9, step=step, stack2=c.host_opt)
        c.assert_equal("step %d" % step)
    c.close()


@pytest.mark.parametrize("flavour", [-2, -3], ids=["lean", "early"])
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N,dtype,opt_dtype", [(5, "f32", "f32"), (16, "f32", None), (17, "f32", "f32"), (33, "bf16", "f32"), (64, "f32", None)])
def test_streaming_flavours_on_dense_and_mixed_selection(N, dtype, opt_dtype, layout, flavour):
    """The streaming kernel's two flavours (permutations drawn after or before the wait for the
    copies; the early one serves N > 16 densely from byte columns) on tensors that are selected
    in full, mostly, half, rarely and not at all, with ragged ends."""
    numel = [9000, 33, 4100, 7, 2600, 1, 5003]
    p_layer = [1.0, 1.0, 0.9, 0.5, 0.45, 1.0, 0.02]
    c = Case(N, numel, layout, dtype, opt_dtype, seed=40 + N)
    B.wash_set_launch(c.gpu.ctx, 0, flavour)
    tot = [0, 0]
    for step in (0, 1, (3 << 32) | 9):
        if opt_dtype is None:
            B.wash_shuffle(c.gpu.ctx, step, 0.0, p_layer, seed=123, stats=c.stats_dev)
        else:
            B.wash_shuffle_both(c.gpu.ctx, step, 0.0, p_layer, seed=123, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, p_layer, seed=123, step=step, stack2=c.host_opt)
        tot[0] += s[0]; tot[1] += s[1]
        c.assert_equal("N=%d layout=%d step=%d" % (N, layout, step))
    assert c.gpu_stats() == tuple(tot)
    c.close()


@pytest.mark.parametrize("code", [-4, -5, 0], ids=["resident", "one-trip", "default"])
@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N,dtype,opt_dtype", [(2, "f32", None), (2, "bf16", "f32"), (3, "f32", "f32"), (4, "bf16", None), (4, "f32", None), (8, "f32", None), (17, "bf16", "bf16")])
def test_resident_warp_streaming_kernel(N, dtype, opt_dtype, layout, code):
    """The streaming kernel for small groups (a resident grid of warps walking tiles with two
    shared-memory stages), forced, excluded and as the library chooses, against the oracle: enough
    coordinates for several trips per warp, tensors selected in full, half, rarely and not at
    all, ragged ends, a tensor boundary inside a tile."""
    numel = [2_600_003 if N <= 4 else 200_003, 33, 4100, 7, 260_000, 1, 5003, 90_001]
    p_layer = [0.004, 1.0, 0.9, 0.5, 0.3, 1.0, 0.0, 1.0]
    c = Case(N, numel, layout, dtype, opt_dtype, seed=70 + N)
    B.wash_set_launch(c.gpu.ctx, 0, code)
    tot = [0, 0]
    for step in (0, 1, (5 << 32) | 2):
        if opt_dtype is None:
            B.wash_shuffle(c.gpu.ctx, step, 0.0, p_layer, seed=77, stats=c.stats_dev)
        else:
            B.wash_shuffle_both(c.gpu.ctx, step, 0.0, p_layer, seed=77, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, p_layer, seed=77, step=step, stack2=c.host_opt)
        tot[0] += s[0]; tot[1] += s[1]
        c.assert_equal("N=%d layout=%d step=%d" % (N, layout, step))
    assert c.gpu_stats() == tuple(tot)
    B.wash_check(c.gpu.ctx)
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
def test_separate_calls_equal_the_fused_call(layout):
    N = 8
    a = Case(N, RAGGED, layout, "f32", "f32", seed=5)
    b = Case(N, RAGGED, layout, "f32", "f32", seed=5)
    B.wash_shuffle_both(a.gpu.ctx, 4, 0.5, None, seed=1, stats=a.stats_dev)
    B.wash_shuffle(b.gpu.ctx, 4, 0.5, None, seed=1, stats=b.stats_dev)
    B.wash_shuffle_opt_state(b.gpu.ctx, 4, 0.5, None, seed=1)
    torch.cuda.synchronize()
    assert torch.equal(a.dev.view(torch.int32), b.dev.view(torch.int32))
    assert torch.equal(a.dev_opt.view(torch.int32), b.dev_opt.view(torch.int32))
    assert a.gpu_stats() == b.gpu_stats()
    oracle.shuffle(a.ora, a.host, 0.5, seed=1, step=4, stack2=a.host_opt)
    a.assert_equal()
    a.close(); b.close()


@pytest.mark.parametrize("N", [3, 10, 11])
def test_sparse_mode_and_launch_shapes_give_the_same_bits(N):
    ref = Case(N, RAGGED, 0, seed=8)
    oracle.shuffle(ref.ora, ref.host, 0.1, seed=2, step=3)
    for mode in (B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE, B.WASH_MODE_AUTO):
        for threads, bps in ((0, 0), (64, 1), (128, 2), (256, -1), (96, 0), (32, 4), (256, 2), (128, 1), (0, -2), (0, -3), (128, -3), (0, -4), (0, -5)):
            c = Case(N, RAGGED, 0, seed=8)
            B.wash_set_mode(c.gpu.ctx, mode)
            B.wash_set_launch(c.gpu.ctx, threads, bps)
            B.wash_shuffle(c.gpu.ctx, 3, 0.1, None, seed=2)
            torch.cuda.synchronize()
            assert (to_host_bits(c.dev) == bits(ref.host)).all(), (mode, threads, bps)
            c.close()
    ref.close()


def test_edge_cases_p0_p1_single_element_and_padding():
    # p = 0: identity, nothing written; p = 1: everything selected
    c = Case(4, [1], 0, seed=1)
    B.wash_shuffle(c.gpu.ctx, 0, 0.0, None, seed=0, stats=c.stats_dev)
    c.assert_equal("p=0")
    assert c.gpu_stats() == (0, 0)
    B.wash_shuffle(c.gpu.ctx, 0, 1.0, None, seed=0, stats=c.stats_dev)
    sel, moved = oracle.shuffle(c.ora, c.host, 1.0, seed=0, step=0)
    c.assert_equal("p=1")     # compares the padding too: it must still hold its NaN pattern
    assert c.gpu_stats() == (1, moved) and sel == 1
    c.close()
    for numel in ([3], [4], [5], [8], [9], [31, 33], [1, 1, 1, 1]):
        for layout in (0, 1):
            c = Case(3, numel, layout, seed=2)
            B.wash_shuffle(c.gpu.ctx, 11, 1.0, None, seed=5)
            oracle.shuffle(c.ora, c.host, 1.0, seed=5, step=11)
            c.assert_equal(str(numel))
            c.close()


def test_last_layer_untouched_and_schedules_agree_with_oracle():
    numel = [640, 1280, 320, 2560, 100]
    c = Case(5, numel, 0, seed=4)
    before = to_host_bits(c.dev).reshape(5, c.P)[:, c.off[-1]:c.off[-1] + 100].copy()
    for sched in (0, 1, 2):
        assert np.array_equal(B.wash_layer_probs(len(numel), 0.4, sched), oracle.layer_probs(len(numel), 0.4, sched))
    pl = B.wash_layer_probs(len(numel), 0.4)
    for step in range(5):
        B.wash_shuffle(c.gpu.ctx, step, 0.4, pl, seed=step)
        oracle.shuffle(c.ora, c.host, pl, seed=step, step=step)
    c.assert_equal()
    after = to_host_bits(c.dev).reshape(5, c.P)[:, c.off[-1]:c.off[-1] + 100]
    assert (before == after).all()
    c.close()


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N", [2, 4])
def test_resident_warp_kernel_with_a_padded_coordinate_major_image(N, dtype):
    """[P][N] with an even N and a quarter of the coordinates selected: the shared-memory image is
    padded against bank conflicts while the small-group streaming kernel is still the one launched
    (forced here for N = 4 in fp32, whose groups it does not take by default)."""
    c = Case(N, [300_007, 12, 40_000], 1, dtype, None, seed=90 + N)
    B.wash_set_launch(c.gpu.ctx, 0, -4)
    tot = [0, 0]
    for step in (0, 1):
        B.wash_shuffle(c.gpu.ctx, step, 0.25, None, seed=5, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, 0.25, seed=5, step=step)
        tot[0] += s[0]; tot[1] += s[1]
        c.assert_equal("N=%d %s step=%d" % (N, dtype, step))
    assert c.gpu_stats() == tuple(tot)
    c.close()


@pytest.mark.parametrize("N", [2, 4])
def test_shards_reproduce_the_unsharded_shuffle(N):
    """Coordinate shards keyed by the global (tensor, coordinate) need no communication
    (N = 2 goes through the streaming kernel for small groups, N = 4 through the one-trip kernel)."""
    numel = [4000, 1000, 36]
    full = Case(N, numel, 0, seed=6)
    dense = W.from_stack(full.host, N, numel, full.off, full.P)
    oracle.shuffle(full.ora, full.host, 0.3, seed=77, step=5)
    want = W.from_stack(full.host, N, numel, full.off, full.P)
    # shard A: tensor 0 [0, 2000) ; shard B: tensor 0 [2000, 4000), tensor 1, tensor 2
    shards = [([2000], [0], [0], dense[:, :2000]),
              ([2000, 1000, 36], [0, 1, 2], [2000, 0, 0], dense[:, 2000:])]
    got = []
    for nm, tid, cb, d in shards:
        c = Case(N, nm, 0, tensor_id=tid, coord_begin=cb, dense=np.ascontiguousarray(d))
        B.wash_shuffle(c.gpu.ctx, 5, 0.3, None, seed=77)
        torch.cuda.synchronize()
        host = to_host_bits(c.dev).view(np.float32)
        got.append(W.from_stack(host, N, nm, c.off, c.P))
        c.close()
    assert (np.concatenate(got, axis=1).view(np.uint32) == want.view(np.uint32)).all()
    full.close()


def test_config1_hundred_steps_then_ema_and_average():
    """N = 3, one flat fp32 vector of 2^20 elements, N(0, 0.05), p = 0.01, 100 steps with
    the step index as the RNG counter; then PAPA's EMA and the final average."""
    N, d = 3, 1 << 20
    c = Case(N, [d], 0, dense=W.flat_population(N, d, seed=0, std=0.05))
    tot = [0, 0]
    for step in range(100):
        B.wash_shuffle(c.gpu.ctx, step, 0.01, None, seed=0, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, 0.01, seed=0, step=step)
        tot[0] += s[0]; tot[1] += s[1]
        if step < 10 or step == 99:
            c.assert_equal("step %d" % step)
    assert c.gpu_stats() == tuple(tot)
    for alpha in (0.99, 0.01):
        B.papa_ema(c.gpu.ctx, B.WASH_STACK_PARAMS, alpha)
        oracle.papa_ema(c.ora, c.host, alpha)
        c.assert_equal("ema %g" % alpha)     # designed to be bit-exact; the bar is 2 ulp
    out = torch.zeros(c.P, dtype=torch.float32, device="cuda")
    B.population_average(c.gpu.ctx, B.WASH_STACK_PARAMS, out, B.WASH_F32)
    want = np.zeros(c.P, dtype=np.float32)
    oracle.population_average(c.ora, c.host, want)
    assert (to_host_bits(out) == want.view(np.uint32)).all()
    c.close()


def test_argument_and_state_errors():
    ctx = B.wash_create(3, [100])
    with pytest.raises(B.WashError) as e:
        B.wash_shuffle(ctx, 0, 0.5)
    assert e.value.code == B.WASH_ERR_STATE
    P, _ = B.wash_stack_elems(ctx, 1)
    t = torch.zeros(3 * P, device="cuda")
    with pytest.raises(B.WashError) as e:
        B.wash_bind(ctx, 0, B.WASH_F32, t, 3 * P - 1)
    assert e.value.code == B.WASH_ERR_ARG
    B.wash_bind(ctx, 0, B.WASH_F32, t, 3 * P)
    for bad in (dict(p=1.5), dict(p=float("nan")), dict(p=-0.1), dict(p=0.5, step=1 << 56), dict(p=0.5, p_layer=[2.0])):
        with pytest.raises(B.WashError) as e:
            B.wash_shuffle(ctx, bad.get("step", 0), bad["p"], bad.get("p_layer"))
        assert e.value.code == B.WASH_ERR_ARG
    with pytest.raises(B.WashError) as e:
        B.wash_shuffle_both(ctx, 0, 0.5)
    assert e.value.code == B.WASH_ERR_STATE
    with pytest.raises(B.WashError):
        B.papa_ema(ctx, 0, 1.0)
    assert (t == 0).all()
    B.wash_check(ctx)
    B.wash_destroy(ctx)


def test_a_rejected_probability_vector_leaves_the_context_consistent():
    """A call refused for one bad entry of p_layer must not change the thresholds the next
    call compares with: the following valid call (which repeats the good entries) has to
    upload its table and match the oracle."""
    N, numel = 4, [3000, 2000, 500]
    c = Case(N, numel, 0, "f32", "f32", seed=13)
    B.wash_shuffle_both(c.gpu.ctx, 0, 0.0, [0.1, 0.1, 0.1], seed=3, stats=c.stats_dev)
    st = list(oracle.shuffle(c.ora, c.host, [0.1, 0.1, 0.1], seed=3, step=0, stack2=c.host_opt))
    for bad in ([0.5, 2.0, 0.0], [0.5, 0.25, float("nan")]):
        with pytest.raises(B.WashError) as e:
            B.wash_shuffle_both(c.gpu.ctx, 1, 0.0, bad, seed=3, stats=c.stats_dev)
        assert e.value.code == B.WASH_ERR_ARG
    c.assert_equal("after the refused calls")          # nothing ran
    for step, pl in ((1, [0.5, 0.0, 0.0]), (2, [0.5, 0.25, 0.0]), (3, [0.1, 0.1, 0.1])):
        B.wash_shuffle_both(c.gpu.ctx, step, 0.0, pl, seed=3, stats=c.stats_dev)
        s = oracle.shuffle(c.ora, c.host, pl, seed=3, step=step, stack2=c.host_opt)
        st[0] += s[0]; st[1] += s[1]
        c.assert_equal("step %d" % step)
    assert c.gpu_stats() == tuple(st)
    c.close()


def test_resume_from_a_host_copy_continues_bit_identically():
    """The shuffle is a pure function of (stack bits, seed, step, tensor table, p): 20 steps
    in one context equal 10 steps, a round trip of the stacks through host memory into a
    fresh context, and 10 more steps."""
    N, numel = 5, [3000, 17, 640]
    a = Case(N, numel, 0, "f32", "f32", seed=31)
    for step in range(20):
        B.wash_shuffle_both(a.gpu.ctx, step, 0.05, None, seed=77)
    b = Case(N, numel, 0, "f32", "f32", seed=31)
    for step in range(10):
        B.wash_shuffle_both(b.gpu.ctx, step, 0.05, None, seed=77)
    torch.cuda.synchronize()
    saved, saved_opt = b.dev.cpu(), b.dev_opt.cpu()
    b.close()
    c = Case(N, numel, 0, "f32", "f32", seed=99)          # different contents, overwritten below
    c.dev.copy_(saved); c.dev_opt.copy_(saved_opt)
    for step in range(10, 20):
        B.wash_shuffle_both(c.gpu.ctx, step, 0.05, None, seed=77)
    torch.cuda.synchronize()
    assert torch.equal(a.dev.view(torch.int32), c.dev.view(torch.int32))
    assert torch.equal(a.dev_opt.view(torch.int32), c.dev_opt.view(torch.int32))
    a.close(); c.close()


def test_auto_mode_takes_either_kernel_and_keeps_the_bits():
    """WASH_MODE_AUTO picks the sparse kernel below a share of expected selection (N = 6 in [N][P]:
    5.8 %) and the streaming one above; a per-layer vector is judged by its expectation over the whole model."""
    N = 6
    numel = [70000, 9, 3000]
    c = Case(N, numel, 0, "f32", "f32", seed=21)
    B.wash_set_mode(c.gpu.ctx, B.WASH_MODE_AUTO)
    for step, (p, pl) in enumerate([(0.001, None), (0.5, None), (0.0, [0.01, 1.0, 0.2]), (0.0, [0.2, 0.0, 0.0])]):
        B.wash_shuffle_both(c.gpu.ctx, step, p, pl, seed=77, stats=c.stats_dev)
        oracle.shuffle(c.ora, c.host, p if pl is None else pl, seed=77, step=step, stack2=c.host_opt)
        c.assert_equal("step %d" % step)
    c.close()


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_configurations_match_oracle(seed):
    """Seeded random draws of population size, layout, dtypes, tensor table, probabilities (uniform
    or per layer), kernel family and forced streaming flavour: stacks, padding and counters equal
    the oracle's after two steps each."""
    import random
    rng = random.Random(seed)
    for it in range(40):
        N = rng.choice([2, 2, 3, 3, 4, 4, 5, 6, 8, 9, 12, 16, 17, 24, 32, 33])
        layout = rng.randint(0, 1)
        dtype = rng.choice(["f32", "bf16"])
        opt = rng.choice([None, None, "f32", "bf16"])
        T = rng.randint(1, 6)
        big = rng.choice([20000, 200000, 700000 if N <= 8 else 60000])
        numel = [rng.choice([1, 3, 4, 5, 8, 31, 33, 260, 4099, rng.randint(1, big)]) for _ in range(T)]
        numel[rng.randrange(T)] = rng.randint(big // 2, big)
        mode = rng.choice([B.WASH_MODE_STREAM, B.WASH_MODE_STREAM, B.WASH_MODE_SPARSE, B.WASH_MODE_AUTO])
        code = rng.choice([0, 0, -4, -5, -2, -3])
        uniform = rng.random() < 0.5
        p = rng.choice([0.0005, 0.003, 0.01, 0.03, 0.1, 0.25, 0.6, 1.0]) if uniform else 0.0
        pl = None if uniform else [rng.choice([0.0, 0.002, 0.01, 0.05, 0.3, 1.0]) for _ in range(T)]
        what = "seed %d case %d: N=%d layout=%d %s/%s numel=%s mode=%d code=%d p=%s" % (seed, it, N, layout, dtype, opt, numel, mode, code, p if uniform else pl)
        c = Case(N, numel, layout, dtype, opt, seed=1000 * seed + it)
        B.wash_set_mode(c.gpu.ctx, mode)
        B.wash_set_launch(c.gpu.ctx, 0, code)
        tot = [0, 0]
        for step in (it, (it << 33) | 7):
            if opt is None:
                B.wash_shuffle(c.gpu.ctx, step, p, pl, seed=it * 77 + 1, stats=c.stats_dev)
            else:
                B.wash_shuffle_both(c.gpu.ctx, step, p, pl, seed=it * 77 + 1, stats=c.stats_dev)
            s = oracle.shuffle(c.ora, c.host, p if uniform else pl, seed=it * 77 + 1, step=step, stack2=c.host_opt)
            tot[0] += s[0]; tot[1] += s[1]
            c.assert_equal(what)
        assert c.gpu_stats() == tuple(tot), what
        B.wash_check(c.gpu.ctx)
        c.close()
