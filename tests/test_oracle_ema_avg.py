"""Pins for the oracle's PAPA EMA (Eq. 1, Eq. 2), final average, layer schedule."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2405_17517_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
EPS = 2.0 ** -24          # unit roundoff of binary32


def _pop(N, numel, layout=0):
    off, P = W.padded_offsets(numel)
    return oracle.Population(N, numel, off, P, layout), off, P


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N,alpha", [(2, 0.5), (3, 0.99), (5, 0.01), (10, 0.999), (8, 0.001)])
def test_ema_against_binary64_statement_of_eq1(N, alpha, layout):
    numel = [1001, 7, 64]
    pop, off, P = _pop(N, numel, layout)
    dense = W.flat_population(N, sum(numel), seed=3 * N, std=0.05)
    x = W.to_stack(dense, numel, off, P, layout)
    oracle.papa_ema(pop, x, alpha)
    got = W.from_stack(x, N, numel, off, P, layout).astype(np.float64)
    th = dense.astype(np.float64)
    a = float(np.float32(alpha))
    mean = th.mean(axis=0, keepdims=True)                       # numpy's binary64 mean
    want = a * th + (1.0 - a) * mean
    # N-1 additions, one division, two products, one sum, (1 - alpha) rounded once:
    bound = (N + 3) * EPS * (np.abs(th).sum(axis=0, keepdims=True) / N + np.abs(th)) * 1.01
    assert (np.abs(got - want) <= bound).all()
    # padding untouched
    pad = x.reshape(N, P)[:, 1001:1008] if layout == 0 else x.reshape(P, N)[1001:1008, :]
    assert np.isnan(pad).all()


def test_ema_contracts_consensus_distance_by_alpha_squared_and_keeps_the_mean():
    """Eq. 2."""
    N, numel, alpha = 5, [4096, 100], 0.9
    pop, off, P = _pop(N, numel)
    x = W.to_stack(W.flat_population(N, sum(numel), seed=8, std=1.0), numel, off, P)
    before = oracle.consensus_sq(pop, x).sum()
    mean_before = W.from_stack(x, N, numel, off, P).astype(np.float64).mean(axis=0)
    oracle.papa_ema(pop, x, alpha)
    after = oracle.consensus_sq(pop, x).sum()
    mean_after = W.from_stack(x, N, numel, off, P).astype(np.float64).mean(axis=0)
    a = float(np.float32(alpha))
    assert abs(after / before - a * a) < 1e-5
    assert np.abs(mean_after - mean_before).max() < 1e-6


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_consensus_distance_per_model_and_per_tensor_range(layout, dtype):
    """Fig. 2's quantity from its definition, written out per model with exact rational
    arithmetic on a small stack and with numpy's binary64 on a larger one: distinct models
    (a sum landing in another model's slot shows), a range that leaves out the first and the
    last tensor (an ignored bound shows), the plain unit scale (a constant factor shows)."""
    N, numel = 4, [5, 12, 3, 9, 6]
    pop, off, P = _pop(N, numel, layout)
    dense = W.flat_population(N, sum(numel), seed=21, std=1.0)
    dense *= (1.0 + np.arange(N, dtype=np.float32))[:, None]         # models at visibly different distances
    if dtype == "bf16":
        x = W.to_stack(W.to_bf16_bits(dense), numel, off, P, layout)
        vals = W.bf16_bits_to_f32(W.to_bf16_bits(dense))
    else:
        x = W.to_stack(dense, numel, off, P, layout)
        vals = dense
    bounds = np.concatenate([[0], np.cumsum(numel)])
    for lo, hi in ((0, 5), (1, 4), (2, 3), (4, 5), (3, 3)):
        got = oracle.consensus_sq(pop, x, lo, hi)
        cols = range(int(bounds[lo]), int(bounds[hi]))
        want = []
        for n in range(N):
            acc = Fraction(0)
            for i in cols:
                mean = sum(Fraction(float(vals[m, i])) for m in range(N)) / N
                acc += (Fraction(float(vals[n, i])) - mean) ** 2
            want.append(float(acc))
        assert np.allclose(got, want, rtol=1e-13, atol=0), (lo, hi, got, want)
        if hi > lo:
            assert len(set(np.round(got, 9))) == N                   # the models really differ
    # a larger stack against numpy, every model and two ranges
    N, numel = 7, [1000, 64, 333, 2048, 17]
    pop, off, P = _pop(N, numel, layout)
    dense = W.flat_population(N, sum(numel), seed=5, std=0.3) + np.linspace(-1, 1, N, dtype=np.float32)[:, None]
    x = W.to_stack(dense, numel, off, P, layout)
    th = dense.astype(np.float64)
    bounds = np.concatenate([[0], np.cumsum(numel)])
    for lo, hi in ((0, 5), (1, 4)):
        sl = th[:, bounds[lo]:bounds[hi]]
        want = ((sl - sl.mean(axis=0, keepdims=True)) ** 2).sum(axis=1)
        assert np.allclose(oracle.consensus_sq(pop, x, lo, hi), want, rtol=1e-11, atol=0)
    # Fig. 2's distance itself, (1/N) sum_n ||theta_n - mean||, for one hand-made case:
    # two models at +-1 on d coordinates are each sqrt(d) away from their mean
    pop2, off2, P2 = _pop(2, [16], layout)
    x2 = W.to_stack(np.stack([np.ones(16, np.float32), -np.ones(16, np.float32)]), [16], off2, P2, layout)
    assert oracle.consensus_sq(pop2, x2).tolist() == [16.0, 16.0]


def test_ema_special_cases():
    # N = 2, alpha = 1/2 on a coarse grid: every operation is exact, so the result is
    # exactly halfway between the model and the midpoint of the two
    pop, off, P = _pop(2, [512])
    rng = np.random.default_rng(0)
    dense = (rng.integers(-1000, 1000, (2, 512)) * 0.25).astype(np.float32)
    x = W.to_stack(dense, [512], off, P)
    oracle.papa_ema(pop, x, 0.5)
    mid = (dense[0].astype(np.float64) + dense[1]) / 2
    want = 0.5 * dense.astype(np.float64) + 0.5 * mid[None, :]
    assert (x.reshape(2, P).astype(np.float64) == want).all()
    # all models equal to v: v stays within one ulp
    pop, off, P = _pop(4, [256])
    v = W.flat_population(1, 256, seed=5)
    x = W.to_stack(np.repeat(v, 4, axis=0), [256], off, P)
    oracle.papa_ema(pop, x, 0.99)
    assert (np.abs(x.reshape(4, P) - v) <= np.spacing(np.abs(v))).all()
    with pytest.raises(ValueError):
        oracle.papa_ema(pop, x, 1.0)
    with pytest.raises(ValueError):
        oracle.papa_ema(pop, x, 0.0)


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N", [1, 2, 3, 7, 16])
def test_average_against_binary64_mean(N, layout):
    numel = [777, 12]
    pop, off, P = _pop(N, numel, layout)
    dense = W.flat_population(N, sum(numel), seed=N, std=0.05)
    x = W.to_stack(dense, numel, off, P, layout)
    out = np.full(P, np.nan, dtype=np.float32)
    oracle.population_average(pop, x, out)
    got = np.concatenate([out[o:o + d] for o, d in zip(off, numel)]).astype(np.float64)
    want = dense.astype(np.float64).mean(axis=0)
    bound = N * EPS * np.abs(dense.astype(np.float64)).sum(axis=0) / N * 1.01
    assert (np.abs(got - want) <= bound).all()
    assert np.isnan(out[777:784]).all()


def test_average_is_exact_on_a_coarse_grid_with_power_of_two_population():
    N, d = 8, 1000
    pop, off, P = _pop(N, [d])
    rng = np.random.default_rng(1)
    dense = (rng.integers(-512, 512, (N, d)) / 64.0).astype(np.float32)
    x = W.to_stack(dense, [d], off, P)
    out = np.zeros(P, dtype=np.float32)
    oracle.population_average(pop, x, out)
    want = [float(sum(Fraction(float(v)) for v in dense[:, i]) / N) for i in range(d)]
    assert out[:d].tolist() == want


def test_average_adds_in_index_order():
    # (big + -big) + small = small, but big + (-big + small) = 0 in binary32
    pop, off, P = _pop(3, [8])
    col = np.array([[1e20], [-1e20], [3.0]], dtype=np.float32)
    x = W.to_stack(np.repeat(col, 8, axis=1), [8], off, P)
    out = np.zeros(P, dtype=np.float32)
    oracle.population_average(pop, x, out)
    assert (out == np.float32(3.0) / np.float32(3.0)).all()
    x2 = W.to_stack(np.repeat(col[[2, 0, 1]], 8, axis=1), [8], off, P)
    oracle.population_average(pop, x2, out)
    assert (out == 0.0).all()


def test_papa_all_writes_the_average_into_every_model():
    N, numel = 5, [100, 9]
    pop, off, P = _pop(N, numel)
    x = W.to_stack(W.flat_population(N, 109, seed=2), numel, off, P)
    avg = np.zeros(P, dtype=np.float32)
    oracle.population_average(pop, x, avg)
    oracle.papa_all(pop, x)
    rows = x.reshape(N, P)
    for o, d in zip(off, numel):
        assert (rows[:, o:o + d] == avg[None, o:o + d]).all()
    assert oracle.consensus_sq(pop, x).sum() == 0.0


def test_bf16_rounding_is_round_to_nearest_even():
    # N = 1: the average of one model is the model, so a bf16 output shows the rounding.
    rng = np.random.default_rng(9)
    bits = rng.integers(0, 1 << 32, 200_000, dtype=np.uint64).astype(np.uint32)
    ties = ((rng.integers(0, 1 << 16, 5000, dtype=np.uint64).astype(np.uint32)) << 16) | np.uint32(0x8000)
    vals = np.concatenate([bits, ties, np.array([0, 0x80000000, 0x7F7FFFFF, 0x7F800000, 0xFF800000, 0x00000001],
                                                dtype=np.uint32)]).view(np.float32)
    d = vals.size
    pop = oracle.Population(1, [d])
    out = np.zeros(d, dtype=np.uint16)
    oracle.population_average(pop, vals.copy(), out)
    want = torch.from_numpy(vals.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    nan = np.isnan(vals)
    assert (out[~nan] == want[~nan]).all()
    assert np.isnan(W.bf16_bits_to_f32(out[nan])).all()
    # widening is exact: bf16 stack, fp32 output
    src = out[~nan][:1000].copy()
    pop = oracle.Population(1, [src.size])
    o32 = np.zeros(src.size, dtype=np.float32)
    oracle.population_average(pop, src, o32)
    assert (o32.view(np.uint32) == (src.astype(np.uint32) << 16)).all()


def test_bf16_stack_ema_and_average():
    N, d = 8, 2048
    pop, off, P = _pop(N, [d])
    dense = W.flat_population(N, d, seed=4)
    xb = W.to_stack(W.to_bf16_bits(dense), [d], off, P)
    wide = W.bf16_bits_to_f32(xb.reshape(N, P)[:, :d]).astype(np.float64)
    out = np.zeros(P, dtype=np.float32)
    oracle.population_average(pop, xb, out)
    assert np.abs(out[:d] - wide.mean(axis=0)).max() <= N * EPS * np.abs(wide).sum(axis=0).max() / N * 1.01
    outb = np.zeros(P, dtype=np.uint16)
    oracle.population_average(pop, xb, outb)
    want = W.to_bf16_bits(out[:d])
    assert (outb[:d] == want).all()
    oracle.papa_ema(pop, xb, 0.999)
    a = float(np.float32(0.999))
    ref = a * wide + (1 - a) * wide.mean(axis=0, keepdims=True)
    got = W.bf16_bits_to_f32(xb.reshape(N, P)[:, :d]).astype(np.float64)
    assert (np.abs(got - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-30).all()       # half an ulp of bf16 (+ fp32 noise)


def test_layer_schedule_endpoints_and_table1():
    """p_0 = p, p_{L-1} = 0, linear in between; averaged over equally sized layers it is
    p/2, which with PAPA's period T gives the ratios printed in Table 1."""
    for L in (2, 5, 62, 161):
        pr = oracle.layer_probs(L, 0.01)
        assert pr[0] == 0.01 and pr[-1] == 0.0
        assert np.allclose(np.diff(pr), -0.01 / (L - 1), rtol=1e-12, atol=0)
        assert (oracle.layer_probs(L, 0.01, oracle.SCHEDULE_CONSTANT) == 0.01).all()
        inc = oracle.layer_probs(L, 0.01, oracle.SCHEDULE_INCREASING)
        assert inc[0] == 0.0 and abs(inc[-1] - 0.01) < 1e-18 and np.allclose(inc, pr[::-1], rtol=1e-12)
    assert oracle.layer_probs(1, 0.3).tolist() == [0.3]
    with open(os.path.join(GOLDEN, "table1_comm_volume.txt")) as f:
        rows = [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 2
    for _, p, T, wash, wash_opt in rows:
        p, T = float(p), int(T)
        mean_p = oracle.layer_probs(101, p).mean()
        assert abs(mean_p * T - float(Fraction(wash))) < 1e-12
        assert abs(2 * mean_p * T - float(Fraction(wash_opt))) < 1e-12
    # and the shuffle itself moves that fraction when layers weigh the same
    L, d, N, p = 21, 20_000, 2, 0.05
    off, P = W.padded_offsets([d] * L)
    pop = oracle.Population(N, [d] * L, off, P)
    x = np.zeros(N * P, dtype=np.float32)
    sel, _ = oracle.shuffle(pop, x, oracle.layer_probs(L, p), seed=1, step=0)
    assert abs(sel / (L * d) - p / 2) < 5 * math.sqrt(p / 2 / (L * d))
