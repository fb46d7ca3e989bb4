"""Pins for the oracle's shuffling step (Eq. 3-5, Algorithm 1) -- CPU only."""
import itertools
import math
from fractions import Fraction

import numpy as np
import pytest

import oracle
from paper_2405_17517_b200 import workloads as W


def _pop(N, numel, layout=0, **kw):
    off, P = W.padded_offsets(numel)
    return oracle.Population(N, numel, off, P, layout, **kw), off, P


def _sentinel(N, P):
    """theta[n][i] = n: after a shuffle, column i spells pi_i (gather form)."""
    return np.repeat(np.arange(N, dtype=np.float32)[:, None], P, axis=1).copy()


def _chi2_quantile_999(dof):
    # Wilson-Hilferty approximation of the 99.9 % quantile
    z = 3.0902
    return dof * (1 - 2 / (9 * dof) + z * math.sqrt(2 / (9 * dof))) ** 3


def test_p_zero_is_identity_and_p_one_selects_everything():
    pop, off, P = _pop(4, [37, 5, 64])
    x = W.to_stack(W.flat_population(4, 106, seed=1), pop.numel, off, P)
    y = x.copy()
    assert oracle.shuffle(pop, y, 0.0, seed=3, step=0) == (0, 0)
    assert y.view(np.uint32).tolist() == x.view(np.uint32).tolist()
    sel, moved = oracle.shuffle(pop, y, 1.0, seed=3, step=0)
    assert sel == 106 and 0 < moved <= 4 * 106
    # padding untouched (NaN pattern), logical part changed somewhere
    assert np.isnan(y.reshape(4, P)[:, 37:40]).all()
    assert (W.from_stack(y, 4, pop.numel, off, P) != W.from_stack(x, 4, pop.numel, off, P)).any()


@pytest.mark.parametrize("layout", [0, 1])
@pytest.mark.parametrize("N", [2, 3, 5, 8])
def test_multiset_per_coordinate_is_preserved(N, layout):
    """Eq. 5: the N values of a coordinate are only permuted, so its sorted column, the
    population mean and the consensus distance cannot change."""
    numel = [1000, 33, 7]
    pop, off, P = _pop(N, numel, layout)
    dense = W.flat_population(N, sum(numel), seed=N)
    x = W.to_stack(dense, numel, off, P, layout)
    y = x.copy()
    sel, moved = oracle.shuffle(pop, y, 0.3, seed=11, step=5)
    a = W.from_stack(x, N, numel, off, P, layout)
    b = W.from_stack(y, N, numel, off, P, layout)
    assert (np.sort(a.view(np.uint32), axis=0) == np.sort(b.view(np.uint32), axis=0)).all()
    changed = (a.view(np.uint32) != b.view(np.uint32))
    assert changed.any(axis=0).sum() <= sel           # only selected coordinates change
    assert changed.sum() == moved                     # distinct values: every moved value shows
    # consensus distance (Eq. 5) in exact arithmetic on a few columns
    for i in np.flatnonzero(changed.any(axis=0))[:20]:
        ca = [Fraction(float(v)) for v in a[:, i]]
        cb = [Fraction(float(v)) for v in b[:, i]]
        ma, mb = sum(ca) / N, sum(cb) / N
        assert ma == mb
        assert sum((v - ma) ** 2 for v in ca) == sum((v - mb) ** 2 for v in cb)


def test_layouts_give_the_same_logical_result():
    N, numel = 5, [513, 40, 9]
    dense = W.flat_population(N, sum(numel), seed=2)
    res = []
    for layout in (0, 1):
        pop, off, P = _pop(N, numel, layout)
        x = W.to_stack(dense, numel, off, P, layout)
        st = oracle.shuffle(pop, x, [0.2, 0.5, 1.0], seed=9, step=77)
        res.append((st, W.from_stack(x, N, numel, off, P, layout)))
    assert res[0][0] == res[1][0]
    assert (res[0][1].view(np.uint32) == res[1][1].view(np.uint32)).all()


def test_selected_fraction_follows_the_binomial_law():
    N, d = 2, 400_000
    pop, off, P = _pop(N, [d])
    for p in (0.001, 0.01, 0.1, 0.5):
        x = _sentinel(N, P)
        sel, _ = oracle.shuffle(pop, x, p, seed=5, step=1)
        q = oracle.threshold(p) / 2 ** 32
        assert abs(sel - d * q) < 5 * math.sqrt(d * q * (1 - q)), (p, sel)


def test_mask_lanes_of_a_group_are_uncorrelated():
    # coordinates 4g .. 4g+3 share one Philox block; their decisions must still be independent
    d, p = 200_000, 0.5
    thr = oracle.threshold(p)
    sel = np.array([oracle.mask_word(7, 3, 0, i) < thr for i in range(d)]).reshape(-1, 4)
    for a, b in itertools.combinations(range(4), 2):
        both = (sel[:, a] & sel[:, b]).sum()
        n = sel.shape[0]
        assert abs(both - n / 4) < 5 * math.sqrt(n * 3 / 16)


@pytest.mark.parametrize("N", [3, 4, 5])
def test_permutations_are_uniform_over_all_of_them(N):
    """Eq. 3 / the sentence after it: pi_i is uniform on the N! permutations (fixed points
    and the identity included).  The sentinel stack makes each pi_i readable."""
    d = 120_000
    pop, off, P = _pop(N, [d])
    x = _sentinel(N, P)
    sel, moved = oracle.shuffle(pop, x, 1.0, seed=2024, step=3)
    assert sel == d
    cols = x.reshape(N, P)[:, :d].astype(np.int64)
    assert (np.sort(cols, axis=0) == np.arange(N)[:, None]).all()      # each column a permutation
    code = sum(cols[n] * N ** n for n in range(N))
    counts = np.array([np.count_nonzero(code == sum(pi[n] * N ** n for n in range(N)))
                       for pi in itertools.permutations(range(N))])
    assert counts.sum() == d
    exp = d / math.factorial(N)
    chi2 = ((counts - exp) ** 2 / exp).sum()
    assert chi2 < _chi2_quantile_999(math.factorial(N) - 1), chi2
    # a uniform permutation has one fixed point on average
    assert abs(moved / d - (N - 1)) < 5 * math.sqrt(1.0 / d)
    assert moved == int((cols != np.arange(N)[:, None]).sum())


def test_gather_direction_and_draw_match_the_exposed_permutation():
    N, d = 6, 300
    pop, off, P = _pop(N, [d])
    x = _sentinel(N, P)
    oracle.shuffle(pop, x, 1.0, seed=8, step=12)
    cols = x.reshape(N, P)[:, :d].astype(int)
    for i in (0, 1, 2, 3, 4, 150, 299):
        assert cols[:, i].tolist() == oracle.draw_permutation(8, 12, 0, i, N)     # new[n] = old[pi(n)]


def test_fisher_yates_restated_from_its_words():
    # textbook Fisher-Yates (Durstenfeld), top index first, j = floor(word * (k+1) / 2^32)
    for N in (2, 3, 7, 16, 33):
        for i in (0, 5, 123456):
            perm = list(range(N))
            for k in range(N - 1, 0, -1):
                w = oracle.perm_word(99, 4, 2, i, N - 1 - k)
                j = (w * (k + 1)) >> 32
                perm[k], perm[j] = perm[j], perm[k]
            assert perm == oracle.draw_permutation(99, 4, 2, i, N)


def test_mask_and_permutation_are_independent():
    # contingency of "mask word below the median" against "which permutation" for N = 3
    N, d = 3, 120_000
    below = np.array([oracle.mask_word(1, 0, 0, i) < (1 << 31) for i in range(d)])
    code = np.array([sum(v * 3 ** n for n, v in enumerate(oracle.draw_permutation(1, 0, 0, i, N))) for i in range(d)])
    keys = sorted(set(code.tolist()))
    assert len(keys) == 6
    table = np.array([[np.count_nonzero((code == k) & (below == b)) for k in keys] for b in (False, True)], dtype=float)
    exp = table.sum(1, keepdims=True) * table.sum(0, keepdims=True) / table.sum()
    chi2 = ((table - exp) ** 2 / exp).sum()
    assert chi2 < _chi2_quantile_999(5), chi2


def test_expectation_matches_eq4():
    """Eq. 4: E[theta_hat_n] = (1 - p) theta_n + p mean, over many seeds."""
    N, d, p, trials = 3, 64, 0.25, 4000
    pop, off, P = _pop(N, [d])
    base = W.to_stack(W.flat_population(N, d, seed=4, std=1.0), [d], off, P)
    acc = np.zeros((N, d), dtype=np.float64)
    for s in range(trials):
        y = base.copy()
        oracle.shuffle(pop, y, p, seed=1000 + s, step=0)
        acc += y.reshape(N, P)[:, :d]
    acc /= trials
    th = base.reshape(N, P)[:, :d].astype(np.float64)
    q = oracle.threshold(p) / 2 ** 32
    want = (1 - q) * th + q * th.mean(axis=0, keepdims=True)
    # per-entry variance of theta_hat is at most the spread of the column
    spread = th.max(axis=0) - th.min(axis=0)
    assert (np.abs(acc - want) < 5 * spread[None, :] / math.sqrt(trials) + 1e-12).all()


def test_last_layer_is_never_shuffled_under_the_default_schedule():
    numel = [64, 128, 32, 256]
    N = 4
    pop, off, P = _pop(N, numel)
    probs = oracle.layer_probs(len(numel), 0.9)
    assert probs[0] == 0.9 and probs[-1] == 0.0
    base = W.to_stack(W.flat_population(N, sum(numel), seed=6), numel, off, P)
    for seed in range(200):
        y = base.copy()
        oracle.shuffle(pop, y, probs, seed=seed, step=seed)
        last = slice(int(off[-1]), int(off[-1]) + numel[-1])
        assert (y.reshape(N, P)[:, last].view(np.uint32) == base.reshape(N, P)[:, last].view(np.uint32)).all()
        assert (y.reshape(N, P)[:, :64].view(np.uint32) != base.reshape(N, P)[:, :64].view(np.uint32)).any()


def test_optimizer_state_follows_the_same_draw():
    N, numel = 5, [300, 12]
    pop, off, P = _pop(N, numel)
    a = _sentinel(N, P)
    b = _sentinel(N, P)
    st_both = oracle.shuffle(pop, a, 0.4, seed=21, step=9, stack2=b)
    assert (a == b).all()
    c = _sentinel(N, P)
    st_one = oracle.shuffle(pop, c, 0.4, seed=21, step=9)
    assert (a == c).all() and st_both == st_one
    # bf16 parameters with fp32 momentum (sentinels survive bf16 exactly)
    ab = W.to_bf16_bits(_sentinel(N, P))
    m = _sentinel(N, P)
    oracle.shuffle(pop, ab, 0.4, seed=21, step=9, stack2=m)
    assert (W.bf16_bits_to_f32(ab) == a).all() and (m == a).all()


def test_a_slice_of_a_tensor_shuffles_like_the_whole():
    """RNG is keyed by (tensor, coordinate): a segment that holds coordinates
    [lo, hi) of tensor t, shuffled alone, equals that slice of the full shuffle."""
    N, d, t_id = 4, 1000, 3
    full = oracle.Population(N, [8, 8, 8, d])
    dense = W.flat_population(N, 24 + d, seed=12)
    x = dense.copy()
    oracle.shuffle(full, x, 0.5, seed=17, step=2)
    for lo, hi in ((0, 400), (400, 1000), (396, 404)):
        seg = oracle.Population(N, [hi - lo], tensor_id=[t_id], coord_begin=[lo])
        y = np.ascontiguousarray(dense[:, 24 + lo:24 + hi])
        oracle.shuffle(seg, y, 0.5, seed=17, step=2)
        assert (y.view(np.uint32) == x[:, 24 + lo:24 + hi].view(np.uint32)).all()


def test_seed_step_and_tensor_change_the_draw():
    N, d = 3, 4096
    pop, off, P = _pop(N, [d])
    outs = []
    for seed, step in ((0, 0), (1, 0), (0, 1), (0, 1 << 32), (1 << 32, 0)):
        x = _sentinel(N, P)
        oracle.shuffle(pop, x, 0.5, seed=seed, step=step)
        outs.append(x.copy())
    for a, b in itertools.combinations(outs, 2):
        assert (a != b).any()
    # same arguments: same result
    x = _sentinel(N, P)
    oracle.shuffle(pop, x, 0.5, seed=0, step=0)
    assert (x == outs[0]).all()
    # two tensors of one stack draw differently
    pop2, off2, P2 = _pop(N, [d, d])
    x = _sentinel(N, P2)
    oracle.shuffle(pop2, x, 0.5, seed=0, step=0)
    r = x.reshape(N, P2)
    assert (r[:, :d] == outs[0].reshape(N, P)[:, :d]).all() and (r[:, d:2 * d] != r[:, :d]).any()


def test_brute_force_on_tiny_stacks():
    """Every coordinate of a tiny stack recomputed by hand from the exposed words."""
    for N, numel, p in ((2, [1], 1.0), (3, [5, 3], 0.6), (4, [9], 0.5), (3, [4, 4, 1], [1.0, 0.5, 0.25])):
        pop, off, P = _pop(N, numel)
        dense = np.arange(N * sum(numel), dtype=np.float32).reshape(N, -1) + 1
        x = W.to_stack(dense, numel, off, P)
        oracle.shuffle(pop, x, p, seed=31, step=6)
        got = W.from_stack(x, N, numel, off, P)
        ps = np.broadcast_to(np.asarray(p, dtype=float), (len(numel),))
        want = dense.copy()
        col = 0
        for t, d in enumerate(numel):
            for i in range(d):
                if oracle.mask_word(31, 6, t, i) < math.floor(ps[t] * 2 ** 32):
                    pi = oracle.draw_permutation(31, 6, t, i, N)
                    want[:, col] = [dense[pi[n], col] for n in range(N)]
                col += 1
        assert (got == want).all()


def test_argument_errors():
    pop, off, P = _pop(3, [16])
    x = np.zeros(3 * P, dtype=np.float32)
    with pytest.raises(ValueError):
        oracle.shuffle(pop, x, 1.5, seed=0, step=0)
    with pytest.raises(ValueError):
        oracle.shuffle(pop, x, float("nan"), seed=0, step=0)
    with pytest.raises(ValueError):
        oracle.shuffle(pop, x, 0.5, seed=0, step=1 << 56)
