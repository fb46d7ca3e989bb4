"""Pins for the oracle's worker form of the shuffling step (one model per worker, values
travelling peer to peer along the permutation) -- CPU only.

The worker form has a plain definition: a send by every worker followed by a receive by
every worker must be the shuffling step of Eq. 3 on the stacked population, which the
other oracle tests pin on its own."""
import math

import numpy as np
import pytest

import oracle
from paper_2405_17517_b200 import workloads as W


def _pop(N, numel, **kw):
    off, P = W.padded_offsets(numel)
    return oracle.Population(N, numel, off, P, 0, **kw), off, P


def _run_workers(pop, rows, p_seg, seed, step, capacity, fill):
    """every worker sends, then every worker receives; returns (staging, filled, stats)"""
    N = pop.N
    staging = [np.full(capacity, fill, dtype=rows[0].dtype) for _ in range(N)]
    filled = np.zeros((N, N), dtype=np.int64)
    for n in range(N):
        filled[n] = oracle.exchange_send(pop, n, rows[n], p_seg, seed, step, staging)
    stats = [oracle.exchange_receive(pop, n, rows[n], p_seg, seed, step, staging[n]) for n in range(N)]
    return staging, filled, stats


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("N", [2, 3, 5, 17])
def test_workers_reproduce_the_population_shuffle(N, dtype):
    numel = [1501, 3, 64, 250]
    pop, off, P = _pop(N, numel)
    dense = W.flat_population(N, sum(numel), seed=20 + N)
    if dtype == "bf16":
        dense = W.to_bf16_bits(dense)
    stack = W.to_stack(dense, numel, off, P, 0)
    p_seg = [0.2, 1.0, 0.0, 0.05]
    for step in (0, 7):
        rows = [stack.reshape(N, P)[n].copy() for n in range(N)]
        want = stack.copy()
        sel, moved = oracle.shuffle(pop, want, p_seg, seed=5, step=step)
        need, sel_c = oracle.exchange_counts(pop, p_seg, seed=5, step=step)
        assert sel_c == sel and int(need.sum()) == moved
        fill = np.array(0x7FC1, dtype=np.uint16) if dtype == "bf16" else np.float32(-77.0)
        staging, filled, stats = _run_workers(pop, rows, p_seg, 5, step, int(need.max()) + 3, fill)
        got = np.stack(rows).reshape(-1)
        a = got.view(np.uint32) if dtype == "f32" else got
        b = want.reshape(-1).view(np.uint32) if dtype == "f32" else want.reshape(-1)
        assert (a == b).all()
        for n in range(N):
            assert stats[n] == (sel, int(need[n]))
            assert filled[:, n].sum() == need[n] and filled[n, n] == 0
            assert (staging[n][need[n]:] == fill).all() or np.isnan(fill)      # slots beyond the need stay untouched
        stack = want


def test_slots_follow_the_permutations_drawn_one_by_one():
    """Brute force on a tiny row: slot k of worker n holds the value that worker pi_i(n) had
    at the k-th selected coordinate i (in loop order) with pi_i(n) != n."""
    N, numel = 4, [9, 5]
    pop, off, P = _pop(N, numel)
    seed, step, p = 31, 2, 0.6
    rows = [(1000.0 * n + np.arange(P)).astype(np.float32) for n in range(N)]
    before = [r.copy() for r in rows]
    need, _ = oracle.exchange_counts(pop, p, seed, step)
    staging, _, _ = _run_workers(pop, rows, p, seed, step, 32, np.float32(-1.0))
    thr = oracle.threshold(p)
    expect = [[] for _ in range(N)]
    for t, d in enumerate(numel):
        for i in range(d):
            if oracle.mask_word(seed, step, t, i) >= thr:
                continue
            perm = oracle.draw_permutation(seed, step, t, i, N)
            for n in range(N):
                if perm[n] != n:
                    expect[n].append(before[perm[n]][off[t] + i])
    assert sum(len(e) for e in expect) > 10
    for n in range(N):
        assert len(expect[n]) == need[n]
        assert staging[n][:need[n]].tolist() == expect[n]


def test_volume_per_worker_matches_the_papers_count():
    """Each model communicates p*d parameters per step in expectation (section "WASH");
    a uniform permutation keeps a value in place with probability 1/N, so p*d*(N-1)/N of
    them actually leave the worker."""
    N, d, p = 5, 200000, 0.01
    pop, _, _ = _pop(N, [d])
    tot = np.zeros(N)
    steps = 4
    for step in range(steps):
        need, sel = oracle.exchange_counts(pop, p, seed=77, step=step)
        tot += need
        assert abs(sel - p * d) < 5 * math.sqrt(p * d)
    mean = steps * p * d * (N - 1) / N
    assert (np.abs(tot - mean) < 5 * math.sqrt(mean)).all()


def test_p_zero_sends_nothing_and_two_workers_swap():
    pop, off, P = _pop(2, [300])
    rows = [np.arange(P, dtype=np.float32), -np.arange(P, dtype=np.float32) - 1]
    keep = [r.copy() for r in rows]
    need, sel = oracle.exchange_counts(pop, 0.0, 1, 1)
    assert sel == 0 and need.tolist() == [0, 0]
    _run_workers(pop, rows, 0.0, 1, 1, 4, np.float32(9.0))
    assert all((rows[n] == keep[n]).all() for n in range(2))
    # N = 2, p = 1: every coordinate is either left alone or swapped between the two
    need, sel = oracle.exchange_counts(pop, 1.0, 1, 1)
    assert sel == 300 and need[0] == need[1] and 100 < need[0] < 200
    _run_workers(pop, rows, 1.0, 1, 1, 300, np.float32(9.0))
    swapped = rows[0][:300] != keep[0][:300]
    assert swapped.sum() == need[0]
    assert (rows[0][:300][swapped] == keep[1][:300][swapped]).all()
    assert (rows[1][:300][swapped] == keep[0][:300][swapped]).all()
    assert (rows[1][:300][~swapped] == keep[1][:300][~swapped]).all()


def test_too_small_a_staging_buffer_is_an_error():
    pop, off, P = _pop(3, [500])
    rows = [np.zeros(P, dtype=np.float32) for _ in range(3)]
    need, _ = oracle.exchange_counts(pop, 0.5, 3, 0)
    small = [np.zeros(int(need.min()) // 2, dtype=np.float32) for _ in range(3)]
    with pytest.raises(ValueError):
        oracle.exchange_send(pop, 0, rows[0], 0.5, 3, 0, small)
    with pytest.raises(ValueError):
        oracle.exchange_receive(pop, 0, rows[0], 0.5, 3, 0, small[0])


def test_shards_of_a_row_exchange_like_the_whole_row():
    """Draws are keyed by (tensor, coordinate): a worker that holds a slice of each tensor
    sends and receives exactly what the whole-row worker does for those coordinates."""
    N, d = 3, 4000
    full, off, P = _pop(N, [d])
    half, offh, Ph = _pop(N, [1200], tensor_id=[0], coord_begin=[2000])
    dense = W.flat_population(N, d, seed=3)
    rows = [dense[n].copy() for n in range(N)]
    rows_h = [dense[n, 2000:3200].copy() for n in range(N)]
    rows = [np.concatenate([r, np.zeros(P - d, np.float32)]) for r in rows]
    rows_h = [np.concatenate([r, np.zeros(Ph - 1200, np.float32)]) for r in rows_h]
    _run_workers(full, rows, 0.3, 8, 4, d, np.float32(0))
    _run_workers(half, rows_h, 0.3, 8, 4, d, np.float32(0))
    for n in range(N):
        assert (rows[n][2000:3200].view(np.uint32) == rows_h[n][:1200].view(np.uint32)).all()
