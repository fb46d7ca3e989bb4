"""wash_shuffle_noalloc against wash_shuffle and against the oracle.

The no-allocation entry point serves callers that cannot call cudaMalloc (all device
memory already owned by a framework's pool, or a loop that cannot take cudaMalloc's
device-wide synchronisation).  It keeps its tables in an array built into the library,
shared by every call, so the things to check are: the bits equal those of the
context-based call and those of the CPU oracle, a second call is not disturbed by what the first one left in the
array (here the second call even uses a different tensor table), and sizes beyond the
array's capacity are refused.  This file is named to be collected last.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_17517_b200 import binding as B
from paper_2405_17517_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _reference(N, numel, layout, dtype_code, stack, step, p, p_layer, seed):
    ctx = B.wash_create(N, numel, layout, 0)
    t = stack.clone()
    stats = torch.zeros(2, dtype=torch.int64, device="cuda")
    B.wash_bind(ctx, B.WASH_STACK_PARAMS, dtype_code, t, t.numel())
    B.wash_shuffle(ctx, step, p, p_layer, seed, None, stats)
    torch.cuda.synchronize()
    B.wash_destroy(ctx)
    return t, stats


def _make(N, numel, layout, bf16, seed):
    off, P = W.padded_offsets(numel)
    dense = W.flat_population(N, int(sum(numel)), seed=seed)
    if bf16:
        host = W.to_stack(W.to_bf16_bits(dense), numel, off, P, layout).reshape(-1)
        return torch.from_numpy(host.view(np.int16).copy()).view(torch.bfloat16).cuda(), P, host, off
    host = W.to_stack(dense, numel, off, P, layout).reshape(-1)
    return torch.from_numpy(host.copy()).cuda(), P, host, off


def _bits(t):
    return t.view(torch.int32 if t.dtype == torch.float32 else torch.int16)


def test_two_calls_in_a_row_match_the_context_based_shuffle():
    calls = [
        dict(N=5, numel=[1000, 33, 7, 1, 4, 8, 5003, 2048], layout=0, bf16=False, step=3, p=0.25, p_layer=None, seed=11),
        # a different table, layout and dtype: whatever call 1 left in the array must not matter
        dict(N=8, numel=[64, 40000, 9], layout=1, bf16=True, step=(2 << 32) | 7, p=0.0, p_layer=[1.0, 0.01, 0.5], seed=12),
        # and the first shape again, next step
        dict(N=5, numel=[1000, 33, 7, 1, 4, 8, 5003, 2048], layout=0, bf16=False, step=4, p=0.25, p_layer=None, seed=11),
        # small groups: the entry point launches the streaming kernel for them (several trips per warp here)
        dict(N=2, numel=[700001, 5, 4099], layout=0, bf16=False, step=9, p=0.02, p_layer=None, seed=13),
        dict(N=3, numel=[33, 90000, 7], layout=1, bf16=False, step=10, p=0.0, p_layer=[1.0, 0.3, 0.0], seed=14),
    ]
    for c in calls:
        stack, P, host, off = _make(c["N"], c["numel"], c["layout"], c["bf16"], seed=c["seed"])
        code = B.WASH_BF16 if c["bf16"] else B.WASH_F32
        want, want_stats = _reference(c["N"], c["numel"], c["layout"], code, stack, c["step"], c["p"], c["p_layer"], c["seed"])
        stats = torch.zeros(2, dtype=torch.int64, device="cuda")
        B.wash_shuffle_noalloc(c["N"], c["numel"], c["layout"], code, stack, stack.numel(), c["step"], c["p"],
                               c["p_layer"], c["seed"], 0, None, stats)
        torch.cuda.synchronize()
        assert torch.equal(_bits(stack), _bits(want))          # bit-exact, as for every shuffle test
        assert torch.equal(stats, want_stats)
        assert int(stats[0]) > 0
        # and the oracle's bits, computed on the host copy of the same stack
        ora = oracle.Population(c["N"], c["numel"], off, P, c["layout"])
        host = np.ascontiguousarray(host)
        sel, moved = oracle.shuffle(ora, host, c["p"] if c["p_layer"] is None else c["p_layer"], seed=c["seed"], step=c["step"])
        got = _bits(stack).cpu().numpy()
        assert (got.view(host.dtype if host.dtype == np.uint16 else np.uint32) == (host if host.dtype == np.uint16 else host.view(np.uint32))).all()
        assert (int(stats[0]), int(stats[1])) == (sel, moved)


def test_a_capturing_stream_is_refused_and_nothing_is_recorded():
    """The call copies its tables from host arrays that are gone when it returns, so it must
    not be recorded into a graph: a stream in capture mode gets WASH_ERR_STATE."""
    stack, P, host, off = _make(3, [256], 0, False, seed=1)
    B.wash_shuffle_noalloc(3, [256], 0, B.WASH_F32, stack, stack.numel(), 0, 0.5)      # first use on the device, outside capture
    torch.cuda.synchronize()
    before = stack.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        graph.capture_begin()
        try:
            with pytest.raises(B.WashError) as e:
                B.wash_shuffle_noalloc(3, [256], 0, B.WASH_F32, stack, stack.numel(), 1, 0.5, stream=side)
        finally:
            graph.capture_end()
    assert e.value.code == B.WASH_ERR_STATE
    torch.cuda.synchronize()
    assert torch.equal(_bits(stack), _bits(before))


def test_sizes_beyond_the_built_in_scratch_are_refused():
    t = torch.zeros(16, device="cuda")
    with pytest.raises(B.WashError) as e:
        B.wash_shuffle_noalloc(2, [8] * 1025, 0, B.WASH_F32, t, 2 * 8 * 1025, 0, 0.5)
    assert e.value.code == B.WASH_ERR_ARG and "1024" in str(e.value)
    with pytest.raises(B.WashError) as e:
        B.wash_shuffle_noalloc(2, [(1 << 26) + 8], 0, B.WASH_F32, t, 2 * ((1 << 26) + 8), 0, 0.5)
    assert e.value.code == B.WASH_ERR_ARG and "2^26" in str(e.value)
    with pytest.raises(B.WashError) as e:
        B.wash_shuffle_noalloc(2, [8], 0, B.WASH_F32, t, 15, 0, 0.5)       # wrong stack size
    assert e.value.code == B.WASH_ERR_ARG
    assert (t == 0).all()
