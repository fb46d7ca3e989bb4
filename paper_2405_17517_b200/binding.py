"""ctypes binding of libwash.so: the same entry points as include/wash.h.

Only argument marshalling happens here; every step of the operators runs in the
library's CUDA kernels.  PyTorch supplies device memory (tensor.data_ptr()) and the
stream.  There is no CPU fallback: if the library cannot be loaded, importing this
module's functions raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwash.so")

WASH_OK = 0
WASH_ERR_ARG, WASH_ERR_STATE, WASH_ERR_ALLOC, WASH_ERR_CUDA, WASH_ERR_UNSUPPORTED, WASH_ERR_DEVICE_CHECK = -1, -2, -3, -4, -5, -6
WASH_LAYOUT_NP, WASH_LAYOUT_PN = 0, 1
WASH_F32, WASH_BF16 = 0, 1
WASH_STACK_PARAMS, WASH_STACK_OPT, WASH_STACK_BOTH = 0, 1, 2
WASH_MAX_CONSENSUS_RANGES = 8
WASH_SCHEDULE_DECREASING, WASH_SCHEDULE_CONSTANT, WASH_SCHEDULE_INCREASING = 0, 1, 2
WASH_MODE_STREAM, WASH_MODE_SPARSE, WASH_MODE_AUTO = 0, 1, 2
WASH_OP_SHUFFLE, WASH_OP_EMA, WASH_OP_AVERAGE = 1, 2, 4
WASH_MAX_N = 64
WASH_ALIGN_ELEMS = 8


class WashError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("libwash error %d: %s" % (code, message))
        self.code = code


class wash_stats(ctypes.Structure):
    _fields_ = [("selected_coords", ctypes.c_uint64), ("moved_values", ctypes.c_uint64)]


_lib = None


def load() -> ctypes.CDLL:
    """Load libwash.so (built in-tree by paper_2405_17517_b200.build). Fails loudly."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError("%s is missing: build it with `python -m paper_2405_17517_b200.build` "
                          "(there is no fallback path)" % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, u64, dbl = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64, ctypes.c_double
    i64p, u32p, dblp = ctypes.POINTER(i64), ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(dbl)
    L.wash_create.argtypes = [ctypes.POINTER(vp), i32, i32, i64p, i32, i32]
    L.wash_create_segments.argtypes = [ctypes.POINTER(vp), i32, i32, i64p, u32p, i64p, i32, i32]
    L.wash_destroy.argtypes = [vp]
    L.wash_stack_elems.argtypes = [vp, i64p, i64p]
    L.wash_bind.argtypes = [vp, i32, i32, vp, i64]
    L.wash_set_mode.argtypes = [vp, i32]
    L.wash_set_launch.argtypes = [vp, i32, i32]
    L.wash_layer_probs.argtypes = [i32, dbl, i32, dblp]
    for name in ("wash_shuffle", "wash_shuffle_opt_state", "wash_shuffle_both"):
        getattr(L, name).argtypes = [vp, u64, dbl, dblp, u64, vp, vp]
    L.wash_shuffle_consensus.argtypes = [vp, i32, u64, dbl, dblp, u64, vp, vp, i32, ctypes.POINTER(i32), vp]
    L.papa_ema.argtypes = [vp, i32, ctypes.c_float, vp]
    L.population_average.argtypes = [vp, i32, vp, i32, vp]
    L.papa_all.argtypes = [vp, i32, vp]
    L.wash_consensus_sq.argtypes = [vp, i32, i32, i32, vp, vp]
    L.wash_step_host.argtypes = [vp, i32, vp, vp, vp, u64, dbl, dblp, u64, ctypes.c_float, vp, ctypes.POINTER(wash_stats)]
    L.wash_check.argtypes = [vp, vp]
    L.wash_philox_probe.argtypes = [u64, u64, vp, i32, vp]
    L.wash_last_error.restype = ctypes.c_char_p
    L.wash_launch_count.restype = ctypes.c_uint64
    L.wash_shuffle_noalloc.argtypes = [i32, i32, i64p, i32, i32, vp, i64, u64, dbl, dblp, u64, i32, vp, vp]
    L.wash_noalloc_last_error.restype = ctypes.c_char_p
    L.wash_exchange_bind.argtypes = [vp, i32, i32, i32, vp, i64]
    L.wash_exchange_staging.argtypes = [vp, i32, i32, ctypes.POINTER(vp), i64]
    L.wash_exchange_staging_create.argtypes = [vp, i32, i32, i64, vp]
    L.wash_exchange_staging_open.argtypes = [vp, i32, i32, vp]
    L.wash_exchange_plan.argtypes = [vp, u64, dbl, dblp, u64, vp]
    L.wash_exchange_send.argtypes = [vp, vp]
    L.wash_exchange_receive.argtypes = [vp, vp, vp]
    L.wash_exchange_counts.argtypes = [vp, ctypes.POINTER(u64), ctypes.POINTER(u64), vp]
    _lib = L
    return L


def _check(rc: int) -> None:
    if rc != WASH_OK:
        raise WashError(rc, load().wash_last_error().decode())


def _i64(a):
    arr = np.ascontiguousarray(a, dtype=np.int64)
    return arr, arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def _dbl_or_null(a):
    if a is None:
        return None, None
    arr = np.ascontiguousarray(a, dtype=np.float64)
    return arr, arr.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if isinstance(x, np.ndarray):
        return x.ctypes.data
    raise TypeError("cannot take the address of %r" % type(x))


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


# ---- the C entry points, one to one ------------------------------------------------

def wash_create(N: int, numel: Sequence[int], layout: int = WASH_LAYOUT_NP, device: int = 0) -> int:
    arr, p = _i64(numel)
    ctx = ctypes.c_void_p()
    _check(load().wash_create(ctypes.byref(ctx), N, arr.size, p, layout, device))
    return ctx.value


def wash_create_segments(N: int, numel, tensor_id=None, coord_begin=None, layout: int = WASH_LAYOUT_NP, device: int = 0) -> int:
    arr, p = _i64(numel)
    tid = None if tensor_id is None else np.ascontiguousarray(tensor_id, dtype=np.uint32)
    cb = None if coord_begin is None else np.ascontiguousarray(coord_begin, dtype=np.int64)
    ctx = ctypes.c_void_p()
    _check(load().wash_create_segments(
        ctypes.byref(ctx), N, arr.size, p,
        None if tid is None else tid.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)),
        None if cb is None else cb.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), layout, device))
    return ctx.value


def wash_destroy(ctx: int) -> None:
    _check(load().wash_destroy(ctx))


def wash_stack_elems(ctx: int, n_tensors: int):
    """-> (padded_P, offsets[n_tensors])"""
    P = ctypes.c_int64()
    offs = np.zeros(n_tensors, dtype=np.int64)
    _check(load().wash_stack_elems(ctx, ctypes.byref(P), offs.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))))
    return int(P.value), offs


def wash_bind(ctx: int, stack: int, dtype: int, dev_ptr, n_elems: int) -> None:
    _check(load().wash_bind(ctx, stack, dtype, _ptr(dev_ptr), n_elems))


def wash_set_mode(ctx: int, mode: int) -> None:
    _check(load().wash_set_mode(ctx, mode))


def wash_set_launch(ctx: int, threads: int = 0, blocks_per_sm: int = 0) -> None:
    _check(load().wash_set_launch(ctx, threads, blocks_per_sm))


def wash_layer_probs(L: int, p: float, schedule: int = WASH_SCHEDULE_DECREASING) -> np.ndarray:
    out = np.zeros(max(L, 0), dtype=np.float64)
    _check(load().wash_layer_probs(L, p, schedule, out.ctypes.data_as(ctypes.POINTER(ctypes.c_double))))
    return out


def _shuffle(fn, ctx, step, p, p_layer, seed, stream, stats):
    keep, pl = _dbl_or_null(p_layer)
    _check(fn(ctx, step, float(p), pl, seed, _stream(stream), _ptr(stats)))


def wash_shuffle(ctx, step, p, p_layer=None, seed=0, stream=None, stats=None) -> None:
    _shuffle(load().wash_shuffle, ctx, step, p, p_layer, seed, stream, stats)


def wash_shuffle_opt_state(ctx, step, p, p_layer=None, seed=0, stream=None, stats=None) -> None:
    _shuffle(load().wash_shuffle_opt_state, ctx, step, p, p_layer, seed, stream, stats)


def wash_shuffle_both(ctx, step, p, p_layer=None, seed=0, stream=None, stats=None) -> None:
    _shuffle(load().wash_shuffle_both, ctx, step, p, p_layer, seed, stream, stats)


def wash_shuffle_consensus(ctx, stacks: int, step, p, p_layer=None, seed=0, stream=None, stats=None,
                           tensor_bounds=(0, 0), dev_sq_out=None) -> None:
    """tensor_bounds: n_ranges + 1 ascending tensor indices; dev_sq_out: [n_ranges][N] doubles on the device"""
    keep, pl = _dbl_or_null(p_layer)
    tb = np.ascontiguousarray(tensor_bounds, dtype=np.int32)
    _check(load().wash_shuffle_consensus(ctx, stacks, step, float(p), pl, seed, _stream(stream), _ptr(stats), tb.size - 1,
                                         tb.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), _ptr(dev_sq_out)))


def papa_ema(ctx, stack: int, alpha: float, stream=None) -> None:
    _check(load().papa_ema(ctx, stack, ctypes.c_float(alpha), _stream(stream)))


def population_average(ctx, stack: int, dev_out, out_dtype: int, stream=None) -> None:
    _check(load().population_average(ctx, stack, _ptr(dev_out), out_dtype, _stream(stream)))


def papa_all(ctx, stack: int, stream=None) -> None:
    _check(load().papa_all(ctx, stack, _stream(stream)))


def wash_consensus_sq(ctx, stack: int, tensor_lo: int, tensor_hi: int, dev_sq_out, stream=None) -> None:
    _check(load().wash_consensus_sq(ctx, stack, tensor_lo, tensor_hi, _ptr(dev_sq_out), _stream(stream)))


def wash_step_host(ctx, ops: int, host_params, host_opt, host_avg, step, p, p_layer=None, seed=0, alpha=0.5,
                   stream=None):
    """-> (selected_coords, moved_values) of this call"""
    keep, pl = _dbl_or_null(p_layer)
    st = wash_stats(0, 0)
    _check(load().wash_step_host(ctx, ops, _ptr(host_params), _ptr(host_opt), _ptr(host_avg), step, float(p), pl,
                                 seed, ctypes.c_float(alpha), _stream(stream), ctypes.byref(st)))
    return int(st.selected_coords), int(st.moved_values)


def wash_shuffle_noalloc(N: int, numel, layout: int, dtype: int, dev_stack, n_elems: int, step: int, p: float,
                         p_layer=None, seed: int = 0, device: int = 0, stream=None, stats=None) -> None:
    """The streaming shuffle without a context and without any allocation (see wash.h)."""
    arr, np_ = _i64(numel)
    keep, pl = _dbl_or_null(p_layer)
    rc = load().wash_shuffle_noalloc(N, arr.size, np_, layout, dtype, _ptr(dev_stack), n_elems, step, float(p), pl,
                                     seed, device, _stream(stream), _ptr(stats))
    if rc != WASH_OK:
        raise WashError(rc, load().wash_noalloc_last_error().decode())


def wash_noalloc_last_error() -> str:
    return load().wash_noalloc_last_error().decode()


def wash_exchange_bind(ctx, self_rank: int, stack: int, dtype: int, dev_row, n_elems: int) -> None:
    _check(load().wash_exchange_bind(ctx, self_rank, stack, dtype, _ptr(dev_row), n_elems))


def wash_exchange_staging(ctx, stack: int, parity: int, buffers, capacity_elems: int) -> None:
    """buffers: one tensor / address per worker (worker n's staging buffer)"""
    ptrs = (ctypes.c_void_p * len(buffers))(*[_ptr(b) for b in buffers])
    _check(load().wash_exchange_staging(ctx, stack, parity, ptrs, capacity_elems))


WASH_IPC_HANDLE_BYTES = 64


def wash_exchange_staging_create(ctx, stack: int, parity: int, capacity_elems: int) -> bytes:
    """-> this worker's inter-process handle (bytes) for the buffer it just allocated"""
    out = ctypes.create_string_buffer(WASH_IPC_HANDLE_BYTES)
    _check(load().wash_exchange_staging_create(ctx, stack, parity, capacity_elems, out))
    return out.raw


def wash_exchange_staging_open(ctx, stack: int, parity: int, handles) -> None:
    """handles: the N workers' handles in worker order (bytes each)"""
    blob = b"".join(bytes(h) for h in handles)
    _check(load().wash_exchange_staging_open(ctx, stack, parity, blob))


def wash_exchange_plan(ctx, step: int, p: float, p_layer=None, seed: int = 0, stream=None) -> None:
    keep, pl = _dbl_or_null(p_layer)
    _check(load().wash_exchange_plan(ctx, step, float(p), pl, seed, _stream(stream)))


def wash_exchange_send(ctx, stream=None) -> None:
    _check(load().wash_exchange_send(ctx, _stream(stream)))


def wash_exchange_receive(ctx, stream=None, stats=None) -> None:
    _check(load().wash_exchange_receive(ctx, _stream(stream), _ptr(stats)))


def wash_exchange_counts(ctx, N: int, stream=None):
    """-> (need[N], selected) of the last plan; waits for the stream"""
    need = (ctypes.c_uint64 * N)()
    sel = ctypes.c_uint64(0)
    _check(load().wash_exchange_counts(ctx, need, ctypes.byref(sel), _stream(stream)))
    return [int(x) for x in need], int(sel.value)


def wash_philox_probe(n_blocks: int, seed: int = 0, dev_checksum=None, device: int = 0, stream=None) -> None:
    _check(load().wash_philox_probe(n_blocks, seed, _ptr(dev_checksum), device, _stream(stream)))


def wash_check(ctx, stream=None) -> None:
    _check(load().wash_check(ctx, _stream(stream)))


def wash_last_error() -> str:
    return load().wash_last_error().decode()


def wash_launch_count() -> int:
    return int(load().wash_launch_count())


# ---- a small convenience wrapper over torch tensors ---------------------------------

def _torch_dtype_code(t) -> int:
    import torch
    if t.dtype == torch.float32:
        return WASH_F32
    if t.dtype == torch.bfloat16:
        return WASH_BF16
    raise TypeError("stacks are float32 or bfloat16 tensors, got %s" % t.dtype)


class Population:
    """A wash_ctx with its row geometry; stacks are torch CUDA tensors the caller owns."""

    def __init__(self, N: int, numel: Sequence[int], layout: int = WASH_LAYOUT_NP, device: int = 0,
                 tensor_id=None, coord_begin=None):
        self.N, self.layout, self.device = int(N), int(layout), int(device)
        self.numel = np.ascontiguousarray(numel, dtype=np.int64)
        self.ctx = wash_create_segments(N, self.numel, tensor_id, coord_begin, layout, device)
        self.padded_P, self.offsets = wash_stack_elems(self.ctx, self.numel.size)
        self._stacks = {}

    @property
    def n_elems(self) -> int:
        return self.N * self.padded_P

    def bind(self, stack: int, tensor) -> None:
        if not tensor.is_cuda or not tensor.is_contiguous():
            raise ValueError("a stack must be a contiguous CUDA tensor")
        wash_bind(self.ctx, stack, _torch_dtype_code(tensor), tensor, tensor.numel())
        self._stacks[stack] = tensor   # keep it alive while bound

    def close(self) -> None:
        if self.ctx:
            wash_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
