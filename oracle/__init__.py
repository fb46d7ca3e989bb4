"""CPU oracle for the WASH population operators -- TEST INFRASTRUCTURE ONLY.

``wash_oracle.c`` is the slow, plain statement of what the GPU library has to
compute (shuffle of Eq. 3 / Algorithm 1, PAPA's EMA of Eq. 1, the final average).
This module compiles it with gcc and exposes it to the tests over numpy arrays.
It imports nothing from the CUDA package and the CUDA package imports nothing from
here; only the tests, the smoke check and the CPU-baseline leg of the benchmark may
use it.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wash_oracle.c")
_LIB = os.path.join(_HERE, "libwash_oracle.so")
_lock = threading.Lock()
_lib = None

LAYOUT_NP, LAYOUT_PN = 0, 1
F32, BF16 = 0, 1
SCHEDULE_DECREASING, SCHEDULE_CONSTANT, SCHEDULE_INCREASING = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle (gcc, no fast-math, no FMA contraction) if it is stale.
    WASH_ORACLE_LIB names an already built library to load instead (used by the test
    that checks the pins against deliberately broken copies of the oracle)."""
    override = os.environ.get("WASH_ORACLE_LIB")
    if override:
        return override
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
                   "-fno-fast-math", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


class _Population(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int32), ("T", ctypes.c_int32),
                ("numel", ctypes.POINTER(ctypes.c_int64)),
                ("offset", ctypes.POINTER(ctypes.c_int64)),
                ("tensor_id", ctypes.POINTER(ctypes.c_uint32)),
                ("coord_begin", ctypes.POINTER(ctypes.c_int64)),
                ("padded_P", ctypes.c_int64), ("layout", ctypes.c_int32)]


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32p, i32p = ctypes.POINTER(ctypes.c_uint32), ctypes.POINTER(ctypes.c_int32)
        f64p, u64p = ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_uint64)
        popp = ctypes.POINTER(_Population)
        L.wo_philox4x32_10.argtypes = [u32p, u32p, u32p]; L.wo_philox4x32_10.restype = None
        L.wo_mask_word.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64]
        L.wo_mask_word.restype = ctypes.c_uint32
        L.wo_perm_word.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_int]
        L.wo_perm_word.restype = ctypes.c_uint32
        L.wo_threshold.argtypes = [ctypes.c_double]; L.wo_threshold.restype = ctypes.c_uint64
        L.wo_draw_permutation.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint64,
                                          ctypes.c_int32, i32p]
        L.wo_draw_permutation.restype = None
        L.wo_layer_probs.argtypes = [ctypes.c_int32, ctypes.c_double, ctypes.c_int32, f64p]
        L.wo_shuffle.argtypes = [popp, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32,
                                 f64p, ctypes.c_uint64, ctypes.c_uint64, u64p]
        L.wo_papa_ema.argtypes = [popp, ctypes.c_void_p, ctypes.c_int32, ctypes.c_float]
        L.wo_population_average.argtypes = [popp, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32]
        L.wo_papa_all.argtypes = [popp, ctypes.c_void_p, ctypes.c_int32]
        L.wo_consensus_sq.argtypes = [popp, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, f64p]
        L.wo_set_threads.argtypes = [ctypes.c_int]; L.wo_set_threads.restype = None
        i64p = ctypes.POINTER(ctypes.c_int64)
        L.wo_exchange_counts.argtypes = [popp, f64p, ctypes.c_uint64, ctypes.c_uint64, i64p, i64p]
        L.wo_exchange_send.argtypes = [popp, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32, f64p, ctypes.c_uint64,
                                       ctypes.c_uint64, ctypes.POINTER(ctypes.c_void_p), ctypes.c_int64, i64p]
        L.wo_exchange_receive.argtypes = [popp, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32, f64p, ctypes.c_uint64,
                                          ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int64, u64p]
        _lib = L
    return _lib


def set_threads(n: int) -> None:
    lib().wo_set_threads(int(n))


def get_threads() -> int:
    return int(lib().wo_get_threads())


def max_threads() -> int:
    return int(lib().wo_max_threads())


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*[int(x) & 0xFFFFFFFF for x in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(x) & 0xFFFFFFFF for x in key])
    o = (ctypes.c_uint32 * 4)()
    lib().wo_philox4x32_10(c, k, o)
    return [int(x) for x in o]


def mask_word(seed, step, t, i) -> int:
    return int(lib().wo_mask_word(seed, step, t, i))


def perm_word(seed, step, t, i, m) -> int:
    return int(lib().wo_perm_word(seed, step, t, i, m))


def threshold(p: float) -> int:
    return int(lib().wo_threshold(float(p)))


def draw_permutation(seed, step, t, i, N):
    out = (ctypes.c_int32 * N)()
    lib().wo_draw_permutation(seed, step, t, i, N, out)
    return [int(x) for x in out]


def layer_probs(L: int, p: float, schedule: int = SCHEDULE_DECREASING) -> np.ndarray:
    out = np.zeros(L, dtype=np.float64)
    rc = lib().wo_layer_probs(L, float(p), schedule, out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc != 0:
        raise ValueError("wo_layer_probs: bad argument")
    return out


class Population:
    """Shape of a stacked population: N copies of T segments (see wash_oracle.c)."""

    def __init__(self, N, numel, offset=None, padded_P=None, layout=LAYOUT_NP,
                 tensor_id=None, coord_begin=None):
        self.N = int(N)
        self.numel = np.ascontiguousarray(numel, dtype=np.int64)
        self.T = int(self.numel.size)
        if offset is None:
            offset = np.concatenate([[0], np.cumsum(self.numel)[:-1]]) if self.T else np.zeros(0)
        self.offset = np.ascontiguousarray(offset, dtype=np.int64)
        if padded_P is None:
            padded_P = int((self.offset + self.numel).max()) if self.T else 0
        self.padded_P = int(padded_P)
        self.layout = int(layout)
        self.tensor_id = None if tensor_id is None else np.ascontiguousarray(tensor_id, dtype=np.uint32)
        self.coord_begin = None if coord_begin is None else np.ascontiguousarray(coord_begin, dtype=np.int64)
        i64p, u32p = ctypes.POINTER(ctypes.c_int64), ctypes.POINTER(ctypes.c_uint32)
        self._c = _Population(
            self.N, self.T, self.numel.ctypes.data_as(i64p), self.offset.ctypes.data_as(i64p),
            None if self.tensor_id is None else self.tensor_id.ctypes.data_as(u32p),
            None if self.coord_begin is None else self.coord_begin.ctypes.data_as(i64p),
            self.padded_P, self.layout)

    @property
    def n_elems(self) -> int:
        return self.N * self.padded_P

    def ref(self):
        return ctypes.byref(self._c)


def _np_dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32 or a.dtype == np.uint32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("stack must be float32/uint32 (fp32) or uint16 (bf16 bits), got %s" % a.dtype)


def _check_stack(pop: Population, a: np.ndarray, rows=None):
    if not (isinstance(a, np.ndarray) and a.flags["C_CONTIGUOUS"] and a.flags["WRITEABLE"]):
        raise TypeError("stack must be a writable C-contiguous numpy array")
    need = pop.n_elems if rows is None else rows * pop.padded_P
    if a.size != need:
        raise ValueError("stack has %d elements, population needs %d" % (a.size, need))


def shuffle(pop: Population, stack: np.ndarray, p_seg, seed: int, step: int, stack2: np.ndarray | None = None):
    """In-place shuffling step (Eq. 3). Returns (selected_coords, moved_values)."""
    _check_stack(pop, stack)
    p = np.ascontiguousarray(np.broadcast_to(np.asarray(p_seg, dtype=np.float64), (pop.T,)))
    stats = (ctypes.c_uint64 * 2)(0, 0)
    s2, d2 = None, 0
    if stack2 is not None:
        _check_stack(pop, stack2)
        s2, d2 = stack2.ctypes.data, _np_dtype_code(stack2)
    rc = lib().wo_shuffle(pop.ref(), stack.ctypes.data, _np_dtype_code(stack), s2, d2,
                          p.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), seed, step, stats)
    if rc != 0:
        raise ValueError("wo_shuffle: bad argument")
    return int(stats[0]), int(stats[1])


def papa_ema(pop: Population, stack: np.ndarray, alpha: float) -> None:
    _check_stack(pop, stack)
    if lib().wo_papa_ema(pop.ref(), stack.ctypes.data, _np_dtype_code(stack), ctypes.c_float(alpha)) != 0:
        raise ValueError("wo_papa_ema: bad argument")


def population_average(pop: Population, stack: np.ndarray, out: np.ndarray) -> None:
    _check_stack(pop, stack)
    _check_stack(pop, out, rows=1)
    if lib().wo_population_average(pop.ref(), stack.ctypes.data, _np_dtype_code(stack),
                                   out.ctypes.data, _np_dtype_code(out)) != 0:
        raise ValueError("wo_population_average: bad argument")


def papa_all(pop: Population, stack: np.ndarray) -> None:
    _check_stack(pop, stack)
    if lib().wo_papa_all(pop.ref(), stack.ctypes.data, _np_dtype_code(stack)) != 0:
        raise ValueError("wo_papa_all: bad argument")


def consensus_sq(pop: Population, stack: np.ndarray, seg_lo: int = 0, seg_hi: int | None = None) -> np.ndarray:
    _check_stack(pop, stack)
    out = np.zeros(pop.N, dtype=np.float64)
    hi = pop.T if seg_hi is None else seg_hi
    if lib().wo_consensus_sq(pop.ref(), stack.ctypes.data, _np_dtype_code(stack), seg_lo, hi,
                             out.ctypes.data_as(ctypes.POINTER(ctypes.c_double))) != 0:
        raise ValueError("wo_consensus_sq: bad argument")
    return out


def _p_seg(pop: Population, p_seg) -> np.ndarray:
    return np.ascontiguousarray(np.broadcast_to(np.asarray(p_seg, dtype=np.float64), (pop.T,)))


def exchange_counts(pop: Population, p_seg, seed: int, step: int):
    """-> (need[N], selected): slots each worker's staging buffer needs in this step."""
    p = _p_seg(pop, p_seg)
    need = np.zeros(pop.N, dtype=np.int64)
    sel = ctypes.c_int64(0)
    rc = lib().wo_exchange_counts(pop.ref(), p.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), seed, step,
                                  need.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), ctypes.byref(sel))
    if rc != 0:
        raise ValueError("wo_exchange_counts: bad argument")
    return need, int(sel.value)


def exchange_send(pop: Population, self_rank: int, row: np.ndarray, p_seg, seed: int, step: int, staging) -> np.ndarray:
    """Worker `self_rank` (holding the model `row`) fills its slots of the other workers'
    staging buffers (a list of N arrays of the row's dtype). -> slots written per worker."""
    _check_stack(pop, row, rows=1)
    p = _p_seg(pop, p_seg)
    code = _np_dtype_code(row)
    cap = min(int(b.size) for k, b in enumerate(staging) if k != self_rank)
    for k, b in enumerate(staging):
        if k != self_rank and _np_dtype_code(b) != code:
            raise TypeError("staging buffers must have the row's element type")
    ptrs = (ctypes.c_void_p * pop.N)(*[b.ctypes.data for b in staging])
    filled = np.zeros(pop.N, dtype=np.int64)
    rc = lib().wo_exchange_send(pop.ref(), self_rank, row.ctypes.data, code,
                                p.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), seed, step, ptrs, cap,
                                filled.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)))
    if rc != 0:
        raise ValueError("wo_exchange_send: bad argument or staging buffer too small")
    return filled


def exchange_receive(pop: Population, self_rank: int, row: np.ndarray, p_seg, seed: int, step: int, staging_self: np.ndarray):
    """Worker `self_rank` takes its new values out of its own staging buffer.
    -> (selected_coords, values received)"""
    _check_stack(pop, row, rows=1)
    p = _p_seg(pop, p_seg)
    if _np_dtype_code(staging_self) != _np_dtype_code(row):
        raise TypeError("staging buffer must have the row's element type")
    stats = (ctypes.c_uint64 * 2)(0, 0)
    rc = lib().wo_exchange_receive(pop.ref(), self_rank, row.ctypes.data, _np_dtype_code(row),
                                   p.ctypes.data_as(ctypes.POINTER(ctypes.c_double)), seed, step,
                                   staging_self.ctypes.data, int(staging_self.size), stats)
    if rc != 0:
        raise ValueError("wo_exchange_receive: bad argument or staging buffer too small")
    return int(stats[0]), int(stats[1])
