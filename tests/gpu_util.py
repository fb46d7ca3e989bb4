"""Helpers for the GPU parity tests: run an operator through the C ABI and through the
oracle on the same seeded input and hand back both results as bit patterns."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2405_17517_b200 import binding as B
from paper_2405_17517_b200 import workloads as W


def to_device(stack: np.ndarray) -> torch.Tensor:
    """numpy float32 / uint16(bf16 bits) stack -> flat CUDA tensor of float32 / bfloat16"""
    flat = np.ascontiguousarray(stack).reshape(-1)
    if flat.dtype == np.float32:
        return torch.from_numpy(flat.copy()).cuda()
    if flat.dtype == np.uint16:
        return torch.from_numpy(flat.view(np.int16).copy()).view(torch.bfloat16).cuda()
    raise TypeError(flat.dtype)


def to_host_bits(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.float32:
        return t.detach().cpu().numpy().view(np.uint32)
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def bits(a: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a).reshape(-1)
    return a.view(np.uint32) if a.dtype == np.float32 else a


class Case:
    """One population on both sides."""

    def __init__(self, N, numel, layout=0, dtype="f32", opt_dtype=None, seed=0, tensor_id=None, coord_begin=None,
                 dense=None, dense_opt=None):
        self.N, self.numel, self.layout = N, [int(d) for d in numel], layout
        self.gpu = B.Population(N, self.numel, layout, 0, tensor_id, coord_begin)
        self.P, self.off = self.gpu.padded_P, self.gpu.offsets
        self.ora = oracle.Population(N, self.numel, self.off, self.P, layout, tensor_id, coord_begin)
        total = sum(self.numel)
        if dense is None:
            dense = W.flat_population(N, total, seed=seed)
        self.host = self._stack(dense, dtype)
        self.dev = to_device(self.host)
        self.gpu.bind(B.WASH_STACK_PARAMS, self.dev)
        self.host_opt = self.dev_opt = None
        if opt_dtype is not None:
            if dense_opt is None:
                dense_opt = W.flat_population(N, total, seed=seed + 1000, std=1e-3)
            self.host_opt = self._stack(dense_opt, opt_dtype)
            self.dev_opt = to_device(self.host_opt)
            self.gpu.bind(B.WASH_STACK_OPT, self.dev_opt)
        self.stats_dev = torch.zeros(2, dtype=torch.int64, device="cuda")

    def _stack(self, dense, dtype):
        if dtype == "bf16":
            dense = W.to_bf16_bits(dense)
        return W.to_stack(dense, self.numel, self.off, self.P, self.layout)

    def gpu_stats(self):
        torch.cuda.synchronize()
        s = self.stats_dev.cpu().numpy().view(np.uint64)
        return int(s[0]), int(s[1])

    def assert_equal(self, what=""):
        torch.cuda.synchronize()
        B.wash_check(self.gpu.ctx)
        got = to_host_bits(self.dev)
        want = bits(self.host)
        bad = np.flatnonzero(got != want)
        assert bad.size == 0, "%s: %d parameter elements differ, first at %d" % (what, bad.size, bad[0])
        if self.dev_opt is not None:
            got = to_host_bits(self.dev_opt)
            want = bits(self.host_opt)
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, "%s: %d optimizer-state elements differ, first at %d" % (what, bad.size, bad[0])

    def close(self):
        self.gpu.close()


def ulp_distance_f32(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """distance in units in the last place between float32 bit patterns (NaN == NaN -> 0)"""
    def key(u):
        u = u.astype(np.int64)
        return np.where(u & 0x80000000, 0x80000000 - u, u)
    a_nan = np.isnan(a_bits.view(np.float32))
    b_nan = np.isnan(b_bits.view(np.float32))
    d = np.abs(key(a_bits) - key(b_bits))
    d[a_nan & b_nan] = 0
    return d
