"""One worker of a population trained one model per process / GPU: the host-side protocol
around the wash_exchange_* kernels.

The paper's deployment (Introduction; Algorithm 1) keeps model n on worker n and shuffles a
few parameters peer to peer after every training step.  Here a process group of N ranks is
the population; rank n is worker n.  Set-up exchanges the inter-process handles of the
staging buffers once (an all-gather of 64-byte handles over the group); a step is

    plan (every rank draws the same mask and permutations)  ->  send (peer stores into the
    other ranks' staging buffers)  ->  one barrier  ->  receive (copy own slots in)

Two staging sets alternate by step parity, which is why one barrier per step is enough: a
rank can only reach the send of step s+2 after the barrier of step s+1, which every rank
enters after its own receive of step s.

The arithmetic is in the library's kernels; this module only orders calls.  `ops` is the
set of entry points used (the ctypes binding by default), so that the protocol itself can
be exercised on CPU ranks with another implementation of the same calls.
"""
from __future__ import annotations

from typing import Optional, Sequence

import torch
import torch.distributed as dist

WASH_STACK_PARAMS, WASH_STACK_OPT = 0, 1


class CudaOps:
    """The C entry points (paper_2405_17517_b200.binding), rows being CUDA tensors."""

    def __init__(self, device: int):
        from . import binding
        self.B = binding
        self.device = device

    def create(self, N, numel):
        return self.B.wash_create_segments(N, numel, None, None, 0, self.device)

    def destroy(self, ctx):
        self.B.wash_destroy(ctx)

    def row_elems(self, ctx, n_tensors):
        return self.B.wash_stack_elems(ctx, n_tensors)[0]

    def bind(self, ctx, rank, stack, row):
        if not row.is_cuda or not row.is_contiguous():
            raise ValueError("a model row must be a contiguous CUDA tensor")
        self.B.wash_exchange_bind(ctx, rank, stack, self.B._torch_dtype_code(row), row, row.numel())

    def staging_create(self, ctx, stack, parity, capacity):
        return self.B.wash_exchange_staging_create(ctx, stack, parity, capacity)

    def staging_open(self, ctx, stack, parity, handles):
        self.B.wash_exchange_staging_open(ctx, stack, parity, handles)

    def plan(self, ctx, step, p, p_layer, seed):
        self.B.wash_exchange_plan(ctx, step, p, p_layer, seed)

    def send(self, ctx):
        self.B.wash_exchange_send(ctx)

    def receive(self, ctx, stats):
        self.B.wash_exchange_receive(ctx, None, stats)

    def check(self, ctx):
        self.B.wash_check(ctx)

    def barrier(self, group, token):
        """All ranks' sends are complete (and visible) before any rank's receive runs."""
        if token is not None:
            # a collective on the current stream: ordered after this rank's send kernel and
            # before its receive kernel without stalling the host
            dist.all_reduce(token, group=group)
        else:
            torch.cuda.current_stream().synchronize()
            dist.barrier(group=group)

    def flush(self):
        torch.cuda.synchronize(self.device)

    def barrier_token(self, group):
        if dist.get_backend(group) == "nccl":
            return torch.zeros(1, dtype=torch.int32, device="cuda:%d" % self.device)
        return None


class ExchangeWorker:
    """Rank `dist.get_rank(group)` of a population of `dist.get_world_size(group)` models."""

    def __init__(self, numel: Sequence[int], row, opt_row=None, capacity: Optional[int] = None, group=None,
                 ops=None, device: Optional[int] = None):
        self.group = group
        self.rank = dist.get_rank(group)
        self.N = dist.get_world_size(group)
        if self.N < 2:
            raise ValueError("a population needs at least two workers")
        if ops is None:
            ops = CudaOps(torch.cuda.current_device() if device is None else device)
        self.ops = ops
        self.numel = [int(d) for d in numel]
        self.ctx = ops.create(self.N, self.numel)
        self.padded_P = ops.row_elems(self.ctx, len(self.numel))
        self.rows = {WASH_STACK_PARAMS: row}
        if opt_row is not None:
            self.rows[WASH_STACK_OPT] = opt_row
        # every rank must use the same capacity: agree on the smallest proposal
        cap = self.padded_P if capacity is None else int(capacity)
        caps = [None] * self.N
        dist.all_gather_object(caps, cap, group=group)
        self.capacity = min(caps)
        if self.capacity < 1:
            raise ValueError("staging capacity must be positive")
        for stack, r in self.rows.items():
            ops.bind(self.ctx, self.rank, stack, r)
        self.handles = {}    # (stack, parity) -> the N workers' buffer handles, as exchanged
        for stack in self.rows:
            for parity in (0, 1):
                mine = ops.staging_create(self.ctx, stack, parity, self.capacity)
                handles = [None] * self.N
                dist.all_gather_object(handles, mine, group=group)
                ops.staging_open(self.ctx, stack, parity, handles)
                self.handles[(stack, parity)] = handles
        self._token = ops.barrier_token(group)
        dist.barrier(group=group)   # every rank has mapped every buffer

    def step(self, step: int, p: float, p_layer=None, seed: int = 0, stats=None) -> None:
        """One shuffling step; `stats` (optional) as for wash_exchange_receive."""
        ops = self.ops
        ops.plan(self.ctx, step, p, p_layer, seed)
        ops.send(self.ctx)
        ops.barrier(self.group, self._token)
        ops.receive(self.ctx, stats)

    def check(self) -> None:
        self.ops.check(self.ctx)

    def close(self) -> None:
        """Collective: every rank must have finished its last step before any mapping goes."""
        if self.ctx is not None:
            self.ops.flush()
            dist.barrier(group=self.group)
            self.ops.destroy(self.ctx)
            self.ctx = None
