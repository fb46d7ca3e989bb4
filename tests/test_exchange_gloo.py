"""The one-model-per-worker protocol (paper_2405_17517_b200.exchange.ExchangeWorker) on CPU
ranks over gloo.  The ranks run the real protocol code -- capacity agreement, exchange of
buffer handles, plan / send / barrier / receive with two alternating staging sets -- with the
oracle's worker functions standing in for the kernels and named shared memory standing in
for peer-mapped device buffers.  Gathered together, the workers' rows must equal the
oracle's population shuffle after every step."""
import os
import socket
from multiprocessing import shared_memory

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2405_17517_b200 import workloads as W
from paper_2405_17517_b200.exchange import ExchangeWorker, WASH_STACK_OPT, WASH_STACK_PARAMS

NUMEL = [3001, 64, 7, 1200]
P_LAYER = [0.3, 1.0, 0.5, 0.02]


class OracleOps:
    """The calls ExchangeWorker makes, implemented by the oracle over numpy rows."""

    def __init__(self):
        self.shms = []

    def create(self, N, numel):
        off, P = W.padded_offsets(numel)
        return {"pop": oracle.Population(N, numel, off, P, 0), "rows": {}, "staging": {}, "own": {}, "plan": None, "N": N}

    def row_elems(self, ctx, n_tensors):
        return ctx["pop"].padded_P

    def bind(self, ctx, rank, stack, row):
        ctx["rank"] = rank
        ctx["rows"][stack] = row

    def staging_create(self, ctx, stack, parity, capacity):
        dt = ctx["rows"][stack].dtype
        shm = shared_memory.SharedMemory(create=True, size=capacity * dt.itemsize)
        self.shms.append((shm, True))
        ctx["own"][(stack, parity)] = np.ndarray(capacity, dtype=dt, buffer=shm.buf)
        ctx["cap"] = capacity
        return shm.name.encode()

    def staging_open(self, ctx, stack, parity, handles):
        bufs = []
        for n, h in enumerate(handles):
            if n == ctx["rank"]:
                bufs.append(ctx["own"][(stack, parity)])
                continue
            shm = shared_memory.SharedMemory(name=h.decode())
            self.shms.append((shm, False))
            bufs.append(np.ndarray(ctx["cap"], dtype=ctx["rows"][stack].dtype, buffer=shm.buf))
        ctx["staging"][(stack, parity)] = bufs

    def plan(self, ctx, step, p, p_layer, seed):
        ctx["plan"] = (step, p if p_layer is None else p_layer, seed)

    def send(self, ctx):
        step, probs, seed = ctx["plan"]
        for stack, row in ctx["rows"].items():
            oracle.exchange_send(ctx["pop"], ctx["rank"], row, probs, seed, step, ctx["staging"][(stack, step & 1)])

    def receive(self, ctx, stats):
        step, probs, seed = ctx["plan"]
        for stack, row in ctx["rows"].items():
            st = oracle.exchange_receive(ctx["pop"], ctx["rank"], row, probs, seed, step,
                                         ctx["staging"][(stack, step & 1)][ctx["rank"]])
            if stats is not None and stack == WASH_STACK_PARAMS:
                stats[0] += st[0]
                stats[1] += st[1]

    def check(self, ctx):
        pass

    def barrier(self, group, token):
        dist.barrier(group=group)

    def barrier_token(self, group):
        return None

    def flush(self):
        pass

    def destroy(self, ctx):
        ctx["staging"].clear()
        ctx["own"].clear()
        for shm, mine in self.shms:
            shm.close()
            if mine:
                shm.unlink()
        self.shms = []


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, steps, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        off, P = W.padded_offsets(NUMEL)
        stack = W.to_stack(W.flat_population(world, sum(NUMEL), seed=31), NUMEL, off, P, 0)
        mom = W.to_stack(W.flat_population(world, sum(NUMEL), seed=32, std=1e-3), NUMEL, off, P, 0)
        row = stack.reshape(world, P)[rank].copy()
        opt = mom.reshape(world, P)[rank].copy()
        # ranks propose different capacities; the smallest must win
        worker = ExchangeWorker(NUMEL, row, opt, capacity=P + 8 * rank, ops=OracleOps())
        assert worker.capacity == P
        pop = oracle.Population(world, NUMEL, off, P, 0)
        ok, stats = True, [0, 0]
        want_sel = want_moved = 0
        for step in range(steps):
            worker.step(step, 0.0, P_LAYER, seed=13, stats=stats)
            rows = [None] * world
            dist.all_gather_object(rows, (row.copy(), opt.copy(), stats[1]))
            sel, moved = oracle.shuffle(pop, stack, P_LAYER, seed=13, step=step, stack2=mom)
            want_sel += sel
            want_moved += moved
            got = np.stack([r[0] for r in rows]).reshape(-1)
            got_m = np.stack([r[1] for r in rows]).reshape(-1)
            ok = ok and (got.view(np.uint32) == stack.reshape(-1).view(np.uint32)).all()
            ok = ok and (got_m.view(np.uint32) == mom.reshape(-1).view(np.uint32)).all()
            ok = ok and stats[0] == want_sel and sum(r[2] for r in rows) == want_moved
        worker.close()
        if rank == 0:
            with open(os.path.join(out_dir, "result.txt"), "w") as f:
                f.write("ok" if ok and want_moved > 0 else "mismatch")
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_workers_over_gloo_reproduce_the_population_shuffle(world, tmp_path):
    oracle.build()
    mp.spawn(_rank_main, args=(world, _free_port(), 4, str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "result.txt").read_text() == "ok"
