"""The shuffling step with one model per worker (wash_exchange_*), on one GPU: N contexts,
one per worker, each bound to one row of a stack, with N staging buffers on the same
device standing for the peers' buffers.  No kernel waits for another: every worker's send
is launched, then every worker's receive, in stream order.  The result must be the
oracle's population shuffle bit for bit, and the staging buffers the oracle's wire format."""
import numpy as np
import pytest
import torch

import oracle
from paper_2405_17517_b200 import binding as B
from paper_2405_17517_b200 import workloads as W
from gpu_util import bits, to_device, to_host_bits

pytestmark = pytest.mark.gpu


class Workers:
    def __init__(self, N, numel, dtype="f32", opt_dtype=None, seed=0, capacity=None, parities=(0,), tensor_id=None,
                 coord_begin=None):
        self.N, self.numel = N, [int(d) for d in numel]
        self.ctx = [B.wash_create_segments(N, self.numel, tensor_id, coord_begin, 0, 0) for _ in range(N)]
        self.P, self.off = B.wash_stack_elems(self.ctx[0], len(self.numel))
        self.ora = oracle.Population(N, self.numel, self.off, self.P, 0, tensor_id, coord_begin)
        total = sum(self.numel)
        dense = W.flat_population(N, total, seed=seed)
        if dtype == "bf16":
            dense = W.to_bf16_bits(dense)
        self.host = [W.to_stack(dense, self.numel, self.off, self.P, 0)]
        if opt_dtype is not None:
            d2 = W.flat_population(N, total, seed=seed + 99, std=1e-3)
            if opt_dtype == "bf16":
                d2 = W.to_bf16_bits(d2)
            self.host.append(W.to_stack(d2, self.numel, self.off, self.P, 0))
        self.dev = [to_device(h) for h in self.host]
        self.capacity = self.P if capacity is None else capacity
        self.guard = 64   # elements after every staging buffer that nothing may touch
        self.staging = {}
        for k, d in enumerate(self.dev):
            eb = d.element_size()
            for n in range(N):
                B.wash_exchange_bind(self.ctx[n], n, k, B._torch_dtype_code(d), d.data_ptr() + n * self.P * eb, self.P)
            for par in parities:
                bufs = [self._fill(torch.empty(self.capacity + self.guard, dtype=d.dtype, device="cuda")) for _ in range(N)]
                self.staging[(par, k)] = bufs
                for n in range(N):
                    B.wash_exchange_staging(self.ctx[n], k, par, bufs, self.capacity)
        self.stats = torch.zeros(N, 2, dtype=torch.int64, device="cuda")

    @staticmethod
    def _fill(t):
        (t.view(torch.int16) if t.dtype == torch.bfloat16 else t.view(torch.int32)).fill_(0x7A7A)
        return t

    def step(self, step, p, p_layer=None, seed=0):
        for n in range(self.N):
            B.wash_exchange_plan(self.ctx[n], step, p, p_layer, seed)
        for n in range(self.N):
            B.wash_exchange_send(self.ctx[n])
        for n in range(self.N):
            B.wash_exchange_receive(self.ctx[n], None, self.stats[n])

    def check(self):
        torch.cuda.synchronize()
        for c in self.ctx:
            B.wash_check(c)

    def close(self):
        for c in self.ctx:
            B.wash_destroy(c)


def _staging_bits(t):
    return to_host_bits(t)


@pytest.mark.parametrize("N,dtype,opt_dtype", [(2, "f32", None), (3, "f32", "f32"), (5, "bf16", "f32"), (8, "bf16", "bf16"),
                                               (16, "f32", None), (17, "f32", "f32"), (64, "f32", None)])
def test_workers_reproduce_the_population_shuffle(N, dtype, opt_dtype):
    numel = [5000, 3, 1027, 64, 2500]
    w = Workers(N, numel, dtype, opt_dtype, seed=N)
    p_layer = [0.05, 1.0, 0.3, 0.0, 0.01]
    sel_total = 0
    need_total = np.zeros(N, dtype=np.int64)
    need_max = np.zeros(N, dtype=np.int64)
    for step in (0, 1, (1 << 40) + 5):
        start = [h.copy() for h in w.host]
        w.step(step, 0.0, p_layer, seed=21)
        sel, moved = oracle.shuffle(w.ora, w.host[0], p_layer, seed=21, step=step,
                                    stack2=w.host[1] if opt_dtype else None)
        need, sel_c = oracle.exchange_counts(w.ora, p_layer, seed=21, step=step)
        w.check()
        for k in range(len(w.host)):
            got, want = to_host_bits(w.dev[k]), bits(w.host[k])
            bad = np.flatnonzero(got != want)
            assert bad.size == 0, "stack %d step %d: %d elements differ, first %d" % (k, step, bad.size, bad[0])
        for n in range(N):
            g_need, g_sel = B.wash_exchange_counts(w.ctx[n], N)
            assert g_need == need.tolist() and g_sel == sel == sel_c
        # wire format: the staging buffers hold what the oracle's workers would have stored
        for k in range(len(w.host)):
            rows = [start[k].reshape(N, w.P)[n] for n in range(N)]
            ora_staging = [np.zeros(w.capacity, dtype=rows[0].dtype) for _ in range(N)]
            for n in range(N):
                oracle.exchange_send(w.ora, n, rows[n], p_layer, 21, step, ora_staging)
            for n in range(N):
                got = _staging_bits(w.staging[(0, k)][n])
                assert (got[:need[n]] == bits(ora_staging[n])[:need[n]]).all()
                need_max[n] = max(need_max[n], need[n])
                assert (got[need_max[n]:] == 0x7A7A).all()      # slots no step needed stay untouched
        sel_total += sel
        need_total += need
    st = w.stats.cpu().numpy()
    assert (st[:, 0] == sel_total).all() and (st[:, 1] == need_total).all()
    w.close()


@pytest.mark.parametrize("p", [1.0, 0.6])
@pytest.mark.parametrize("N", [3, 20])
def test_dense_selection_needs_several_passes_over_a_tile(N, p):
    """More selected coordinates in a tile than the send kernel lists at once."""
    w = Workers(N, [9000, 5, 4099], "f32", "f32", seed=50 + N)
    for step in (0, 3):
        w.step(step, p, None, seed=6)
        oracle.shuffle(w.ora, w.host[0], p, seed=6, step=step, stack2=w.host[1])
    w.check()
    for k in range(2):
        assert (to_host_bits(w.dev[k]) == bits(w.host[k])).all()
    need, sel = oracle.exchange_counts(w.ora, p, seed=6, step=3)
    assert B.wash_exchange_counts(w.ctx[1], N) == (need.tolist(), sel)
    w.close()


def test_resnet_rows_with_the_layer_schedule():
    """ResNet-18 tensor table, N = 5, the default layer-wise schedule, parameters and momentum."""
    numel = W.numels(W.resnet18_table(100))
    N = 5
    w = Workers(N, numel, "f32", "f32", seed=3, capacity=1 << 17)
    pl = B.wash_layer_probs(len(numel), 0.01, 0)
    for step in (0, 1):
        w.step(step, 0.0, pl, seed=5)
        oracle.shuffle(w.ora, w.host[0], pl, seed=5, step=step, stack2=w.host[1])
    w.check()
    for k in range(2):
        assert (to_host_bits(w.dev[k]) == bits(w.host[k])).all()
    w.close()


def test_two_staging_sets_alternate_by_step():
    N, numel = 4, [3000, 40]
    w = Workers(N, numel, "f32", None, seed=8, parities=(0, 1))
    for step in range(4):
        before = [to_host_bits(b).copy() for b in w.staging[((step + 1) & 1, 0)]]
        w.step(step, 0.2, None, seed=2)
        oracle.shuffle(w.ora, w.host[0], 0.2, seed=2, step=step)
        w.check()
        assert (to_host_bits(w.dev[0]) == bits(w.host[0])).all()
        for n in range(N):   # the other set is left alone
            assert (to_host_bits(w.staging[((step + 1) & 1, 0)][n]) == before[n]).all()
    w.close()


def test_too_small_a_staging_buffer_is_reported_and_nothing_is_written_beyond_it():
    N, numel = 3, [20000]
    need, _ = oracle.exchange_counts(oracle.Population(N, numel), 0.5, seed=1, step=0)
    cap = int(need.min()) // 2
    w = Workers(N, numel, "f32", None, seed=9, capacity=cap)
    w.step(0, 0.5, None, seed=1)
    torch.cuda.synchronize()
    with pytest.raises(B.WashError) as e:
        B.wash_check(w.ctx[0])
    assert e.value.code == B.WASH_ERR_DEVICE_CHECK and "staging" in str(e.value)
    for n in range(N):
        assert (to_host_bits(w.staging[(0, 0)][n])[cap:] == 0x7A7A).all()
    w.close()


def test_slices_of_a_model_exchange_like_the_whole_model():
    """A worker may hold a slice of every tensor (coordinate sharding inside a worker): the
    draws are keyed by (tensor, coordinate), so the slice gets the whole model's bits."""
    N, d = 3, 40000
    full = Workers(N, [d], "f32", None, seed=4)
    part = Workers(N, [12000], "f32", None, seed=4, tensor_id=[0], coord_begin=[20000])
    # give the slice workers the matching values
    src = full.dev[0].view(N, full.P)[:, 20000:32000]
    part.dev[0].view(N, part.P)[:, :12000].copy_(src)
    full.step(6, 0.1, None, seed=3)
    part.step(6, 0.1, None, seed=3)
    full.check(); part.check()
    a = to_host_bits(full.dev[0]).reshape(N, full.P)[:, 20000:32000]
    b = to_host_bits(part.dev[0]).reshape(N, part.P)[:, :12000]
    assert (a == b).all()
    full.close(); part.close()


def test_state_errors_are_reported_before_any_launch():
    ctx = B.wash_create_segments(3, [64], None, None, 0, 0)
    with pytest.raises(B.WashError) as e:
        B.wash_exchange_plan(ctx, 0, 0.1)
    assert e.value.code == B.WASH_ERR_STATE
    row = torch.zeros(64, device="cuda")
    with pytest.raises(B.WashError):
        B.wash_exchange_bind(ctx, 3, 0, B.WASH_F32, row, 64)
    with pytest.raises(B.WashError):
        B.wash_exchange_bind(ctx, 1, 0, B.WASH_F32, row, 63)
    B.wash_exchange_bind(ctx, 1, 0, B.WASH_F32, row, 64)
    with pytest.raises(B.WashError) as e:
        B.wash_exchange_send(ctx)
    assert e.value.code == B.WASH_ERR_STATE          # nothing planned
    B.wash_exchange_plan(ctx, 0, 0.1)
    with pytest.raises(B.WashError) as e:
        B.wash_exchange_send(ctx)
    assert e.value.code == B.WASH_ERR_STATE          # no staging buffers
    with pytest.raises(B.WashError):
        B.wash_exchange_bind(ctx, 2, 0, B.WASH_F32, row, 64)   # already worker 1
    torch.cuda.synchronize()
    B.wash_destroy(ctx)


# ---- workers in separate processes: buffers mapped through inter-process handles ----------
# Two processes share the one GPU; they are ordered on the host (gloo), no kernel waits for
# another process's kernel.

def _process_worker(rank, world, port, out_dir):
    import os
    import torch.distributed as dist
    from paper_2405_17517_b200.exchange import ExchangeWorker
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        torch.cuda.set_device(0)
        numel = [70001, 9, 4000]
        off, P = W.padded_offsets(numel)
        stack = W.to_stack(W.flat_population(world, sum(numel), seed=41), numel, off, P, 0)
        mom = W.to_stack(W.flat_population(world, sum(numel), seed=42, std=1e-3), numel, off, P, 0)
        row = to_device(stack.reshape(world, P)[rank])
        opt = to_device(mom.reshape(world, P)[rank])
        stats = torch.zeros(2, dtype=torch.int64, device="cuda")
        worker = ExchangeWorker(numel, row, opt, capacity=P // 2)
        # a set of peers' buffers is mapped once: a second open is refused and changes nothing
        refused = False
        try:
            B.wash_exchange_staging_open(worker.ctx, 0, 0, worker.handles[(0, 0)])
        except B.WashError as err:
            refused = err.code == B.WASH_ERR_STATE
        pop = oracle.Population(world, numel, off, P, 0)
        pl = [0.05, 1.0, 0.2]
        ok = refused
        for step in range(3):
            worker.step(step, 0.0, pl, seed=17, stats=stats)
            torch.cuda.synchronize()
            worker.check()
            rows = [None] * world
            dist.all_gather_object(rows, (to_host_bits(row), to_host_bits(opt), int(stats[1].item())))
            sel, moved = oracle.shuffle(pop, stack, pl, seed=17, step=step, stack2=mom)
            ok = ok and (np.concatenate([r[0] for r in rows]) == bits(stack)).all()
            ok = ok and (np.concatenate([r[1] for r in rows]) == bits(mom)).all()
        worker.close()
        if rank == 0:
            with open(os.path.join(out_dir, "result.txt"), "w") as f:
                f.write("ok" if ok else "mismatch")
    finally:
        dist.destroy_process_group()


def test_workers_in_two_processes_exchange_through_mapped_buffers(tmp_path):
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_process_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    assert (tmp_path / "result.txt").read_text() == "ok"


def test_bench_arm_with_two_ranks_on_one_device():
    """bench.py --exchange-ranks under torchrun with two ranks that share the one GPU (gloo,
    barrier on the host): the step runs through ExchangeWorker and the plan's slot counts
    equal the oracle's."""
    import json
    import os
    import socket
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.join(root, "bench.py"), "--gpus", "2", "--exchange-ranks", "--workload",
           "cfg2_resnet18_n5", "--steps", "4", "--warmup", "3"]
    res = subprocess.run(cmd, capture_output=True, text=True, cwd=root, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    line = [json.loads(ln) for ln in res.stdout.splitlines() if ln.startswith("{")][-1]
    assert line["arm"] == "exchange-ranks" and line["ranks"] == 2
    assert line["counts_match_oracle"] is True
    expect = line["expected_values_per_rank_per_step"]
    assert abs(line["values_received_per_rank_per_step"] - expect) < 6 * expect ** 0.5
