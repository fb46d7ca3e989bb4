"""The multi-GPU path is "shards, no collective": its host logic (who owns which
coordinates, which probabilities go with them) is exercised here with two CPU ranks over
gloo.  Each rank shuffles only its own shard with the oracle, keyed by global (tensor,
coordinate); gathered together the shards must equal the unsharded shuffle bit for bit."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2405_17517_b200 import sharding
from paper_2405_17517_b200 import workloads as W

NUMEL = [4001, 64, 7, 1200, 3, 36, 2048]
N = 4
P_LAYER = oracle.layer_probs(len(NUMEL), 0.6).tolist()[:-1] + [0.3]


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, steps, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        dense = W.flat_population(N, sum(NUMEL), seed=11)              # every rank can build the full input
        mom = W.flat_population(N, sum(NUMEL), seed=12, std=1e-3)
        segs = sharding.plan_shards(NUMEL, world)[rank]
        numel, tensor_id, coord_begin = sharding.segment_arrays(segs)
        cols = sharding.dense_slices(NUMEL, segs)
        mine = np.ascontiguousarray(np.concatenate([dense[:, c] for c in cols], axis=1))
        mine_m = np.ascontiguousarray(np.concatenate([mom[:, c] for c in cols], axis=1))
        pop = oracle.Population(N, numel, tensor_id=tensor_id, coord_begin=coord_begin)
        probs = sharding.segment_probs(P_LAYER, segs)
        sel = 0
        for step in range(steps):
            sel += oracle.shuffle(pop, mine, probs, seed=5, step=step, stack2=mine_m)[0]
        gathered = [None] * world
        dist.all_gather_object(gathered, (segs, mine, mine_m, sel))
        if rank == 0:
            full = dense.copy(); full_m = mom.copy(); total_sel = 0
            for segs_r, vals, vals_m, sel_r in gathered:
                pos = 0
                for c in sharding.dense_slices(NUMEL, segs_r):
                    w = c.stop - c.start
                    full[:, c] = vals[:, pos:pos + w]; full_m[:, c] = vals_m[:, pos:pos + w]
                    pos += w
                total_sel += sel_r
            ref = dense.copy(); ref_m = mom.copy()
            whole = oracle.Population(N, NUMEL)
            ref_sel = 0
            for step in range(steps):
                ref_sel += oracle.shuffle(whole, ref, P_LAYER, seed=5, step=step, stack2=ref_m)[0]
            ok = (full.view(np.uint32) == ref.view(np.uint32)).all() and (full_m.view(np.uint32) == ref_m.view(np.uint32)).all() \
                and total_sel == ref_sel and ref_sel > 0
            with open(os.path.join(out_dir, "result.txt"), "w") as f:
                f.write("ok" if ok else "mismatch")
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_shards_over_gloo_reproduce_the_unsharded_shuffle(world, tmp_path):
    oracle.build()
    mp.spawn(_rank_main, args=(world, _free_port(), 3, str(tmp_path)), nprocs=world, join=True)
    assert (tmp_path / "result.txt").read_text() == "ok"


def test_plan_properties():
    for numel in ([10], [1, 1, 1], NUMEL, [4, 4, 4, 4], [1000003, 17]):
        total = sum(numel)
        for world in (1, 2, 3, 8, 64):
            plans = sharding.plan_shards(numel, world)
            assert len(plans) == world
            covered = np.zeros(total, dtype=np.int32)
            for segs in plans:
                for c in sharding.dense_slices(numel, segs):
                    covered[c] += 1
                for t, c0, cnt in segs:
                    assert c0 % 4 == 0 and cnt > 0 and c0 + cnt <= numel[t]
            assert (covered == 1).all()
            sizes = [sum(s[2] for s in segs) for segs in plans]
            assert max(sizes) - min(sizes) <= 8        # every cut moves down by fewer than 4 coordinates
    with pytest.raises(ValueError):
        sharding.plan_shards([4, 0], 2)
