#!/usr/bin/env python
"""Benchmark of the WASH hot path on B200: one JSON line on stdout.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg2_resnet18_n5|cfg3_resnet50_n10|cfg4_resnet50_bf16_n8|cfg1_flat_n3]

A step is one pass of the whole hot path over one synthetic population: the shuffle of
the parameter and momentum stacks (WASH+Opt, one launch), PAPA's EMA on the parameters
and the final average -- three kernel launches.  `value` is the bytes those kernels
must stream (see algorithmic_bytes) divided by the step time, in GB/s, with the stacks
resident in HBM; `e2e` is the same through wash_step_host with the stacks in pinned
host memory (copies inside the timed region).  For N > 1 (torchrun) every rank holds
its own shard of an N-times deeper population (tensor indices offset by rank), no
communication: weak scaling.

--impl reference times the CPU oracle (oracle/) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_17517_b200 import workloads as W  # noqa: E402

METRIC = "shuffle GB/s and parameter-swaps/s at 1 B200; % of HBM roofline"
FALLBACK_HBM_GBS = 6650.0
ALPHA = 0.99
SEED = 0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (no MEASURED_PEAKS.json)"


class Workload:
    def __init__(self, name: str, rank: int = 0):
        cfg = W.CONFIGS[name]
        self.name, self.cfg = name, cfg
        self.N = cfg["N"]
        self.table = W.table_from_spec(cfg["table"])
        self.numel = W.numels(self.table)
        self.T = len(self.table)
        self.P = int(self.numel.sum())
        self.p = cfg["p"]
        self.bf16 = cfg["dtype"] == "bf16"
        self.opt = cfg["opt"]
        self.E = 2 if self.bf16 else 4
        self.E_opt = 4 if self.opt else 0
        # rank r holds tensors r*T .. r*T+T-1 of a world_size-times deeper population
        self.tensor_id = np.arange(self.T, dtype=np.uint32) + np.uint32(rank * self.T)
        self.schedule = cfg["schedule"]     # None = uniform p; each arm derives p_layer with its own routine
        self.p_layer = None
        self.rank = rank

    def algorithmic_bytes(self, selected: float) -> dict:
        """Bytes each kernel must move per launch (logical coordinates only)."""
        N, P = self.N, self.P
        shuffle = N * P * (self.E + self.E_opt) + selected * N * (self.E + self.E_opt)   # read all, write selected
        ema = 2 * N * P * self.E
        avg = N * P * self.E + P * self.E
        return {"shuffle": shuffle, "ema": ema, "average": avg, "step": shuffle + ema + avg}

    def host_stacks(self, offsets, padded_P):
        dense = W.init_population(self.table, self.N, seed=SEED + 17 * self.rank) if self.T > 1 else \
            W.flat_population(self.N, self.P, seed=SEED + 17 * self.rank, std=0.05)
        if self.bf16:
            dense = W.to_bf16_bits(dense)
        params = W.to_stack(dense, self.numel, offsets, padded_P)
        opt = None
        if self.opt:
            opt = W.to_stack(W.init_momentum(self.table, self.N, seed=SEED + 1 + 17 * self.rank), self.numel, offsets, padded_P)
        return params, opt


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons (read-only NVML queries) while running."""

    def __init__(self, index: int, period: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self) -> dict:
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


# ------------------------------------------------------------------------------------
def run_reference(args, rank: int, world: int) -> None:
    """The CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import oracle
    wl = Workload(args.workload, 0)
    offsets, padded_P = W.padded_offsets(wl.numel)
    threads = oracle.max_threads()
    oracle.set_threads(threads)
    params, opt = wl.host_stacks(offsets, padded_P)
    if wl.schedule == "decreasing":
        wl.p_layer = oracle.layer_probs(wl.T, wl.p, oracle.SCHEDULE_DECREASING)

    def one_step(pop, a, b, out, step, p_layer):
        p = wl.p if p_layer is None else p_layer
        st = oracle.shuffle(pop, a, p, seed=SEED, step=step, stack2=b)
        oracle.papa_ema(pop, a, ALPHA)
        oracle.population_average(pop, a, out)
        return st

    full = oracle.Population(wl.N, wl.numel, offsets, padded_P, oracle.LAYOUT_NP, wl.tensor_id)
    out = np.zeros(padded_P, dtype=params.dtype)
    t0 = time.perf_counter()
    one_step(full, params, opt, out, 0, wl.p_layer)
    t_full = time.perf_counter() - t0
    # bounded sample: a prefix of the tensor table, so that warmup + steps stay near a minute
    budget = 60.0
    frac = min(1.0, budget / max(t_full * (args.steps + args.warmup), 1e-9))
    cum = np.cumsum(wl.numel)
    n_t = int(np.searchsorted(cum, frac * wl.P, side="left")) + 1 if frac < 1.0 else wl.T
    n_t = max(1, min(wl.T, n_t))
    sub_numel = wl.numel[:n_t]
    sub_P = int(sub_numel.sum())
    sub_off, sub_padded = W.padded_offsets(sub_numel)
    rows = params.reshape(wl.N, padded_P)
    sp = np.ascontiguousarray(rows[:, :sub_padded])
    so = np.ascontiguousarray(opt.reshape(wl.N, padded_P)[:, :sub_padded]) if opt is not None else None
    sub = oracle.Population(wl.N, sub_numel, sub_off, sub_padded, oracle.LAYOUT_NP, wl.tensor_id[:n_t])
    sub_pl = None if wl.p_layer is None else wl.p_layer[:n_t]
    sout = np.zeros(sub_padded, dtype=params.dtype)
    for w in range(args.warmup):
        one_step(sub, sp, so, sout, w, sub_pl)
    sel = 0
    t0 = time.perf_counter()
    for k in range(args.steps):
        sel += one_step(sub, sp, so, sout, args.warmup + k, sub_pl)[0]
    dt = time.perf_counter() - t0
    scale = sub_P / wl.P
    bytes_step = wl.algorithmic_bytes(sel / max(args.steps, 1) / scale)["step"] * scale
    gbs = bytes_step * args.steps / dt / 1e9
    sample = "first %d of %d tensors (%d of %d coordinates per model) per step" % (n_t, wl.T, sub_P, wl.P)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16+f32" if wl.bf16 else "f32", "data": "synthetic",
        "config": {"workload": wl.name, "N": wl.N, "tensors": wl.T, "P": wl.P, "p": wl.p, "sample": sample},
        "param_swaps_per_s": sel * wl.N / dt,
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------
def run_ours(args, rank: int, world: int, local_rank: int) -> None:
    import torch
    from paper_2405_17517_b200 import binding as B

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    if not os.path.exists(B.LIB_PATH):
        if rank == 0:
            from paper_2405_17517_b200 import build as wash_build
            wash_build.build()
    dist = None
    if world > 1 or os.environ.get("WASH_BENCH_DIST") == "1":   # the second form exercises the multi-rank path on one GPU
        import torch.distributed as dist_mod
        dist = dist_mod
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    else:
        torch.cuda.set_device(local_rank)
    B.load()
    dev = local_rank
    wl = Workload(args.workload, rank)
    pop = B.Population(wl.N, wl.numel, B.WASH_LAYOUT_NP, dev, wl.tensor_id)
    params_h, opt_h = wl.host_stacks(pop.offsets, pop.padded_P)

    def to_torch(a):
        t = torch.from_numpy(a.reshape(-1).view(np.int16) if a.dtype == np.uint16 else a.reshape(-1))
        return t.view(torch.bfloat16) if a.dtype == np.uint16 else t

    params_pin = to_torch(params_h).pin_memory()
    opt_pin = to_torch(opt_h).pin_memory() if opt_h is not None else None
    params_d = params_pin.cuda(non_blocking=True)
    opt_d = opt_pin.cuda(non_blocking=True) if opt_pin is not None else None
    avg_d = torch.zeros(pop.padded_P, dtype=params_d.dtype, device="cuda")
    avg_pin = torch.zeros(pop.padded_P, dtype=params_d.dtype).pin_memory()
    stats_d = torch.zeros(2, dtype=torch.int64, device="cuda")
    pop.bind(B.WASH_STACK_PARAMS, params_d)
    if opt_d is not None:
        pop.bind(B.WASH_STACK_OPT, opt_d)
    if args.mode != "stream":
        B.wash_set_mode(pop.ctx, {"sparse": B.WASH_MODE_SPARSE, "staged": B.WASH_MODE_STREAM_STAGED, "registers": B.WASH_MODE_STREAM_REGISTERS}[args.mode])
    if args.threads or args.blocks_per_sm:
        B.wash_set_launch(pop.ctx, args.threads, args.blocks_per_sm)
    pdt = B.WASH_BF16 if wl.bf16 else B.WASH_F32
    if wl.schedule == "decreasing":
        wl.p_layer = B.wash_layer_probs(wl.T, wl.p, B.WASH_SCHEDULE_DECREASING)
    p_layer = wl.p_layer
    stream = torch.cuda.current_stream()

    def step_shuffle(i):
        if opt_d is not None:
            B.wash_shuffle_both(pop.ctx, i, wl.p, p_layer, SEED, stream, stats_d)
        else:
            B.wash_shuffle(pop.ctx, i, wl.p, p_layer, SEED, stream, stats_d)

    def step(i, ev=None):
        if ev is not None:
            ev[0].record(stream)
        step_shuffle(i)
        if ev is not None:
            ev[1].record(stream)
        B.papa_ema(pop.ctx, B.WASH_STACK_PARAMS, ALPHA, stream)
        if ev is not None:
            ev[2].record(stream)
        B.population_average(pop.ctx, B.WASH_STACK_PARAMS, avg_d, pdt, stream)
        if ev is not None:
            ev[3].record(stream)

    def fence():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for w in range(args.warmup):
        step(w)
    fence()
    stats_d.zero_()
    launches0 = B.wash_launch_count()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(args.steps)]
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    fence()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for k in range(args.steps):
        step(args.warmup + k, events[k] if args.inline_kernel_events else None)
    t_end.record(stream)
    fence()
    clocks = sampler.stop()
    launches = B.wash_launch_count() - launches0
    B.wash_check(pop.ctx)
    total_ms = t_begin.elapsed_time(t_end)
    st = stats_d.cpu().numpy().view(np.uint64)
    selected_total, moved_total = int(st[0]), int(st[1])
    if not args.inline_kernel_events:
        # Per-kernel times come from a second, instrumented pass over the same steps' work:
        # an event between every two launches costs the step about 5 % (measured), so the
        # timed region above carries none.
        fence()
        for k in range(min(args.steps, 300)):
            step(args.warmup + args.steps + k, events[k])
        fence()
        events = events[:min(args.steps, 300)]
    k_ms = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(3)] for e in events])   # shuffle, ema, average
    mean_ms = k_ms.mean(axis=0)

    # ---- the shuffle alone, launched back to back (no event between launches), in the
    # streaming mode and in the sparse mode: context for the per-kernel figures above, which
    # carry an event pair per launch, and the parameter-swaps/s the sparse kernel reaches
    def shuffle_alone(mode, n):
        B.wash_set_mode(pop.ctx, mode)
        first = args.warmup + 2 * args.steps + 1000
        for k in range(3):
            step_shuffle(first + k)
        fence()
        a0 = torch.cuda.Event(enable_timing=True)
        a1 = torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for k in range(n):
            step_shuffle(first + 3 + k)
        a1.record(stream)
        fence()
        return a0.elapsed_time(a1) / n

    alone_ms = None
    if args.mode == "stream":
        n_alone = max(1, min(args.steps, 300))
        alone_ms = [shuffle_alone(B.WASH_MODE_STREAM, n_alone), shuffle_alone(B.WASH_MODE_SPARSE, n_alone)]
        B.wash_set_mode(pop.ctx, B.WASH_MODE_STREAM)

    # ---- end to end through the host-buffer entry point --------------------------------
    e2e_steps = max(1, min(args.steps, 5))
    ops = B.WASH_OP_SHUFFLE | B.WASH_OP_EMA | B.WASH_OP_AVERAGE
    B.wash_step_host(pop.ctx, ops, params_pin, opt_pin, avg_pin, 0, wl.p, p_layer, SEED, ALPHA, stream)   # warm
    fence()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for k in range(e2e_steps):
        B.wash_step_host(pop.ctx, ops, params_pin, opt_pin, avg_pin, 1 + k, wl.p, p_layer, SEED, ALPHA, stream)
    e1.record(stream)
    fence()
    e2e_ms = e0.elapsed_time(e1)
    stack_bytes = params_pin.numel() * params_pin.element_size() + (opt_pin.numel() * opt_pin.element_size() if opt_pin is not None else 0)
    h2d = stack_bytes
    d2h = stack_bytes + avg_pin.numel() * avg_pin.element_size() + 16

    # ---- max over ranks ------------------------------------------------------------------
    if dist is not None:
        t = torch.tensor([total_ms, e2e_ms, mean_ms[0], mean_ms[1], mean_ms[2]] + (alone_ms or [0.0, 0.0]), dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, e2e_ms = float(t[0]), float(t[1])
        mean_ms = t[2:5].cpu().numpy()
        if alone_ms is not None:
            alone_ms = [float(t[5]), float(t[6])]
        c = torch.tensor([selected_total, moved_total], dtype=torch.int64, device="cuda")
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
        selected_total, moved_total = int(c[0]), int(c[1])

    if rank == 0:
        sel_per_step_rank = selected_total / args.steps / world
        ab = wl.algorithmic_bytes(sel_per_step_rank)
        step_ms = total_ms / args.steps
        value = ab["step"] * world / (step_ms * 1e-3) / 1e9
        peak, peak_src = measured_peak()
        shuffle_gbs = ab["shuffle"] / (mean_ms[0] * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16+f32" if wl.bf16 else "f32", "data": "synthetic",
            "value_definition": "bytes the three kernels of one step must stream (shuffle: read both stacks + write selected; "
                                "EMA: read+write parameters; average: read parameters + write one row) / step time, all ranks",
            "config": {"workload": wl.name, "N": wl.N, "tensors": wl.T, "P": wl.P, "p": wl.p,
                       "per_layer_p": wl.p_layer is not None, "opt_state": wl.opt, "layout": "[N][P]", "mode": args.mode,
                       "footprint_bytes_per_gpu": stack_bytes, "l2": "inputs larger than L2 (no flush)" if stack_bytes > 2.5e8 else "L2-resident: footprint below 2x L2",
                       "sharding": "one population shard per rank, no collective"},
            "param_swaps_per_s": selected_total * wl.N / (total_ms * 1e-3),
            "moved_values_per_s": moved_total / (total_ms * 1e-3),
            "selected_coords_per_step": selected_total / args.steps,
            "kernel_times": "CUDA events on the launching stream, " + ("inside the timed region" if args.inline_kernel_events
                                                                      else "instrumented pass of %d steps right after the timed region" % min(args.steps, 300)),
            "kernels": {
                "shuffle": {"ms": float(mean_ms[0]), "GBps": shuffle_gbs, "frac_of_hbm": shuffle_gbs / peak},
                "papa_ema": {"ms": float(mean_ms[1]), "GBps": ab["ema"] / (mean_ms[1] * 1e-3) / 1e9},
                "population_average": {"ms": float(mean_ms[2]), "GBps": ab["average"] / (mean_ms[2] * 1e-3) / 1e9},
            },
            "roofline": {"kernel": "shuffle kernel, mode %s (params + momentum)" % args.mode, "bound": "hbm", "achieved": shuffle_gbs,
                         "peak": peak, "peak_source": peak_src, "unit": "GB/s", "frac": shuffle_gbs / peak,
                         "traffic": TRAFFIC.get(wl.name, {}).get("dram_bytes") if args.mode == "stream" else None,
                         "traffic_source": TRAFFIC.get(wl.name, {}).get("source") if args.mode == "stream" else None},
            "e2e": {"value": ab["step"] * world / (e2e_ms / e2e_steps * 1e-3) / 1e9, "unit": "GB/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps,
                    "api": "wash_step_host (pinned host stacks)"},
            "gpu_launches": int(launches),
            "clocks": clocks,
        }
        if alone_ms is not None:
            sel_step = selected_total / args.steps
            line["shuffle_back_to_back"] = {
                "launches": max(1, min(args.steps, 300)),
                "stream": {"ms": alone_ms[0], "GBps": ab["shuffle"] / (alone_ms[0] * 1e-3) / 1e9,
                           "frac_of_hbm": ab["shuffle"] / (alone_ms[0] * 1e-3) / 1e9 / peak,
                           "param_swaps_per_s": sel_step * wl.N / (alone_ms[0] * 1e-3)},
                "sparse": {"ms": alone_ms[1], "param_swaps_per_s": sel_step * wl.N / (alone_ms[1] * 1e-3),
                           "bound": "integer pipes (one Philox block per 4 coordinates), not HBM"},
                "note": "the step's shuffle launched alone, two events around the whole series; WASH_MODE_AUTO picks the sparse kernel below 3 % expected selection",
            }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(wl)
        print(json.dumps(line), flush=True)
    pop.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# DRAM bytes per shuffle launch from the ncu capture summarised under profiles/ (None
# until a capture of the current kernel exists).
TRAFFIC = {
    # shuffle_async_kernel<F32, F32, [N][P], 1>: 448.9 MB read + 5.9 MB written per launch
    "cfg2_resnet18_n5": {"dram_bytes": 448.9e6 + 5.9e6,
                         "source": "profiles/shuffle_async_kernel_cfg2_resnet18_n5.md"},
}


def cpu_baseline(wl: Workload) -> dict:
    """The oracle as it stands on the host cores, on a bounded number of full steps."""
    import oracle
    offsets, padded_P = W.padded_offsets(wl.numel)
    params, opt = wl.host_stacks(offsets, padded_P)
    pop = oracle.Population(wl.N, wl.numel, offsets, padded_P, oracle.LAYOUT_NP, wl.tensor_id)
    out = np.zeros(padded_P, dtype=params.dtype)
    threads = oracle.max_threads()
    oracle.set_threads(threads)
    p = wl.p if wl.schedule is None else oracle.layer_probs(wl.T, wl.p, oracle.SCHEDULE_DECREASING)
    steps, sel, t0 = 0, 0, time.perf_counter()
    while True:
        sel += oracle.shuffle(pop, params, p, seed=SEED, step=steps, stack2=opt)[0]
        oracle.papa_ema(pop, params, ALPHA)
        oracle.population_average(pop, params, out)
        steps += 1
        dt = time.perf_counter() - t0
        if dt > 10.0 or steps >= 2000:
            break
    gbs = wl.algorithmic_bytes(sel / steps)["step"] * steps / dt / 1e9
    return {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": "%d full steps of the same workload (%.1f s)" % (steps, dt), "ms_per_step": dt / steps * 1e3}


def run_sweep(args) -> None:
    """Config 5: flat fp32 populations, N x P x p x layout, shuffle only.  One JSON line
    per cell (not the default bench line)."""
    import torch
    from paper_2405_17517_b200 import binding as B

    torch.cuda.set_device(0)
    B.load()
    peak, _ = measured_peak()
    modes = {"stream": B.WASH_MODE_STREAM, "sparse": B.WASH_MODE_SPARSE, "registers": B.WASH_MODE_STREAM_REGISTERS,
             "staged": B.WASH_MODE_STREAM_STAGED}
    stream = torch.cuda.current_stream()
    # integer-pipe ceiling of the mask: Philox blocks per second with no memory traffic
    chk = torch.zeros(1, dtype=torch.int32, device="cuda")
    n_blocks = 1 << 28
    for _ in range(3):
        B.wash_philox_probe(n_blocks, SEED, chk, 0, stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(5):
        B.wash_philox_probe(n_blocks, SEED, chk, 0, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    rate = 5 * n_blocks / (e0.elapsed_time(e1) * 1e-3)
    print(json.dumps({"philox_blocks_per_s": rate, "mask_coordinates_per_s": 4 * rate,
                      "note": "ceiling of the mask draw alone; N*16 bytes of fp32 stack per block"}), flush=True)
    pick = lambda text, default, conv: [conv(x) for x in text.split(",")] if text else default
    for N in pick(args.sweep_N, [2, 4, 8, 16, 32], int):
        for logP in pick(args.sweep_logP, [20, 24, 27], int):
            P = 1 << logP
            for layout, lname in ((B.WASH_LAYOUT_NP, "[N][P]"), (B.WASH_LAYOUT_PN, "[P][N]")):
                if args.sweep_layout and args.sweep_layout != ("np" if layout == B.WASH_LAYOUT_NP else "pn"):
                    continue
                pop = B.Population(N, [P], layout, 0)
                gen = torch.Generator(device="cuda").manual_seed(N * 100 + logP)
                stack = torch.randn(N * pop.padded_P, generator=gen, device="cuda", dtype=torch.float32) * 0.05
                pop.bind(B.WASH_STACK_PARAMS, stack)
                if args.threads or args.blocks_per_sm:
                    B.wash_set_launch(pop.ctx, args.threads, args.blocks_per_sm)
                stats = torch.zeros(2, dtype=torch.int64, device="cuda")
                for p in pick(args.sweep_p, [1e-4, 1e-3, 1e-2, 1e-1, 1.0], float):
                    for mode in args.sweep_modes.split(","):
                        B.wash_set_mode(pop.ctx, modes[mode])
                        for w in range(3):
                            B.wash_shuffle(pop.ctx, w, p, None, SEED, stream, stats)
                        torch.cuda.synchronize()
                        stats.zero_()
                        reps = 20 if N * P * 4 < (4 << 30) else 8
                        ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
                        ev[0].record(stream)
                        for k in range(reps):
                            B.wash_shuffle(pop.ctx, 3 + k, p, None, SEED, stream, stats)
                            ev[k + 1].record(stream)
                        torch.cuda.synchronize()
                        ms = float(np.median([ev[k].elapsed_time(ev[k + 1]) for k in range(reps)]))
                        sel = int(stats[0]) / reps
                        footprint = N * P * 4
                        streamed = footprint + sel * N * 4
                        line = {"N": N, "P": P, "p": p, "layout": lname, "mode": mode, "ms": ms,
                                "selected_per_launch": sel, "param_swaps_per_s": sel * N / (ms * 1e-3),
                                "algorithmic_GBps": 2 * 4 * N * sel / (ms * 1e-3) / 1e9}
                        if mode != "sparse":
                            line["streamed_GBps"] = streamed / (ms * 1e-3) / 1e9
                            line["frac_of_hbm"] = line["streamed_GBps"] / peak
                        line["l2"] = "L2-influenced" if footprint < (256 << 20) else "beyond L2"
                        print(json.dumps(line), flush=True)
                B.wash_check(pop.ctx)
                pop.close()
                del stack
                torch.cuda.empty_cache()


def run_exchange(args) -> None:
    """One worker of the one-model-per-device form, timed alone on this GPU: plan (mask,
    permutations, slot offsets), send (stores into the peers' staging buffers, here plain
    buffers on the same device) and receive, per workload.  One JSON line each (not the
    driver's bench line)."""
    import torch
    from paper_2405_17517_b200 import binding as B

    torch.cuda.set_device(0)
    B.load()
    stream = torch.cuda.current_stream()
    names = [args.workload] if args.workload_given else ["cfg2_resnet18_n5", "cfg3_resnet50_n10", "cfg4_resnet50_bf16_n8"]
    for name in names:
        wl = Workload(name)
        ctx = B.wash_create_segments(wl.N, wl.numel, None, None, 0, 0)
        P = B.wash_stack_elems(ctx, wl.T)[0]
        p_layer = B.wash_layer_probs(wl.T, wl.p, 0) if wl.schedule == "decreasing" else None
        gen = torch.Generator(device="cuda").manual_seed(SEED)
        row = (torch.randn(P, generator=gen, device="cuda") * 0.05).to(torch.bfloat16 if wl.bf16 else torch.float32)
        rows = [row]
        B.wash_exchange_bind(ctx, 0, 0, B.WASH_BF16 if wl.bf16 else B.WASH_F32, row, P)
        if wl.opt:
            rows.append(torch.randn(P, generator=gen, device="cuda") * 1e-3)
            B.wash_exchange_bind(ctx, 0, 1, B.WASH_F32, rows[1], P)
        cap = max(1 << 16, int(4 * wl.p * wl.P))
        keep = []
        for k, r in enumerate(rows):
            for parity in (0, 1):
                bufs = [torch.zeros(cap, dtype=r.dtype, device="cuda") for _ in range(wl.N)]
                keep.append(bufs)
                B.wash_exchange_staging(ctx, k, parity, bufs, cap)
        stats = torch.zeros(2, dtype=torch.int64, device="cuda")
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")   # larger than L2
        reps = 30
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(reps)]
        for i in range(3 + reps):
            if not args.exchange_warm:
                flush.zero_()
            e = ev[max(i - 3, 0)]
            e[0].record(stream)
            B.wash_exchange_plan(ctx, i, wl.p, p_layer, SEED, stream)
            e[1].record(stream)
            B.wash_exchange_send(ctx, stream)
            e[2].record(stream)
            B.wash_exchange_receive(ctx, stream, stats if i >= 3 else None)
            e[3].record(stream)
        torch.cuda.synchronize()
        B.wash_check(ctx)
        med = lambda a, b: float(np.median([e[a].elapsed_time(e[b]) for e in ev])) * 1e3
        sel, recv = int(stats[0]) / reps, int(stats[1]) / reps
        elem = (wl.E + wl.E_opt)
        print(json.dumps({
            "workload": name, "worker": 0, "N": wl.N, "coordinates": wl.P,
            "plan_us": med(0, 1), "send_us": med(1, 2), "receive_us": med(2, 3), "step_us": med(0, 3),
            "selected_per_step": sel, "values_received_per_step": recv,
            "link_bytes_in_per_step": recv * elem, "model_bytes": wl.P * elem,
            "mask_coordinates_per_s": wl.P / (med(0, 1) * 1e-6),
            "note": ("steps back to back (row and tables may stay in L2)" if args.exchange_warm else "L2 flushed before every step")
                    + "; peers' buffers are on the same device",
        }), flush=True)
        B.wash_destroy(ctx)
        del keep, rows, row, flush
        torch.cuda.empty_cache()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2_resnet18_n5", choices=sorted(W.CONFIGS))
    ap.add_argument("--mode", default="stream", choices=["stream", "sparse", "staged", "registers"])
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--blocks-per-sm", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--inline-kernel-events", action="store_true",
                    help="record the per-kernel events inside the timed region instead of in a second pass")
    ap.add_argument("--sweep", action="store_true", help="config-5 sweep of the shuffle kernel (many JSON lines)")
    ap.add_argument("--sweep-modes", default="stream,sparse")
    ap.add_argument("--sweep-N", default="", help="comma list; default 2,4,8,16,32")
    ap.add_argument("--sweep-logP", default="", help="comma list; default 20,24,27")
    ap.add_argument("--sweep-p", default="", help="comma list; default 1e-4..1")
    ap.add_argument("--sweep-layout", default="", choices=["", "np", "pn"])
    ap.add_argument("--exchange-warm", action="store_true", help="with --exchange: no L2 flush between steps")
    ap.add_argument("--exchange", action="store_true", help="time one worker of the one-model-per-device form (JSON line per workload)")
    args = ap.parse_args()
    args.workload_given = any(a == "--workload" or a.startswith("--workload=") for a in sys.argv[1:])
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.sweep:
        run_sweep(args)
        return
    if args.exchange:
        run_exchange(args)
        return
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
