#!/usr/bin/env python
"""Benchmark of the WASH hot path on B200: one JSON line on stdout.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload cfg3_resnet50_n10|cfg2_resnet18_n5|cfg4_resnet50_bf16_n8|cfg1_flat_n3]

A step is one pass of the whole hot path over one synthetic population: the shuffle of
the parameter and momentum stacks (WASH+Opt, one launch), PAPA's EMA on the parameters
and the final average -- three kernel launches.  `value` is the shuffle's own
throughput: the bytes the shuffle must move (see algorithmic_bytes) divided by the time
of the shuffle kernel inside the step, in GB/s, with the stacks resident in HBM;
`ms_per_step` and the `step` record cover the three kernels; `e2e` is the shuffle
through wash_step_host with the stacks in pinned host memory (copies inside the timed
region).  The timed block of --steps steps is repeated until at least half a second of
GPU time has been measured; medians over the blocks are reported.  `configs` holds the
other configurations and cells of the config-5 sweep, timed in the same run with both
ceilings (HBM copy bandwidth and the integer pipes' Philox rate).  For N > 1 (torchrun)
every rank holds its own shard of an N-times deeper population (tensor indices offset
by rank), no communication: weak scaling.

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
        self.Es = (self.E, 4) if self.opt else (self.E,)
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

    def one_step(pop, a, b, out, step, p_layer, clock=None):
        p = wl.p if p_layer is None else p_layer
        t0 = time.perf_counter()
        st = oracle.shuffle(pop, a, p, seed=SEED, step=step, stack2=b)
        if clock is not None:
            clock[0] += time.perf_counter() - t0
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
    clock = [0.0]
    t0 = time.perf_counter()
    for k in range(args.steps):
        sel += one_step(sub, sp, so, sout, args.warmup + k, sub_pl, clock)[0]
    dt = time.perf_counter() - t0
    scale = sub_P / wl.P
    ab = wl.algorithmic_bytes(sel / max(args.steps, 1) / scale)
    gbs = ab["shuffle"] * scale * args.steps / clock[0] / 1e9           # the headline metric: the shuffle's own throughput
    sample = "first %d of %d tensors (%d of %d coordinates per model) per step" % (n_t, wl.T, sub_P, wl.P)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16+f32" if wl.bf16 else "f32", "data": "synthetic",
        "value_definition": "the oracle's shuffle: bytes the shuffle of both stacks must move / the time spent in the oracle's shuffle; "
                            "ms_per_step is the whole step (shuffle + EMA + average) on the sample",
        "config": {"workload": wl.name, "N": wl.N, "tensors": wl.T, "P": wl.P, "p": wl.p, "sample": sample},
        "param_swaps_per_s": sel * wl.N / clock[0],
        "step": {"ms": dt / max(args.steps, 1) * 1e3, "GBps": ab["step"] * scale * args.steps / dt / 1e9},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------
MIN_TIMED_S = 0.5          # the timed blocks are repeated until this much GPU time has been measured
MAX_REPEATS = 400


def philox_blocks(P: int, N: int, selected: float) -> float:
    """Philox4x32-10 blocks one shuffle launch must draw: one per 4 coordinates for the mask and
    ceil((N-1)/4) per selected coordinate for its permutation."""
    return P / 4.0 + selected * ((N - 1 + 3) // 4)


def sector_write_share(p_eff: float, N: int, E: int, layout: str) -> float:
    """Share of a stack's 32-byte DRAM sectors that hold at least one moved value when every
    coordinate is selected with probability p_eff (all N values of a selected coordinate are
    counted as moved).  [N][P]: a sector holds 32/E neighbouring coordinates of one model;
    [P][N]: a coordinate's N values lie side by side, a sector holds 32/(E N) coordinates (at
    least part of one)."""
    per_sector = 32.0 / E if layout == "[N][P]" else max(1.0, 32.0 / (E * N))
    return 1.0 - (1.0 - p_eff) ** per_sector


def measure_philox_rate(B, torch, stream) -> float:
    """Philox blocks per second of a kernel that draws mask blocks and nothing else: the ceiling
    the integer pipes put on any shuffle, measured in this run."""
    chk = torch.zeros(1, dtype=torch.int32, device="cuda")
    n_blocks = 1 << 28
    for _ in range(3):
        B.wash_philox_probe(n_blocks, SEED, chk, torch.cuda.current_device(), stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(5):
        B.wash_philox_probe(n_blocks, SEED, chk, torch.cuda.current_device(), stream)
    e1.record(stream)
    torch.cuda.synchronize()
    return 5 * n_blocks / (e0.elapsed_time(e1) * 1e-3)


B2B_MIN_S = 0.06           # GPU time of a back-to-back series (set to 0 together with --min-timed-s 0)


def time_launches(torch, stream, launch, first_step: int, min_s: float = None, blocks: int = 3, max_n: int = 2000):
    """Median and minimum per-launch time (ms) of `launch(step)` issued back to back, two events
    around each block of launches; the block length is chosen so that a block lasts min_s / blocks."""
    if min_s is None:
        min_s = B2B_MIN_S
    for k in range(3):
        launch(first_step + k)
    torch.cuda.synchronize()
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record(stream)
    launch(first_step + 3)
    a1.record(stream)
    torch.cuda.synchronize()
    est = max(a0.elapsed_time(a1) * 1e-3, 1e-6)
    n = int(max(2, min(max_n, min_s / blocks / est)))
    per = []
    step = first_step + 4
    for _ in range(blocks):
        a0.record(stream)
        for k in range(n):
            launch(step + k)
        a1.record(stream)
        torch.cuda.synchronize()
        per.append(a0.elapsed_time(a1) / n)
        step += n
    return float(np.median(per)), float(min(per)), n * blocks


def shuffle_cell(B, torch, stream, pop, shuffle_fn, N, P, Es, p_eff, layout, peak, philox_rate, modes=("stream", "sparse"),
                 consensus_fn=None):
    """Times one population's shuffle in the given modes and relates it to both ceilings:
    t_HBM = bytes / measured copy bandwidth, t_ALU = Philox blocks / measured probe rate."""
    stats = torch.zeros(2, dtype=torch.int64, device="cuda")
    out = {}
    E_sum = sum(Es)             # Es: element size of every stack the launch shuffles
    for mode in modes:
        B.wash_set_mode(pop.ctx, {"stream": B.WASH_MODE_STREAM, "sparse": B.WASH_MODE_SPARSE}[mode])
        stats.zero_()
        med, lo, n = time_launches(torch, stream, lambda i: shuffle_fn(i, stats), 100)
        torch.cuda.synchronize()
        sel = int(stats[0]) / (n + 4)          # time_launches issues 4 launches before its blocks
        blocks = philox_blocks(P, N, sel)
        t_alu = blocks / philox_rate
        rec = {"ms": med, "ms_min": lo, "launches": n, "selected_per_launch": sel,
               "param_swaps_per_s": sel * N / (med * 1e-3), "philox_blocks_per_launch": blocks,
               "alu_frac": t_alu / (med * 1e-3)}
        if mode == "stream":
            algorithmic = N * P * E_sum + sel * N * E_sum                         # read everything, write the selected values
            dram_model = sum(N * P * E * (1.0 + sector_write_share(p_eff, N, E, layout)) for E in Es)
            t_hbm = algorithmic / (peak * 1e9)
            t_hbm_sectors = dram_model / (peak * 1e9)
            rec.update({"GBps": algorithmic / (med * 1e-3) / 1e9, "frac_of_hbm": t_hbm / (med * 1e-3),
                        "dram_model_GBps": dram_model / (med * 1e-3) / 1e9, "hbm_frac_sector_model": t_hbm_sectors / (med * 1e-3),
                        "bound": "alu" if t_alu > t_hbm_sectors else "hbm",
                        "frac_of_bound": max(t_alu, t_hbm_sectors) / (med * 1e-3)})
        else:
            rec.update({"algorithmic_GBps": 2.0 * sel * N * E_sum / (med * 1e-3) / 1e9, "bound": "alu"})
        out[mode] = rec
    B.wash_set_mode(pop.ctx, B.WASH_MODE_STREAM)
    if consensus_fn is not None:
        # the streaming shuffle with the distance to the consensus (per quarter of the tensor
        # table) gathered in the same pass
        med, lo, n = time_launches(torch, stream, lambda i: consensus_fn(i, stats), 100)
        out["stream_with_consensus"] = {"ms": med, "ms_min": lo, "launches": n, "ratio_to_stream": med / out["stream"]["ms"]}
    return out


def configs_record(B, torch, stream, peak, philox_rate, main_name, main_cell) -> dict:
    """The other configurations, timed in the same run: configs 1-4 (device-generated values of
    the configs' shapes: the shuffle's time does not depend on the values) and the cells
    N in {2, 8, 32} x P = 2^27 x p in {1e-3, 1e-2, 1e-1} x both layouts of config 5."""
    rec = {"note": "shuffle only, launched back to back (median of 3 blocks); frac_of_hbm = algorithmic bytes (read all + write "
                   "selected values) / time / measured copy bandwidth; hbm_frac_sector_model counts writes in whole 32-byte sectors; "
                   "alu_frac = Philox blocks per second / the probe's rate; bound = the larger of the two times",
           "philox_probe_blocks_per_s": philox_rate}
    for name in ("cfg1_flat_n3", "cfg2_resnet18_n5", "cfg3_resnet50_n10", "cfg4_resnet50_bf16_n8"):
        if name == main_name:
            rec[name] = main_cell
            continue
        wl = Workload(name)
        pop = B.Population(wl.N, wl.numel, B.WASH_LAYOUT_NP, torch.cuda.current_device(), wl.tensor_id)
        gen = torch.Generator(device="cuda").manual_seed(SEED)
        params = (torch.randn(wl.N * pop.padded_P, generator=gen, device="cuda") * 0.05).to(torch.bfloat16 if wl.bf16 else torch.float32)
        pop.bind(B.WASH_STACK_PARAMS, params)
        opt = None
        if wl.opt:
            opt = torch.randn(wl.N * pop.padded_P, generator=gen, device="cuda") * 1e-3
            pop.bind(B.WASH_STACK_OPT, opt)
        p_layer = B.wash_layer_probs(wl.T, wl.p, B.WASH_SCHEDULE_DECREASING) if wl.schedule == "decreasing" else None
        fn = (lambda i, st: B.wash_shuffle_both(pop.ctx, i, wl.p, p_layer, SEED, stream, st)) if wl.opt else \
             (lambda i, st: B.wash_shuffle(pop.ctx, i, wl.p, p_layer, SEED, stream, st))
        p_eff = wl.p if p_layer is None else float((p_layer * wl.numel).sum() / wl.P)
        sq = torch.zeros(4 * wl.N, dtype=torch.float64, device="cuda")
        quarters = [0, wl.T // 4, wl.T // 2, 3 * wl.T // 4, wl.T] if wl.T >= 4 else [0, wl.T]
        cfn = lambda i, st: B.wash_shuffle_consensus(pop.ctx, B.WASH_STACK_BOTH if wl.opt else B.WASH_STACK_PARAMS, i, wl.p, p_layer, SEED, stream, st, quarters, sq)
        cell = shuffle_cell(B, torch, stream, pop, fn, wl.N, wl.P, wl.Es, p_eff, "[N][P]", peak, philox_rate, consensus_fn=cfn)
        cell["footprint_bytes"] = wl.N * pop.padded_P * (wl.E + wl.E_opt)
        cell["l2"] = "beyond L2" if cell["footprint_bytes"] > 2.5e8 else "L2-resident"
        rec[name] = cell
        B.wash_check(pop.ctx)
        pop.close()
        del params, opt
        torch.cuda.empty_cache()
    cells = []
    P = 1 << 27
    for N in (2, 8, 32):
        for layout, lname in ((B.WASH_LAYOUT_NP, "[N][P]"), (B.WASH_LAYOUT_PN, "[P][N]")):
            pop = B.Population(N, [P], layout, torch.cuda.current_device())
            gen = torch.Generator(device="cuda").manual_seed(N)
            stack = torch.empty(N * pop.padded_P, device="cuda", dtype=torch.float32)
            for lo in range(0, stack.numel(), 1 << 28):
                stack[lo:lo + (1 << 28)].normal_(0.0, 0.05, generator=gen)
            pop.bind(B.WASH_STACK_PARAMS, stack)
            for p in (1e-3, 1e-2, 1e-1):
                fn = lambda i, st, p=p: B.wash_shuffle(pop.ctx, i, p, None, SEED, stream, st)
                cell = shuffle_cell(B, torch, stream, pop, fn, N, P, (4,), p, lname, peak, philox_rate)
                cell.update({"N": N, "P": P, "p": p, "layout": lname})
                cells.append(cell)
            B.wash_check(pop.ctx)
            pop.close()
            del stack
            torch.cuda.empty_cache()
    rec["cfg5_cells"] = cells
    return rec


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
    del params_h, opt_h
    params_d = params_pin.cuda(non_blocking=True)
    opt_d = opt_pin.cuda(non_blocking=True) if opt_pin is not None else None
    avg_d = torch.zeros(pop.padded_P, dtype=params_d.dtype, device="cuda")
    avg_pin = torch.zeros(pop.padded_P, dtype=params_d.dtype).pin_memory()
    stats_d = torch.zeros(2, dtype=torch.int64, device="cuda")
    pop.bind(B.WASH_STACK_PARAMS, params_d)
    if opt_d is not None:
        pop.bind(B.WASH_STACK_OPT, opt_d)
    mode_code = {"stream": B.WASH_MODE_STREAM, "sparse": B.WASH_MODE_SPARSE, "auto": B.WASH_MODE_AUTO}[args.mode]
    B.wash_set_mode(pop.ctx, mode_code)
    if args.threads or args.blocks_per_sm:
        B.wash_set_launch(pop.ctx, args.threads, args.blocks_per_sm)
    pdt = B.WASH_BF16 if wl.bf16 else B.WASH_F32
    if wl.schedule == "decreasing":
        wl.p_layer = B.wash_layer_probs(wl.T, wl.p, B.WASH_SCHEDULE_DECREASING)
    p_layer = wl.p_layer
    p_eff = wl.p if p_layer is None else float((p_layer * wl.numel).sum() / wl.P)
    stream = torch.cuda.current_stream()

    def step_shuffle(i, st=stats_d):
        if opt_d is not None:
            B.wash_shuffle_both(pop.ctx, i, wl.p, p_layer, SEED, stream, st)
        else:
            B.wash_shuffle(pop.ctx, i, wl.p, p_layer, SEED, stream, st)

    def step(i, ev):
        """One pass of the hot path: shuffle of both stacks, PAPA's EMA, the average; an event
        before and after each kernel, on the launching stream."""
        ev[0].record(stream)
        step_shuffle(i)
        ev[1].record(stream)
        B.papa_ema(pop.ctx, B.WASH_STACK_PARAMS, ALPHA, stream)
        ev[2].record(stream)
        B.population_average(pop.ctx, B.WASH_STACK_PARAMS, avg_d, pdt, stream)
        ev[3].record(stream)

    def fence():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    K = args.steps
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(K)]
    for w in range(args.warmup):
        step(w, events[0])
    fence()
    stats_d.zero_()
    launches0 = B.wash_launch_count()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()

    # ---- timed blocks of exactly K steps each, repeated until MIN_TIMED_S of GPU time --------
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    block_ms, kernel_ms = [], []          # per block: total time (max over ranks), mean time of each kernel
    next_step = args.warmup
    repeats_wanted = 1
    while len(block_ms) < repeats_wanted:
        fence()
        t_begin.record(stream)
        for k in range(K):
            step(next_step + k, events[k])
        t_end.record(stream)
        fence()
        next_step += K
        total = t_begin.elapsed_time(t_end)
        per_kernel = np.array([[e[i].elapsed_time(e[i + 1]) for i in range(3)] for e in events]).mean(axis=0)
        if dist is not None:
            t = torch.tensor([total] + per_kernel.tolist(), dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            total, per_kernel = float(t[0]), t[1:].cpu().numpy()
        block_ms.append(total)
        kernel_ms.append(per_kernel)
        if len(block_ms) == 1:       # the same count on every rank: derived from the all-reduced first block
            repeats_wanted = int(min(MAX_REPEATS, max(1, np.ceil(args.min_timed_s * 1e3 / max(total, 1e-3)))))
    clocks = sampler.stop()
    launches = B.wash_launch_count() - launches0
    B.wash_check(pop.ctx)
    repeats = len(block_ms)
    st = stats_d.cpu().numpy().view(np.uint64)
    selected_total, moved_total = int(st[0]), int(st[1])
    steps_timed = K * repeats
    block_ms = np.array(block_ms)
    kernel_ms = np.array(kernel_ms)
    med_ms = np.median(kernel_ms, axis=0)          # shuffle, ema, average
    min_ms = kernel_ms.min(axis=0)
    step_ms = float(np.median(block_ms)) / K
    step_ms_min = float(block_ms.min()) / K

    # ---- the shuffle alone, launched back to back, in the streaming and the sparse mode, with
    # both ceilings (world == 1; with several ranks only the streaming time is taken)
    peak, peak_src = measured_peak()
    philox_rate = measure_philox_rate(B, torch, stream)
    fence()
    sq_d = torch.zeros(4 * wl.N, dtype=torch.float64, device="cuda")
    quarters = [0, wl.T // 4, wl.T // 2, 3 * wl.T // 4, wl.T] if wl.T >= 4 else [0, wl.T]
    main_cell = shuffle_cell(B, torch, stream, pop, lambda i, st_: step_shuffle(i, st_), wl.N, wl.P, wl.Es, p_eff,
                             "[N][P]", peak, philox_rate,
                             consensus_fn=lambda i, st_: B.wash_shuffle_consensus(pop.ctx, B.WASH_STACK_BOTH if wl.opt else B.WASH_STACK_PARAMS, i, wl.p,
                                                                                  p_layer, SEED, stream, st_, quarters, sq_d))
    B.wash_set_mode(pop.ctx, mode_code)
    fence()

    # ---- end to end through the host-buffer entry point --------------------------------
    # The headline metric (the shuffle) through wash_step_host with the stacks in pinned host
    # memory: copy in, shuffle, copy out, every step, inside the timed region; then the same
    # with the whole step (shuffle + EMA + average).
    e2e_steps = max(1, min(K, 5))

    def host_steps(ops, first):
        B.wash_step_host(pop.ctx, ops, params_pin, opt_pin, avg_pin, first, wl.p, p_layer, SEED, ALPHA, stream)   # warm
        fence()
        e0 = torch.cuda.Event(enable_timing=True)
        e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        sel = 0
        for k in range(e2e_steps):
            sel += B.wash_step_host(pop.ctx, ops, params_pin, opt_pin, avg_pin, first + 1 + k, wl.p, p_layer, SEED, ALPHA, stream)[0]
        e1.record(stream)
        fence()
        return e0.elapsed_time(e1), sel

    e2e_ms, sel_e2e = host_steps(B.WASH_OP_SHUFFLE, 0)
    e2e_full_ms, _ = host_steps(B.WASH_OP_SHUFFLE | B.WASH_OP_EMA | B.WASH_OP_AVERAGE, 100)
    stack_bytes = params_pin.numel() * params_pin.element_size() + (opt_pin.numel() * opt_pin.element_size() if opt_pin is not None else 0)
    h2d = stack_bytes
    d2h = stack_bytes + 16
    d2h_full = stack_bytes + avg_pin.numel() * avg_pin.element_size() + 16

    # ---- max / sum over ranks ----------------------------------------------------------------
    if dist is not None:
        t = torch.tensor([e2e_ms, e2e_full_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms, e2e_full_ms = float(t[0]), float(t[1])
        c = torch.tensor([selected_total, moved_total, sel_e2e], dtype=torch.int64, device="cuda")
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
        selected_total, moved_total, sel_e2e = int(c[0]), int(c[1]), int(c[2])

    if rank == 0:
        sel_per_step_rank = selected_total / steps_timed / world
        ab = wl.algorithmic_bytes(sel_per_step_rank)
        shuffle_gbs = ab["shuffle"] / (med_ms[0] * 1e-3) / 1e9          # one rank's kernel
        blocks_launch = philox_blocks(wl.P, wl.N, sel_per_step_rank)
        traffic = TRAFFIC.get((wl.name, args.mode), {})
        line = {
            "metric": METRIC, "value": shuffle_gbs * world, "unit": "GB/s", "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16+f32" if wl.bf16 else "f32", "data": "synthetic",
            "value_definition": "the shuffle's own throughput: bytes the shuffle of both stacks must move (read every value, write the "
                                "selected ones) / the shuffle kernel's time inside the step (CUDA events on the launching stream, median "
                                "over the timed blocks of the per-block mean, max over ranks), summed over ranks; ms_per_step is the whole "
                                "step (shuffle + EMA + average)",
            "repeats": repeats, "steps_timed": steps_timed, "timed_gpu_s": float(block_ms.sum()) * 1e-3,
            "ms_per_step_min": step_ms_min,
            "config": {"workload": wl.name, "N": wl.N, "tensors": wl.T, "P": wl.P, "p": wl.p,
                       "per_layer_p": wl.p_layer is not None, "opt_state": wl.opt, "layout": "[N][P]", "mode": args.mode,
                       "footprint_bytes_per_gpu": stack_bytes, "l2": "inputs larger than L2 (no flush)" if stack_bytes > 2.5e8 else "L2-resident: footprint below 2x L2",
                       "sharding": "one population shard per rank, no collective"},
            "param_swaps_per_s": sel_per_step_rank * wl.N * world / (med_ms[0] * 1e-3),
            "moved_values_per_s": moved_total / steps_timed / (med_ms[0] * 1e-3),
            "selected_coords_per_step": selected_total / steps_timed,
            "step": {"kernels": "wash_shuffle_both + papa_ema + population_average" if wl.opt else "wash_shuffle + papa_ema + population_average",
                     "ms": step_ms, "ms_min": step_ms_min, "GBps": ab["step"] * world / (step_ms * 1e-3) / 1e9,
                     "bytes": "shuffle: read both stacks + write selected; EMA: read + write parameters; average: read parameters + write one row"},
            "kernel_times": "CUDA events on the launching stream around every kernel, inside the timed blocks; median (and min) over %d blocks of the mean over the block's %d steps" % (repeats, K),
            "kernels": {
                "shuffle": {"ms": float(med_ms[0]), "ms_min": float(min_ms[0]), "GBps": shuffle_gbs, "frac_of_hbm": shuffle_gbs / peak},
                "papa_ema": {"ms": float(med_ms[1]), "ms_min": float(min_ms[1]), "GBps": ab["ema"] / (med_ms[1] * 1e-3) / 1e9,
                             "frac_of_hbm": ab["ema"] / (med_ms[1] * 1e-3) / 1e9 / peak},
                "population_average": {"ms": float(med_ms[2]), "ms_min": float(min_ms[2]), "GBps": ab["average"] / (med_ms[2] * 1e-3) / 1e9,
                                       "frac_of_hbm": ab["average"] / (med_ms[2] * 1e-3) / 1e9 / peak},
            },
            "roofline": {"kernel": "shuffle kernel, mode %s (params + momentum)" % args.mode, "bound": "hbm", "achieved": shuffle_gbs,
                         "peak": peak, "peak_source": peak_src, "unit": "GB/s", "frac": shuffle_gbs / peak,
                         "alu_frac": blocks_launch / philox_rate / (med_ms[0] * 1e-3),
                         "alu_peak_philox_blocks_per_s": philox_rate,
                         "traffic": traffic.get("dram_bytes"), "traffic_source": traffic.get("source")},
            "e2e": {"value": wl.algorithmic_bytes(sel_e2e / e2e_steps / world)["shuffle"] * world / (e2e_ms / e2e_steps * 1e-3) / 1e9, "unit": "GB/s",
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                    "api": "wash_step_host(WASH_OP_SHUFFLE) on pinned host stacks: copy in, shuffle, copy out inside the timed region",
                    "full_step": {"ms_per_step": e2e_full_ms / e2e_steps, "d2h_bytes_per_step": d2h_full,
                                  "GBps": ab["step"] * world / (e2e_full_ms / e2e_steps * 1e-3) / 1e9,
                                  "api": "wash_step_host with shuffle + EMA + average"}},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "shuffle_back_to_back": main_cell,
        }
        if clocks.get("sm_mhz"):
            line["roofline"]["ms_x_sm_mhz"] = float(med_ms[0]) * clocks["sm_mhz"]
        if world == 1 and not args.no_configs:
            line["configs"] = configs_record(B, torch, stream, peak, philox_rate, wl.name, main_cell)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(wl)
        print(json.dumps(line), flush=True)
    pop.close()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


# DRAM bytes per shuffle launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture
# of the kernel as it stands, summarised under profiles/), per (workload, mode).  A workload
# without a capture of the current kernel has no entry and the bench line says null.
TRAFFIC = {
    # shuffle_async_kernel<F32, F32, [N][P], 1, lean>: 2045.02 MB read + 34.07 MB written per launch (mean of two launches)
    ("cfg3_resnet50_n10", "stream"): {"dram_bytes": 2045.02e6 + 34.07e6,
                                      "source": "profiles/shuffle_async_kernel_cfg3_resnet50_n10.md"},
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
    steps, sel, t_shuffle, t0 = 0, 0, 0.0, time.perf_counter()
    while True:
        t1 = time.perf_counter()
        sel += oracle.shuffle(pop, params, p, seed=SEED, step=steps, stack2=opt)[0]
        t_shuffle += time.perf_counter() - t1
        oracle.papa_ema(pop, params, ALPHA)
        oracle.population_average(pop, params, out)
        steps += 1
        dt = time.perf_counter() - t0
        if dt > 10.0 or steps >= 2000:
            break
    ab = wl.algorithmic_bytes(sel / steps)
    return {"value": ab["shuffle"] * steps / t_shuffle / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": "%d full steps of the same workload (%.1f s); value = the shuffle's bytes / the time inside the oracle's shuffle" % (steps, dt),
            "ms_per_step": dt / steps * 1e3, "step_GBps": ab["step"] * steps / dt / 1e9,
            "param_swaps_per_s": sel * wl.N / t_shuffle}


def run_sweep(args) -> None:
    """Config 5: flat fp32 populations, N x P x p x layout, shuffle only.  One JSON line
    per cell (not the default bench line)."""
    import torch
    from paper_2405_17517_b200 import binding as B

    torch.cuda.set_device(0)
    B.load()
    peak, _ = measured_peak()
    modes = {"stream": B.WASH_MODE_STREAM, "sparse": B.WASH_MODE_SPARSE}
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


def run_exchange_ranks(args, rank: int, world: int, local_rank: int) -> None:
    """The paper's own deployment: one model per rank, the ranks of the process group being the
    population.  Every rank builds an ExchangeWorker on its model's row (and momentum), runs
    --steps steps (plan, send by peer stores, barrier, receive) and rank 0 prints one JSON line:
    step time (CUDA events on the launching stream, max over ranks), values and bytes a rank
    receives per step, and whether the plan's slot counts equal the oracle's for the last step.
    With one GPU per rank the group is NCCL and the barrier between send and receive is an
    all-reduce on the stream; when the ranks have to share a device the group is gloo and the
    barrier is on the host (a functional stand-in, not a measurement of the link)."""
    import torch
    import torch.distributed as dist
    from paper_2405_17517_b200 import binding as B
    from paper_2405_17517_b200.exchange import ExchangeWorker

    if world < 2:
        raise SystemExit("--exchange-ranks needs a population: launch with torchrun, --nproc-per-node >= 2")
    own_gpu = torch.cuda.device_count() >= world
    device = local_rank if own_gpu else 0
    torch.cuda.set_device(device)
    if own_gpu:
        dist.init_process_group("nccl", device_id=torch.device("cuda", device))
    else:
        dist.init_process_group("gloo")
    B.load()
    wl = Workload(args.workload)
    N = world                                   # the population is the process group
    stream = torch.cuda.current_stream()
    ctx_probe = B.wash_create(N, wl.numel, B.WASH_LAYOUT_NP, device)
    P = B.wash_stack_elems(ctx_probe, wl.T)[0]
    B.wash_destroy(ctx_probe)
    gen = torch.Generator(device="cuda").manual_seed(SEED + 31 * rank)
    row = (torch.randn(P, generator=gen, device="cuda") * 0.05).to(torch.bfloat16 if wl.bf16 else torch.float32)
    opt = torch.randn(P, generator=gen, device="cuda") * 1e-3 if wl.opt else None
    p_layer = B.wash_layer_probs(wl.T, wl.p, B.WASH_SCHEDULE_DECREASING) if wl.schedule == "decreasing" else None
    p_eff = wl.p if p_layer is None else float((p_layer * wl.numel).sum() / wl.P)
    capacity = max(1 << 14, int(4 * p_eff * wl.P))
    worker = ExchangeWorker(wl.numel, row, opt, capacity=capacity, device=device)
    stats = torch.zeros(2, dtype=torch.int64, device="cuda")

    def fence():
        torch.cuda.synchronize()
        dist.barrier()

    for w in range(args.warmup):
        worker.step(w, wl.p, p_layer, SEED)
    fence()
    worker.check()
    K = args.steps
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
    t0 = time.perf_counter()
    ev[0].record(stream)
    for k in range(K):
        worker.step(args.warmup + k, wl.p, p_layer, SEED, stats)
        ev[k + 1].record(stream)
    fence()
    wall = time.perf_counter() - t0
    worker.check()
    per_step = np.array([ev[k].elapsed_time(ev[k + 1]) for k in range(K)])
    need, selected = B.wash_exchange_counts(worker.ctx, N)          # the plan of the last step
    t = torch.tensor([float(np.median(per_step)), float(per_step.min()), wall / K * 1e3], dtype=torch.float64,
                     device="cuda" if own_gpu else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    c = torch.tensor([int(stats[1])], dtype=torch.int64, device="cuda" if own_gpu else "cpu")
    dist.all_reduce(c, op=dist.ReduceOp.SUM)
    if rank == 0:
        import oracle
        offsets, padded_P = W.padded_offsets(wl.numel)
        ora = oracle.Population(N, wl.numel, offsets, padded_P, oracle.LAYOUT_NP)
        oracle.set_threads(oracle.max_threads())
        want_need, want_sel = oracle.exchange_counts(ora, wl.p if p_layer is None else p_layer, SEED, args.warmup + K - 1)
        received = int(c[0]) / K / N                       # values one rank receives per step
        elem = wl.E + wl.E_opt
        step_ms = float(t[0]) if own_gpu else float(t[2])  # host-ordered steps are not bracketed by stream events alone
        print(json.dumps({
            "arm": "exchange-ranks", "workload": wl.name, "ranks": N, "backend": "nccl" if own_gpu else "gloo (ranks share device 0, barrier on the host)",
            "steps": K, "warmup": args.warmup, "step_us": step_ms * 1e3, "step_us_min": float(t[1]) * 1e3 if own_gpu else None,
            "selected_coords_per_step": selected, "values_received_per_rank_per_step": received,
            "expected_values_per_rank_per_step": p_eff * wl.P * (N - 1) / N,
            "link_bytes_in_per_rank_per_step": received * elem, "model_bytes_per_rank": wl.P * elem,
            "counts_match_oracle": bool(list(need) == [int(x) for x in want_need] and selected == want_sel),
            "staging_capacity_elems": worker.capacity,
            "timing": "CUDA events on the launching stream per step, median, max over ranks" if own_gpu else "wall clock per step, max over ranks",
        }), flush=True)
    worker.close()
    dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_resnet50_n10", choices=sorted(W.CONFIGS))
    ap.add_argument("--mode", default="stream", choices=["stream", "sparse", "auto"])
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--blocks-per-sm", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--min-timed-s", type=float, default=MIN_TIMED_S,
                    help="repeat the timed block of --steps steps until this much GPU time has been measured (0: one block; for profiler runs)")
    ap.add_argument("--no-configs", action="store_true", help="skip the record of the other configurations (configs 1-4, cells of config 5)")
    ap.add_argument("--sweep", action="store_true", help="config-5 sweep of the shuffle kernel (many JSON lines)")
    ap.add_argument("--sweep-modes", default="stream,sparse")
    ap.add_argument("--sweep-N", default="", help="comma list; default 2,4,8,16,32")
    ap.add_argument("--sweep-logP", default="", help="comma list; default 20,24,27")
    ap.add_argument("--sweep-p", default="", help="comma list; default 1e-4..1")
    ap.add_argument("--sweep-layout", default="", choices=["", "np", "pn"])
    ap.add_argument("--exchange-warm", action="store_true", help="with --exchange: no L2 flush between steps")
    ap.add_argument("--exchange", action="store_true", help="time one worker of the one-model-per-device form (JSON line per workload)")
    ap.add_argument("--exchange-ranks", action="store_true",
                    help="under torchrun: the ranks are the population, one model per rank, steps through ExchangeWorker (one JSON line)")
    args = ap.parse_args()
    args.workload_given = any(a == "--workload" or a.startswith("--workload=") for a in sys.argv[1:])
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.min_timed_s <= 0:
        global B2B_MIN_S
        B2B_MIN_S = 0.0
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.sweep:
        run_sweep(args)
        return
    if args.exchange:
        run_exchange(args)
        return
    if args.exchange_ranks:
        run_exchange_ranks(args, rank, world, local_rank)
        return
    if args.impl == "reference":
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
