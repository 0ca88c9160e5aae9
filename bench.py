#!/usr/bin/env python
"""Benchmark of the allocation search: candidate x level pairs scored per second.

A step is one pass of the whole hot path -- level preparation, scoring of every
(candidate, demand level) pair, cross-block reduction, winner decode -- over one
demand sweep of the named workload.  One process per GPU; with N > 1 every rank
solves its own sweep of the same length (the path shards by demand level with no
exchange), so scaling is weak and the value is the sum over ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C4]
    python bench.py --impl reference ...     # the CPU oracle on a bounded sample
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2407_03583_b200 import workloads as W  # noqa: E402

METRIC = "candidate-level pairs scored per second (allocation search)"
UNIT = "pairs/s"
SM_COUNT_NOMINAL = 148
# Algorithmic work of one (candidate, level) pair on the direct path: one FP64
# fused multiply-add per option part (the exact worker count of that part).  The
# FP64 pipe is the unit that bounds the kernel: 64 lanes per SM.
FMA_PER_PART = 1
FP64_LANES_PER_SM = 64


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except Exception:
        return None


def profiled_traffic(kernel: str, workload: str):
    """Executed FP64 thread-instructions per scoring launch from the committed ncu
    summary, in Gfma -- or None when there is none for this kernel/workload or the
    kernel source has changed since the counters were taken."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "counters.json")) as f:
            table = json.load(f)
        entry = table["%s_score_kernel/%s" % (kernel, workload)]
        h = hashlib.sha1()
        for name in entry["sources"]:
            h.update(open(os.path.join(ROOT, "paper_2407_03583_b200", "csrc", name), "rb").read())
        if h.hexdigest() != entry["sources_sha1"]:
            return None
        return entry["fp64_thread_inst_per_launch"] / 1e9
    except Exception:
        return None


def latency_feasible_fraction(w):
    """Share of the candidates that pass the latency bound on every root-to-leaf path, counted
    on the host with numpy (single-option workloads only).  The level-lane kernel executes fmas
    for these candidates alone, so its roofline line counts only them."""
    import numpy as np
    if w.split_mode:
        return None
    T, nb = w.n_tasks, len(w.batch_sizes)
    lat = np.asarray(w.latency_us, dtype=np.int64).reshape(-1, nb)
    off = np.cumsum([0] + list(w.n_variants))
    per = [lat[off[i]:off[i + 1]].reshape(-1).astype(np.int32) for i in range(T)]
    leaves = [i for i in range(T) if i not in w.parent]
    ok = None
    for lf in leaves:
        path, i = [], lf
        while i >= 0:
            path.append(i)
            i = w.parent[i]
        total = np.zeros([len(p) for p in per], dtype=np.int32)
        for i in path:
            shape = [1] * T
            shape[i] = len(per[i])
            total = total + per[i].reshape(shape)
        good = 2 * total.astype(np.int64) <= w.slo_us - len(path) * w.comm_us
        ok = good if ok is None else (ok & good)
    return float(ok.mean())


def fp64_probe():
    """Runs the package's stand-alone FP64 issue-rate probe (built beside the library) and
    returns its JSON, or None when it is not built or fails."""
    exe = os.path.join(ROOT, "paper_2407_03583_b200", "fp64_issue_probe")
    if not os.path.exists(exe):
        return None
    try:
        r = subprocess.run([exe], capture_output=True, text=True, timeout=60)
        return json.loads(r.stdout.strip().splitlines()[-1]) if r.returncode == 0 else None
    except Exception:
        return None


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.lines = []
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "25"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.perf_counter(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [l for (t, l) in self.lines if t0 - 0.05 <= t <= t1 + 0.15] or [l for (_t, l) in self.lines]
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            parts = [x.strip() for x in l.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None,
                "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_sample(w, seconds_target: float, n_threads: int):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload:
    a leading candidate range times all levels, grown until it takes about
    ``seconds_target`` seconds.  Returns (pairs_per_second, description, seconds)."""
    import oracle
    n = w.n_candidates()
    m = w.n_levels
    span = min(n, 1 << 16)
    while True:
        t0 = time.perf_counter()
        oracle.solve(w, n_threads=n_threads, cand_range=(0, span))
        dt = time.perf_counter() - t0
        if dt >= 0.5 * seconds_target or span >= n:
            break
        grow = max(2.0, min(16.0, seconds_target / max(dt, 1e-3)))
        span = min(n, int(span * grow))
    pairs = span * m
    return pairs / dt, "candidates [0, %d) of %d x all %d levels" % (span, n, m), dt


def run_reference(args):
    """The reference arm: the CPU oracle on the machine's host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    w = W.make_workload(args.workload)
    cores = os.cpu_count() or 1
    per_step = max(1.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    for _ in range(args.warmup):
        oracle_sample(w, per_step, cores)
    vals, secs, desc = [], [], ""
    for _ in range(args.steps):
        v, desc, dt = oracle_sample(w, per_step, cores)
        vals.append(v)
        secs.append(dt)
    value = statistics.mean(vals)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(secs),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int64+f64",
        "data": "synthetic",
        "config": {"workload": args.workload, "n_candidates": w.n_candidates(), "n_levels": w.n_levels,
                   "note": "CPU oracle, each step a bounded sample of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4", choices=list(W.WORKLOAD_NAMES))
    ap.add_argument("--path", default="auto", choices=["auto", "generic", "direct", "hoisted", "uniform", "fastest"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--variant-factors", action="store_true",
                    help="give every variant a seeded multiplicative factor in 1.0..2.0 (the paper's Eq. 1 model); "
                         "the library then takes its root-first level-lane kernel")
    ap.add_argument("--fp64-probe", action="store_true",
                    help="only run the FP64 issue-rate probe and print its JSON line")
    args = ap.parse_args()
    if args.fp64_probe:
        print(json.dumps(fp64_probe()))
        return 0
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist
    from paper_2407_03583_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    base = W.make_workload(args.workload)
    m = base.n_levels
    # every rank solves its own sweep of the workload's length (weak scaling by level)
    w = W.shard_sweep(args.workload, rank, world)
    if args.variant_factors:
        frng = W.SplitMix64(99)
        w.variant_fanout_milli = [1000 + int(frng.randint(0, 8)) * 125 for _ in range(sum(w.n_variants))]
        base.variant_fanout_milli = list(w.variant_fanout_milli)
    n_cand = w.n_candidates()
    pairs_per_step = n_cand * m

    alloc = B.Allocator(w, device="cuda:%d" % local_rank)
    alloc.set_path({"auto": B.LOKI_PATH_AUTO, "generic": B.LOKI_PATH_GENERIC,
                    "direct": B.LOKI_PATH_DIRECT, "hoisted": B.LOKI_PATH_HOISTED,
                    "uniform": B.LOKI_PATH_UNIFORM, "fastest": B.LOKI_PATH_FASTEST}[args.path])
    B.loki_alloc_set_timing(alloc.handle, True)
    alloc.upload(w.demand_mqps)
    alloc.solve_device(m)                   # untimed: also resolves which kernel this sweep takes
    torch.cuda.synchronize(dev)
    info = alloc.info()
    path_name = {B.LOKI_PATH_GENERIC: "generic", B.LOKI_PATH_DIRECT: "direct",
                 B.LOKI_PATH_HOISTED: "hoisted", B.LOKI_PATH_UNIFORM: "uniform"}[info.path_last]
    alloc.h_demand[:m] = torch.tensor(w.demand_mqps, dtype=torch.int64)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2
    torch.cuda.synchronize(dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    # ---- device-resident timing --------------------------------------------
    for _ in range(args.warmup):
        alloc.solve_device(m)
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    stops = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    score_ms, score_launches = [], 0
    barrier()
    t_region0 = time.perf_counter()
    for k in range(args.steps):
        flush.fill_(k & 0xFF)                 # L2 flush between timed iterations (untimed)
        starts[k].record()
        alloc.solve_device(m)
        stops[k].record()
        ms, nl = B.loki_alloc_last_score_ms(alloc.handle)
        score_ms.append(ms)
        score_launches = nl
    barrier()
    t_region1 = time.perf_counter()
    clocks = sampler.stop(t_region0, t_region1) if rank == 0 else None
    step_ms = [s.elapsed_time(e) for s, e in zip(starts, stops)]
    total_ms = sum(step_ms)
    launches_per_step = alloc.info().n_launches_last
    n_tiles = score_launches
    kernels_per_step = launches_per_step - (n_tiles if path_name == "direct" else 0)

    # ---- end-to-end through the host-buffer entry point ----------------------
    for _ in range(2):
        alloc.solve_host(m)
    barrier()
    e2e_t0 = time.perf_counter()
    for k in range(args.steps):
        alloc.solve_host(m)
    torch.cuda.synchronize(dev)
    e2e_s = time.perf_counter() - e2e_t0

    # ---- request routing for the same sweep (reported beside the step, not part of it) ----
    import ctypes
    mw, me = w.cluster_size, 2 * w.cluster_size + w.n_tasks
    d_rh = torch.empty(m * ctypes.sizeof(B.loki_route_header_t), dtype=torch.uint8, device=dev)
    d_rw = torch.empty(m * mw * ctypes.sizeof(B.loki_route_worker_t), dtype=torch.uint8, device=dev)
    d_re = torch.empty(m * me * ctypes.sizeof(B.loki_route_entry_t), dtype=torch.uint8, device=dev)
    alloc.solve_device(m)
    r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    route_ms = []
    for k in range(5):
        r0.record()
        B.loki_alloc_route(alloc.handle, alloc.d_demand.data_ptr(), alloc.d_out.data_ptr(), m, mw, me,
                           torch.cuda.current_stream(dev).cuda_stream, d_rh.data_ptr(), d_rw.data_ptr(),
                           d_re.data_ptr())
        r1.record()
        torch.cuda.synchronize(dev)
        route_ms.append(r0.elapsed_time(r1))

    # ---- the tabulated (hoisted) scoring kernel on the same sweep, reported beside the step ----
    tab_ms = None
    if path_name != "hoisted" and info.hoisted_ok:
        alloc.set_path(B.LOKI_PATH_HOISTED)
        ms_list, step_list = [], []
        t0e, t1e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for k in range(13):
            flush.fill_(k & 0xFF)
            t0e.record()
            alloc.solve_device(m)
            t1e.record()
            ms, _nl = B.loki_alloc_last_score_ms(alloc.handle)
            torch.cuda.synchronize(dev)
            if k >= 3:
                ms_list.append(ms)
                step_list.append(t0e.elapsed_time(t1e))
        tab_ms = statistics.mean(ms_list)
        tab_step_ms = statistics.mean(step_list)
        alloc.set_path(info.path_current)

    t_dev = torch.tensor([total_ms, e2e_s * 1e3], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t_dev, op=dist.ReduceOp.MAX)
    total_ms_max, e2e_ms_max = [float(x) for x in t_dev.cpu()]

    rc = 0
    if rank == 0:
        value = pairs_per_step * world * args.steps / (total_ms_max * 1e-3)
        e2e_value = pairs_per_step * world * args.steps / (e2e_ms_max * 1e-3)
        k1_ms = statistics.mean(score_ms) / max(1, n_tiles)        # average scoring launch
        parts = w.n_tasks * (2 if w.split_mode else 1)
        fma_per_pair = FMA_PER_PART * parts
        pairs_per_launch = pairs_per_step / max(1, n_tiles)
        root_first = path_name == "uniform"     # the level-lane path: the root-first kernel
        executed_share = None
        achieved = pairs_per_launch * fma_per_pair * (executed_share or 1.0) / (k1_ms * 1e-3) / 1e9
        peaks = measured_peaks()
        sm_max_mhz = (peaks or {}).get("sm_max_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
        n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
        peak = n_sms * FP64_LANES_PER_SM * sm_max_mhz * 1e6 / 1e9
        traffic = profiled_traffic(path_name, args.workload)
        peak_src = "%d SMs x %%s x %.0f MHz (max SM clock%s)" % (
            n_sms, sm_max_mhz, " of MEASURED_PEAKS.json" if peaks else ", nominal")
        variant = root_first        # the root-first kernel, with or without per-variant factors
        if path_name == "hoisted" or variant:
            # these kernels score a pair with a handful of plain instructions, not with one fma per part:
            # their ceiling is instruction issue (4 warp-instructions per clock per SM), and the algorithmic
            # work is counted on the pairs of latency-feasible candidates, the only ones they visit
            share = latency_feasible_fraction(w)
            per_pair = (2 if w.split_mode else 1) + 3 if variant else 3
            issue_peak = n_sms * 4 * sm_max_mhz * 1e6 / 1e9
            ach = pairs_per_launch * (share or 1.0) * per_pair / 32.0 / (k1_ms * 1e-3) / 1e9
            roof = {"bound": "alu", "kernel": "variant_score_kernel" if variant else "hoisted_score_kernel",
                    "achieved": ach, "peak": issue_peak, "unit": "G warp-instructions/s (issue)",
                    "frac": ach / issue_peak, "traffic": None, "launch_ms": k1_ms,
                    "thread_instructions_per_pair": per_pair, "pairs_per_launch": pairs_per_launch,
                    "pairs_counted": ("latency-feasible pairs only (share %.4f)" % share) if share else "all pairs",
                    "peak_source": peak_src % "4 schedulers"}
        else:
            roof = {"bound": "alu", "kernel": "%s_score_kernel" % path_name,
                    "achieved": achieved, "peak": peak, "unit": "Gfma/s (FP64)",
                    "frac": achieved / peak, "traffic": traffic,
                    "launch_ms": k1_ms, "fma_per_pair": fma_per_pair, "pairs_per_launch": pairs_per_launch,
                    "fma_counted": ("latency-feasible pairs only (share %.4f): the kernel skips the rest"
                                    % executed_share) if executed_share else "all pairs",
                    "peak_source": peak_src % ("%d FP64 lanes" % FP64_LANES_PER_SM)}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms_max / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32/u64+f64",
            "data": "synthetic",
            "config": {"workload": args.workload, "n_candidates": n_cand, "n_levels_per_gpu": m,
                       "pairs_per_step_per_gpu": pairs_per_step, "kernel": path_name,
                       "variant_factors": bool(args.variant_factors),
                       "parallelism": "levels sharded, no exchange" if world > 1 else "1 GPU",
                       "l2": "flushed between timed iterations (256 MiB write)",
                       "checksum": "%016x" % w.checksum()},
            "solves_per_s": m * world * args.steps / (total_ms_max * 1e-3),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 8 * m,
                    "d2h_bytes_per_step": B.CONFIG_SIZE * m, "ms_per_step": e2e_ms_max / args.steps},
            "gpu_launches": kernels_per_step * args.steps,
            "routing": {"kernel": "route_kernel", "levels": m, "ms_per_sweep": min(route_ms[1:]),
                        "note": "MostAccurateFirst tables for the sweep's plans; outside the timed step"},
            "tabulated": None if tab_ms is None else {
                "kernel": "hoisted_score_kernel", "score_ms_per_sweep": tab_ms,
                "pairs_per_s_scoring": pairs_per_step / (tab_ms * 1e-3),
                "ms_per_step": tab_step_ms, "pairs_per_s_step": pairs_per_step / (tab_step_ms * 1e-3),
                "note": "worker arithmetic once per (level, task, option), one table read + add + min per pair; "
                        "opt-in path, outside the timed step"},
            "roofline": roof,
        }
        if world == 1 and not args.no_cpu_baseline:
            # measured issue rate of the fma forms, after the timed regions: what the FP64 pipe
            # delivers with three register sources (the direct kernel's form) and with one
            # uniform source (the rate the nominal peak assumes)
            probe = fp64_probe()
            if probe and "fma_warp_inst_per_clk_per_sm" in probe and "fma_per_pair" in roof:
                rates = probe["fma_warp_inst_per_clk_per_sm"]
                line["roofline"]["fp64_probe"] = rates
                reg_peak = peak * rates["register_sources"] / 2.0
                line["roofline"]["frac_of_register_source_rate"] = achieved / reg_peak
        if world == 1 and not args.no_cpu_baseline:
            cores = os.cpu_count() or 1
            v, desc, dt = oracle_sample(base, 12.0, cores)
            v1, desc1, dt1 = oracle_sample(base, 4.0, 1)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": desc + " (%.1f s)" % dt,
                                    "one_core": {"value": v1, "sample": desc1 + " (%.1f s)" % dt1}}
        else:
            line["cpu_baseline"] = None
        bad = set((clocks or {}).get("reasons") or []) & {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
        if bad:
            line["clocks"]["rejected"] = sorted(bad)
        print(json.dumps(line))
    alloc.close()
    if world > 1:
        dist.destroy_process_group()
    return rc


if __name__ == "__main__":
    sys.exit(main())
