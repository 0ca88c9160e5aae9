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


def profiled_counters(kernel: str, workload: str):
    """The committed ncu counters of one scoring launch (profiles/counters.json: DRAM bytes,
    executed instructions) -- or None when there are none for this kernel/workload or the
    kernel source has changed since they were taken.  A cross-check only: what the bench
    line reports as executed work is counted by the kernel in this very run."""
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
        return entry
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
    """Runs the stand-alone FP64 issue-rate probe (fp64_issue_probe.cu beside this file, built by
    __graft_entry__.build) and returns its JSON, or None when it is not built or fails."""
    exe = os.path.join(ROOT, "fp64_issue_probe")
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


PATHS = {"auto": 0, "generic": 1, "direct": 2, "hoisted": 3, "uniform": 4, "fastest": 5, "prefix": 6, "shared": 7}
PATH_NAMES = {1: "generic", 2: "direct", 3: "hoisted", 4: "uniform", 6: "prefix", 7: "prefix"}


def roofline_for(B, alloc, w, path_name, k1_ms_total, n_launches, n_sms, sm_max_mhz, peaks, workload):
    """The roofline object of the scoring kernel that ran ("Measurement")."""
    m = w.n_levels
    parts = w.n_tasks * (2 if w.split_mode else 1)
    pairs = w.n_candidates() * m
    k1_ms = k1_ms_total / max(1, n_launches)             # average scoring launch
    peak_src = "%d SMs x %%s x %.0f MHz (max SM clock%s)" % (
        n_sms, sm_max_mhz, " of MEASURED_PEAKS.json" if peaks else ", nominal")
    if path_name == "direct":
        # bound by the FP64 pipe: one fma per (staged candidate, level, option part); the kernel counts
        # the rows of 32 candidates it scores, so `executed` is what ran in this very solve
        peak = n_sms * FP64_LANES_PER_SM * sm_max_mhz * 1e6 / 1e9
        executed = B.loki_alloc_last_fma_count(alloc.handle)
        achieved = executed / max(1, n_launches) / (k1_ms * 1e-3) / 1e9
        all_pairs = pairs * parts / (k1_ms_total * 1e-3) / 1e9
        prof = profiled_counters(path_name, workload)
        return {"bound": "alu", "kernel": "direct_score_kernel", "achieved": achieved, "peak": peak,
                "unit": "Gfma/s (FP64)", "frac": achieved / peak, "frac_executed": achieved / peak,
                "frac_all_pairs": all_pairs / peak,
                "traffic": None if prof is None else prof.get("dram_bytes_per_launch"),
                "launch_ms": k1_ms, "launches": n_launches, "fma_per_pair": parts,
                "fma_executed_per_launch": executed / max(1, n_launches),
                "fma_all_pairs_per_launch": pairs * parts / max(1, n_launches),
                "fma_counted": "executed: counted by the kernel in this run (latency-feasible candidates only, "
                               "the ragged last row of a class tuple's share and a tile's padding levels, if any, included); frac_all_pairs credits "
                               "one fma per part of every pair, also of candidates the latency bound removed",
                "peak_source": peak_src % ("%d FP64 lanes" % FP64_LANES_PER_SM)}
    # the other kernels score a pair with a handful of plain instructions: their ceiling is instruction
    # issue (4 warp-instructions per clock per SM); the work is MODELLED, not counted: thread-instructions
    # per pair of the innermost loop times the pairs of latency-feasible candidates (the only ones visited)
    if path_name == "prefix":
        # the hoisted tables with prefix minima: the innermost task's candidates are not visited one by
        # one, so there is no per-pair instruction count to hold against the issue rate
        return {"bound": "alu", "kernel": "hoisted_score_kernel (prefix minima)", "achieved": None, "peak": None,
                "unit": "G warp-instructions/s (issue)", "frac": None, "traffic": None,
                "launch_ms": k1_ms, "launches": n_launches,
                "pairs_counted": "none: the answer covers all pairs, the kernel reads one table row per fitting prefix"}
    share = latency_feasible_fraction(w) if path_name in ("hoisted", "uniform") else None
    per_pair = {"hoisted": 3, "uniform": (2 if w.split_mode else 1) + 3, "generic": 13 * parts + 8}[path_name]
    issue_peak = n_sms * 4 * sm_max_mhz * 1e6 / 1e9
    ach = pairs * (share or 1.0) * per_pair / 32.0 / (k1_ms_total * 1e-3) / 1e9
    prof = profiled_counters(path_name, workload) if n_launches == 1 else None
    return {"bound": "alu", "kernel": {"hoisted": "hoisted_score_kernel", "uniform": "variant_score_kernel",
                                       "generic": "generic_score_kernel"}[path_name],
            "achieved": ach, "peak": issue_peak, "unit": "G warp-instructions/s (issue)", "frac": ach / issue_peak,
            "modelled": True,
            # all warp instructions of the launch (committed ncu count, while the sources are unchanged) against the
            # same issue peak: how busy the schedulers are, useful work or not
            "frac_issued": None if prof is None else prof["warp_inst_per_launch"] / (k1_ms * 1e-3) / 1e9 / issue_peak,
            "traffic": None if prof is None else prof.get("dram_bytes_per_launch"),
            "launch_ms": k1_ms, "launches": n_launches,
            "thread_instructions_per_pair": per_pair,
            "pairs_counted": ("latency-feasible pairs only (share %.4f)" % share) if share else "all pairs",
            "peak_source": peak_src % "4 schedulers"}


def run_one(B, torch, dist, args, name, path, dev, rank, world, local_rank, flush, extras):
    """Times one workload on one path; returns the JSON line (rank 0) or None."""
    base = W.make_workload(name)
    m = base.n_levels
    # every rank solves its own sweep of the workload's length (weak scaling by level)
    w = W.shard_sweep(name, rank, world)
    if args.variant_factors:
        frng = W.SplitMix64(99)
        w.variant_fanout_milli = [1000 + int(frng.randint(0, 8)) * 125 for _ in range(sum(w.n_variants))]
        base.variant_fanout_milli = list(w.variant_fanout_milli)
    n_cand = w.n_candidates()
    pairs_per_step = n_cand * m

    alloc = B.Allocator(w, device="cuda:%d" % local_rank)
    try:
        alloc.set_path(PATHS[path])
    except B.LokiError:
        alloc.close()
        return None                          # this kernel does not apply to this problem
    B.loki_alloc_set_timing(alloc.handle, True)
    alloc.upload(w.demand_mqps)
    alloc.solve_device(m)                   # untimed: also resolves which kernel this sweep takes
    torch.cuda.synchronize(dev)
    info = alloc.info()
    path_name = PATH_NAMES[info.path_last]
    alloc.h_demand[:m] = torch.tensor(w.demand_mqps, dtype=torch.int64)
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
    info = alloc.info()
    launches_per_step = info.n_launches_last
    # the direct kernel's demand tile is refreshed by one device-to-device copy per scoring launch
    kernels_per_step = launches_per_step - (score_launches if path_name == "direct" else 0)

    # ---- sustained: back-to-back solves for a few seconds, clocks sampled meanwhile ----
    sustained = None
    if extras and args.sustain > 0 and world == 1:
        n_est = max(10, int(args.sustain * 1e3 / max(1e-3, total_ms / args.steps)))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        smp = ClockSampler(local_rank)
        smp.start()
        time.sleep(0.2)
        torch.cuda.synchronize(dev)
        ts0 = time.perf_counter()
        s0.record()
        for _ in range(n_est):
            alloc.solve_device(m)
        s1.record()
        torch.cuda.synchronize(dev)
        ts1 = time.perf_counter()
        ck = smp.stop(ts0, ts1)
        sus_ms = s0.elapsed_time(s1) / n_est
        sustained = {"seconds": ts1 - ts0, "solves": n_est, "ms_per_step": sus_ms,
                     "pairs_per_s": pairs_per_step / (sus_ms * 1e-3), "clocks": ck,
                     "ms_x_sm_mhz": None if not ck.get("sm_mhz") else sus_ms * ck["sm_mhz"],
                     "note": "no L2 flush and no host synchronisation between solves (tables are L2-resident by design)"}

    # ---- end-to-end through the host-buffer entry point ----------------------
    for _ in range(2):
        alloc.solve_host(m)
    barrier()
    e2e_t0 = time.perf_counter()
    for k in range(args.steps):
        alloc.solve_host(m)
    torch.cuda.synchronize(dev)
    e2e_s = time.perf_counter() - e2e_t0

    route_ms = tab = None
    if extras:
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

        # ---- the kernel LOKI_PATH_FASTEST picks for the same sweep, reported beside the step; its
        #      plans must be the bytes the timed kernel wrote ----
        want = alloc.d_out[: m * B.CONFIG_SIZE].clone()
        alloc.set_path(B.LOKI_PATH_FASTEST)
        alloc.solve_device(m)
        torch.cuda.synchronize(dev)
        fast_name = PATH_NAMES[alloc.info().path_last]
        if fast_name != path_name:
            same = bool(torch.equal(want, alloc.d_out[: m * B.CONFIG_SIZE]))
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
            share = latency_feasible_fraction(w)
            tab_ms, tab_step_ms = statistics.mean(ms_list), statistics.mean(step_list)
            if fast_name == "prefix":
                share = None                  # its walk does not visit the innermost task's candidates one by one
            tab = {"kernel": {"uniform": "variant_score_kernel", "prefix": "hoisted_score_kernel (prefix minima)"}.get(
                       fast_name, fast_name + "_score_kernel"),
                   "plans_equal_to_timed_kernel": same, "score_ms_per_sweep": tab_ms, "ms_per_step": tab_step_ms,
                   "pairs_per_s_step": pairs_per_step / (tab_step_ms * 1e-3),
                   "pairs_visited_per_s_step": None if share is None else pairs_per_step * share / (tab_step_ms * 1e-3),
                   "note": "what LOKI_PATH_AUTO runs for this sweep; pairs_per_s counts all N x M pairs the answer "
                           "covers, pairs_visited only those the kernel walks one by one (latency-feasible "
                           "candidates; none with prefix minima); outside the timed step"}
        alloc.set_path(PATHS[path])

    slo_sweep = None
    if extras and world == 1:
        # ---- the SLO study (Section 6.4) as one call: workload SM's sweep under 16 SLOs; the hoisted kernel
        #      takes the SLOs as a second batched axis of its launches, the direct path loops over them ----
        wsm = W.make_workload("SM")
        slos = [15_000 + 25_000 * k for k in range(16)]
        asm = B.Allocator(wsm, device="cuda:%d" % local_rank)
        nsm = asm.upload(wsm.demand_mqps)
        out_sm = torch.empty(len(slos) * nsm * B.CONFIG_SIZE, dtype=torch.uint8, device=dev)
        stream = torch.cuda.current_stream(dev).cuda_stream
        res, keep = {}, {}
        for nm, pth in (("fused_hoisted", B.LOKI_PATH_FASTEST), ("looped_direct", B.LOKI_PATH_DIRECT)):
            asm.set_path(pth)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ts = []
            for k in range(8):
                e0.record()
                B.loki_alloc_solve_slos(asm.handle, asm.d_demand.data_ptr(), nsm, slos, stream, out_sm.data_ptr())
                e1.record()
                torch.cuda.synchronize(dev)
                if k >= 3:
                    ts.append(e0.elapsed_time(e1))
            res[nm] = {"ms": statistics.mean(ts), "launches": asm.info().n_launches_last}
            keep[nm] = out_sm.clone()
        slo_sweep = {"workload": "SM", "n_levels": nsm, "n_slos": len(slos), **res,
                     "plans_equal": bool(torch.equal(keep["fused_hoisted"], keep["looped_direct"])),
                     "solves_per_s_fused": nsm * len(slos) / (res["fused_hoisted"]["ms"] * 1e-3)}
        asm.close()

    t_dev = torch.tensor([total_ms, e2e_s * 1e3], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t_dev, op=dist.ReduceOp.MAX)
    total_ms_max, e2e_ms_max = [float(x) for x in t_dev.cpu()]

    line = None
    if rank == 0:
        value = pairs_per_step * world * args.steps / (total_ms_max * 1e-3)
        e2e_value = pairs_per_step * world * args.steps / (e2e_ms_max * 1e-3)
        peaks = measured_peaks()
        sm_max_mhz = (peaks or {}).get("sm_max_mhz") or (clocks or {}).get("sm_max_mhz") or 1965.0
        n_sms = torch.cuda.get_device_properties(dev).multi_processor_count
        alloc.solve_device(m)                 # the executed-work counter is read for this solve
        torch.cuda.synchronize(dev)
        roof = roofline_for(B, alloc, w, path_name, statistics.mean(score_ms), score_launches, n_sms,
                            sm_max_mhz, peaks, name)
        if (clocks or {}).get("sm_mhz") and roof["frac"] is not None:
            # the same fraction against the clock seen during the timed region
            roof["frac_at_sampled_clock"] = roof["frac"] * sm_max_mhz / clocks["sm_mhz"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms_max / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32/u64+f64",
            "data": "synthetic",
            "config": {"workload": name, "n_candidates": n_cand, "n_levels": m,
                       "pairs_per_step_per_gpu": pairs_per_step, "kernel": path_name, "path": path,
                       "variant_factors": bool(args.variant_factors),
                       "parallelism": "levels sharded, no exchange" if world > 1 else "1 GPU",
                       "l2": "flushed between timed iterations (256 MiB write)",
                       "checksum": "%016x" % w.checksum()},
            "solves_per_s": m * world * args.steps / (total_ms_max * 1e-3),
            "step_minus_scoring_ms": total_ms_max / args.steps - statistics.mean(score_ms),
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 8 * m,
                    "d2h_bytes_per_step": B.CONFIG_SIZE * m, "ms_per_step": e2e_ms_max / args.steps},
            "gpu_launches": kernels_per_step * args.steps,
            "launches_per_step": {"kernels": kernels_per_step, "copies": launches_per_step - kernels_per_step},
            "roofline": roof,
        }
        if sustained is not None:
            line["sustained"] = sustained
        if route_ms is not None:
            line["routing"] = {"kernel": "route_kernel", "levels": m, "ms_per_sweep": min(route_ms[1:]),
                               "note": "MostAccurateFirst tables for the sweep's plans; outside the timed step"}
        if extras:
            line["tabulated"] = tab
            line["slo_sweep"] = slo_sweep
        bad = set((clocks or {}).get("reasons") or []) & {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
        if bad:
            line["clocks"]["rejected"] = sorted(bad)
    alloc.close()
    return line


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C4", choices=list(W.WORKLOAD_NAMES))
    ap.add_argument("--path", default="direct", choices=list(PATHS),
                    help="scoring kernel; the default is the per-pair arithmetic path the target is stated on, "
                         "`fastest` what the library picks by itself")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustain", type=float, default=2.0,
                    help="seconds of back-to-back solves for the sustained-clock leg (0: skip)")
    ap.add_argument("--no-extras", action="store_true",
                    help="only the timed step: skip the routing, fastest-path and SLO-sweep measurements that are "
                         "reported beside it (keeps a profiler's launch list to the step's own kernels)")
    ap.add_argument("--all", action="store_true",
                    help="one line per named workload, on the direct path and on the path the library picks")
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
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2

    if args.all:
        # a table of every named workload: the direct kernel and what the library picks by itself
        args.steps = min(args.steps, 20)
        for name in W.WORKLOAD_NAMES:
            for path in ("direct", "fastest"):
                line = run_one(B, torch, dist, args, name, path, dev, rank, world, local_rank, flush, extras=False)
                if rank == 0 and line is not None:
                    print(json.dumps(line), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return 0

    path = "auto" if args.variant_factors and args.path == "direct" else args.path
    line = run_one(B, torch, dist, args, args.workload, path, dev, rank, world, local_rank, flush,
                   extras=not args.no_extras)
    if rank == 0:
        if line is None:
            raise SystemExit("path %r does not apply to workload %s" % (args.path, args.workload))
        if world == 1 and not args.no_cpu_baseline:
            # measured issue rate of the fma forms: with one uniform source (the direct kernel's form and the
            # rate the nominal peak assumes) and with three register sources
            probe = fp64_probe()
            if probe and "fma_warp_inst_per_clk_per_sm" in probe:
                line["roofline"]["fp64_probe"] = probe["fma_warp_inst_per_clk_per_sm"]
            base = W.make_workload(args.workload)
            if args.variant_factors:
                frng = W.SplitMix64(99)
                base.variant_fanout_milli = [1000 + int(frng.randint(0, 8)) * 125 for _ in range(sum(base.n_variants))]
            cores = os.cpu_count() or 1
            v, desc, dt = oracle_sample(base, 12.0, cores)
            v1, desc1, dt1 = oracle_sample(base, 4.0, 1)
            line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": desc + " (%.1f s)" % dt,
                                    "one_core": {"value": v1, "sample": desc1 + " (%.1f s)" % dt1}}
        else:
            line["cpu_baseline"] = None
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
