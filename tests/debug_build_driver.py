"""Driver of tests/test_gpu_debug_build.py: runs in a process of its own with LOKI_ALLOC_LIB
pointing at the bounds-checked build, solves small named workloads and random problems on every
scoring kernel (plus an SLO sweep and the allocation-free entry point), compares every plan with
the CPU oracle and prints one JSON line with what the checked build recorded."""
import json
import os
import random
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

import torch  # noqa: E402

import oracle  # noqa: E402
from paper_2407_03583_b200 import binding as B  # noqa: E402
from paper_2407_03583_b200 import workloads as W  # noqa: E402

PATHS = [B.LOKI_PATH_GENERIC, B.LOKI_PATH_DIRECT, B.LOKI_PATH_HOISTED, B.LOKI_PATH_UNIFORM, B.LOKI_PATH_PREFIX,
         B.LOKI_PATH_SHARED]


def same(w, got, ref):
    for g, r in zip(got, ref):
        o = oracle.result_to_dict(r, w.n_tasks)
        if (g.status, g.cand_index, g.total_workers, g.accuracy) != (o["status"], o["cand_index"], o["total_workers"], o["accuracy"]):
            return False
    return True


def main():
    out = {"checked_build": None, "site_mask": 0, "n_violations": 0, "n_solves": 0, "n_mismatch": 0}
    cases = [W.make_workload(n, v=v, n_levels=m) for n, v, m in
             (("C1", None, None), ("C2", 5, 300), ("C3", 3, 140), ("C4", 3, 64), ("C5", 2, 70), ("SM", None, 200))]
    rnd = random.Random(5)
    for seed in range(16):
        T = rnd.randint(1, 5)
        split = seed % 4 == 0
        cases.append(W.random_workload(9000 + seed, n_tasks=min(T, 3) if split else T,
                                       n_variants=rnd.randint(1, 3), batch_sizes=[1, 2, 8][: rnd.randint(1, 3)],
                                       split_mode=int(split), n_levels=[7, 64, 150, 300][seed % 4],
                                       fan_fractional=seed % 2 == 1, variant_fan=seed % 5 == 2))
    for w in cases:
        ref = oracle.solve(w, n_threads=os.cpu_count() or 1)
        a = B.Allocator(w)
        try:
            for path in PATHS:
                try:
                    a.set_path(path)
                except B.LokiError:
                    continue
                out["n_solves"] += 1
                out["n_mismatch"] += 0 if same(w, a.solve(w.demand_mqps), ref) else 1
            # the allocation-free entry point and an SLO sweep on the path the library picks
            n = a.upload(w.demand_mqps[:64])
            torch.cuda.synchronize()
            assert B.loki_alloc_solve_static(a.handle, a.d_demand.data_ptr(), n, torch.cuda.current_stream().cuda_stream,
                                             a.d_out.data_ptr()) == B.LOKI_OK
            out["n_solves"] += 1
            out["n_mismatch"] += 0 if same(w, a.read_device(n), ref[:n]) else 1
            a.set_path(B.LOKI_PATH_FASTEST)
            n = a.upload(w.demand_mqps)
            slos = [w.slo_us // 2, w.slo_us, 2 * w.slo_us]
            d_out = torch.empty(len(slos) * n * B.CONFIG_SIZE, dtype=torch.uint8, device=a.device)
            B.loki_alloc_solve_slos(a.handle, a.d_demand.data_ptr(), n, slos, torch.cuda.current_stream().cuda_stream,
                                    d_out.data_ptr())
            torch.cuda.synchronize()
            arr = (B.loki_config_t * (len(slos) * n)).from_buffer_copy(d_out.cpu().numpy().tobytes())
            for s, slo in enumerate(slos):
                ws = w.with_demands(w.demand_mqps)
                ws.slo_us = slo
                out["n_solves"] += 1
                out["n_mismatch"] += 0 if same(ws, [arr[s * n + l] for l in range(n)],
                                               oracle.solve(ws, n_threads=os.cpu_count() or 1)) else 1
            cb, mask, nv = B.loki_alloc_debug_status(a.handle)
            out["checked_build"] = cb
            out["site_mask"] |= mask
            out["n_violations"] += nv
        finally:
            a.close()
    print(json.dumps(out))


if __name__ == "__main__":
    main()
