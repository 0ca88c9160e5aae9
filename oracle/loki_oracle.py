"""ctypes front end of ``loki_oracle.cpp`` (test infrastructure only).

``build()`` compiles the C++ file with ``g++ -O2 -ffp-contract=off`` into
``oracle/libloki_oracle.so``; ``solve()`` runs the enumerator on host arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "loki_oracle.cpp")
_LIB = os.path.join(_HERE, "libloki_oracle.so")
MAX_TASKS = 8


class OracleResult(ctypes.Structure):
    _fields_ = [
        ("cand_index", ctypes.c_int64),
        ("accuracy", ctypes.c_double),
        ("total_workers", ctypes.c_int64),
        ("status", ctypes.c_int32),
        ("pad", ctypes.c_int32),
        ("variant", (ctypes.c_int32 * 2) * MAX_TASKS),
        ("batch", (ctypes.c_int32 * 2) * MAX_TASKS),
        ("workers", (ctypes.c_int64 * 2) * MAX_TASKS),
        ("split_k", ctypes.c_int32 * MAX_TASKS),
        ("latency_budget_us", ctypes.c_int64 * MAX_TASKS),
        ("stage_demand_mqps", ctypes.c_int64 * MAX_TASKS),
    ]


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than the source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
           "-o", tmp, _SRC]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.loki_oracle_result_size.restype = ctypes.c_int
        assert lib.loki_oracle_result_size() == ctypes.sizeof(OracleResult)
        lib.loki_oracle_solve_range.restype = ctypes.c_int
        _lib = lib
    return _lib


def _arr(ctype, values: Sequence):
    return (ctype * len(values))(*values)


def solve(w, demand_mqps: Sequence[int] | None = None, n_threads: int = 1,
          cand_range: tuple | None = None) -> List[OracleResult]:
    """Run the oracle on workload ``w`` (any object with the fields of
    ``workloads.Workload``).  ``demand_mqps`` overrides ``w.demand_mqps``;
    ``cand_range=(begin, end)`` restricts the search to those candidate indices."""
    lib = _load()
    dem = list(w.demand_mqps if demand_mqps is None else demand_mqps)
    out = (OracleResult * max(1, len(dem)))()
    cb, ce = (0, -1) if cand_range is None else cand_range
    rc = lib.loki_oracle_solve_range(
        ctypes.c_int(w.n_tasks), _arr(ctypes.c_int32, w.parent), _arr(ctypes.c_int32, w.fanout_milli),
        _arr(ctypes.c_int32, w.n_variants), ctypes.c_int(len(w.batch_sizes)),
        _arr(ctypes.c_int32, w.batch_sizes), _arr(ctypes.c_double, w.accuracy),
        _arr(ctypes.c_int64, w.latency_us),
        None if getattr(w, "variant_fanout_milli", None) is None else _arr(ctypes.c_int32, w.variant_fanout_milli),
        ctypes.c_int64(w.slo_us), ctypes.c_int64(w.comm_us),
        ctypes.c_int32(w.cluster_size), ctypes.c_int32(w.split_mode),
        ctypes.c_int64(w.max_demand_mqps), _arr(ctypes.c_int64, dem), ctypes.c_int(len(dem)),
        ctypes.c_int(n_threads), ctypes.c_int64(cb), ctypes.c_int64(ce), out)
    if rc != 0:
        raise ValueError("oracle rejected the input (code %d)" % rc)
    return [out[i] for i in range(len(dem))]


def result_to_dict(r: OracleResult, n_tasks: int) -> dict:
    """Plain-Python view of one level's result (only the first ``n_tasks`` rows)."""
    return {
        "cand_index": int(r.cand_index),
        "accuracy": float(r.accuracy),
        "total_workers": int(r.total_workers),
        "status": int(r.status),
        "variant": [[int(r.variant[i][s]) for s in range(2)] for i in range(n_tasks)],
        "batch": [[int(r.batch[i][s]) for s in range(2)] for i in range(n_tasks)],
        "workers": [[int(r.workers[i][s]) for s in range(2)] for i in range(n_tasks)],
        "split_k": [int(r.split_k[i]) for i in range(n_tasks)],
        "latency_budget_us": [int(r.latency_budget_us[i]) for i in range(n_tasks)],
        "stage_demand_mqps": [int(r.stage_demand_mqps[i]) for i in range(n_tasks)],
    }
