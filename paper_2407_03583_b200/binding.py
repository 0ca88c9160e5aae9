"""Thin ctypes binding of ``libloki_alloc.so`` (argument marshalling only).

The functions carry the names of the C entry points declared in
``include/loki_alloc.h``; ``Allocator`` bundles a handle with the buffers a
caller usually wants.  PyTorch supplies device memory and streams.  There is no
CPU fallback: if the shared library is missing or no CUDA device is usable the
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Sequence

MAX_TASKS = 8
LOKI_OK = 0
LOKI_ERR_INVALID_ARG, LOKI_ERR_INVALID_GRAPH, LOKI_ERR_RANGE, LOKI_ERR_CUDA, LOKI_ERR_NOMEM = -1, -2, -3, -4, -5
LOKI_LEVEL_FEASIBLE, LOKI_LEVEL_INFEASIBLE, LOKI_LEVEL_BAD_DEMAND, LOKI_LEVEL_INTERNAL_ERROR = 0, 1, 2, 3
LOKI_PATH_AUTO, LOKI_PATH_GENERIC, LOKI_PATH_DIRECT, LOKI_PATH_HOISTED, LOKI_PATH_UNIFORM, LOKI_PATH_FASTEST = 0, 1, 2, 3, 4, 5
LOKI_PATH_PREFIX = 6
LOKI_PATH_SHARED = 7

_PKG = os.path.dirname(os.path.abspath(__file__))
# LOKI_ALLOC_LIB selects another build of the same library (the bounds-checked libloki_alloc_debug.so)
LIB_PATH = os.environ.get("LOKI_ALLOC_LIB") or os.path.join(_PKG, "libloki_alloc.so")

EXPORTS = (
    "loki_alloc_validate", "loki_alloc_plan_selfcheck", "loki_alloc_create", "loki_alloc_solve",
    "loki_alloc_solve_host", "loki_alloc_destroy", "loki_alloc_set_path", "loki_alloc_set_timing",
    "loki_alloc_last_score_ms", "loki_alloc_num_candidates", "loki_alloc_get_info",
    "loki_alloc_strerror", "loki_alloc_config_size", "loki_alloc_solve_static", "loki_alloc_set_slo",
    "loki_alloc_route", "loki_alloc_solve_slos", "loki_alloc_last_fma_count",
    "loki_alloc_debug_status",
)


class LokiError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s: %s (code %d)" % (what, loki_alloc_strerror(code), code))
        self.code = code


class loki_alloc_desc_t(ctypes.Structure):
    _fields_ = [
        ("n_tasks", ctypes.c_int32),
        ("parent", ctypes.POINTER(ctypes.c_int32)),
        ("fanout_milli", ctypes.POINTER(ctypes.c_int32)),
        ("n_variants", ctypes.POINTER(ctypes.c_int32)),
        ("n_batches", ctypes.c_int32),
        ("batch_sizes", ctypes.POINTER(ctypes.c_int32)),
        ("accuracy", ctypes.POINTER(ctypes.c_double)),
        ("latency_us", ctypes.POINTER(ctypes.c_int64)),
        ("slo_us", ctypes.c_int64),
        ("comm_us", ctypes.c_int64),
        ("cluster_size", ctypes.c_int32),
        ("split_mode", ctypes.c_int32),
        ("max_demand_mqps", ctypes.c_int64),
        ("max_levels", ctypes.c_int32),
        ("variant_fanout_milli", ctypes.POINTER(ctypes.c_int32)),
    ]


class loki_config_t(ctypes.Structure):
    _fields_ = [
        ("cand_index", ctypes.c_int64),
        ("accuracy", ctypes.c_double),
        ("total_workers", ctypes.c_int32),
        ("status", ctypes.c_int32),
        ("variant", (ctypes.c_int32 * 2) * MAX_TASKS),
        ("batch", (ctypes.c_int32 * 2) * MAX_TASKS),
        ("workers", (ctypes.c_int32 * 2) * MAX_TASKS),
        ("split_k", ctypes.c_int32 * MAX_TASKS),
        ("latency_budget_us", ctypes.c_int64 * MAX_TASKS),
    ]


class loki_alloc_info_t(ctypes.Structure):
    _fields_ = [
        ("n_candidates", ctypes.c_int64),
        ("path_auto", ctypes.c_int32),
        ("path_current", ctypes.c_int32),
        ("direct_ok", ctypes.c_int32),
        ("direct_level_tile", ctypes.c_int32),
        ("n_blocks", ctypes.c_int32),
        ("n_launches_last", ctypes.c_int32),
        ("hoisted_ok", ctypes.c_int32),
        ("path_last", ctypes.c_int32),
        ("uniform_ok", ctypes.c_int32),
        ("level_tile_last", ctypes.c_int32),
        ("scratch_bytes", ctypes.c_int64),
        ("table_bytes", ctypes.c_int64),
    ]


LOKI_ROUTE_OK, LOKI_ROUTE_NO_PLAN, LOKI_ROUTE_TABLE_FULL = 0, 1, 2


class loki_route_header_t(ctypes.Structure):
    _fields_ = [("status", ctypes.c_int32), ("n_workers", ctypes.c_int32), ("n_entries", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("unrouted_qps", ctypes.c_double)]


class loki_route_worker_t(ctypes.Structure):
    _fields_ = [("task", ctypes.c_int32), ("variant", ctypes.c_int32), ("batch", ctypes.c_int32),
                ("reserved", ctypes.c_int32), ("capacity_qps", ctypes.c_double),
                ("incoming_qps", ctypes.c_double), ("leftover_qps", ctypes.c_double)]


class loki_route_entry_t(ctypes.Structure):
    _fields_ = [("src_worker", ctypes.c_int32), ("dst_worker", ctypes.c_int32), ("probability", ctypes.c_double)]


CONFIG_SIZE = ctypes.sizeof(loki_config_t)
_lib = None


def load_library() -> ctypes.CDLL:
    """Load ``libloki_alloc.so`` (built in-tree by ``paper_2407_03583_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise OSError("libloki_alloc.so is not built: run `python -m paper_2407_03583_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int64)
    lib.loki_alloc_validate.argtypes = [ctypes.POINTER(loki_alloc_desc_t)]
    lib.loki_alloc_plan_selfcheck.argtypes = [ctypes.POINTER(loki_alloc_desc_t), ctypes.POINTER(i32), i64p, i64p]
    lib.loki_alloc_create.argtypes = [ctypes.POINTER(loki_alloc_desc_t), ctypes.POINTER(vp)]
    lib.loki_alloc_solve.argtypes = [vp, vp, i32, vp, vp]
    lib.loki_alloc_solve_host.argtypes = [vp, vp, i32, vp, vp]
    lib.loki_alloc_solve_static.argtypes = [vp, vp, i32, vp, vp]
    lib.loki_alloc_solve_slos.argtypes = [vp, vp, i32, i64p, i32, vp, vp]
    lib.loki_alloc_route.argtypes = [vp, vp, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.loki_alloc_destroy.argtypes = [vp]
    lib.loki_alloc_set_path.argtypes = [vp, i32]
    lib.loki_alloc_set_timing.argtypes = [vp, i32]
    lib.loki_alloc_set_slo.argtypes = [vp, ctypes.c_int64, ctypes.c_int64]
    lib.loki_alloc_last_score_ms.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(i32)]
    lib.loki_alloc_last_fma_count.argtypes = [vp, i64p]
    lib.loki_alloc_debug_status.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_uint32),
                                            ctypes.POINTER(ctypes.c_uint32)]
    lib.loki_alloc_num_candidates.argtypes = [vp, i64p]
    lib.loki_alloc_get_info.argtypes = [vp, ctypes.POINTER(loki_alloc_info_t)]
    lib.loki_alloc_strerror.argtypes = [ctypes.c_int]
    lib.loki_alloc_strerror.restype = ctypes.c_char_p
    lib.loki_alloc_config_size.restype = ctypes.c_int32
    for name in EXPORTS:
        getattr(lib, name)
    if lib.loki_alloc_config_size() != CONFIG_SIZE:
        raise OSError("loki_config_t layout mismatch between the binding and the library")
    _lib = lib
    return lib


def _arr(ctype, values: Sequence):
    return (ctype * len(values))(*values)


def make_desc(w, max_levels: int | None = None):
    """``loki_alloc_desc_t`` for a workload-like object; returns ``(desc, keepalive)``."""
    keep = [
        _arr(ctypes.c_int32, w.parent), _arr(ctypes.c_int32, w.fanout_milli),
        _arr(ctypes.c_int32, w.n_variants), _arr(ctypes.c_int32, w.batch_sizes),
        _arr(ctypes.c_double, w.accuracy), _arr(ctypes.c_int64, w.latency_us),
    ]
    d = loki_alloc_desc_t()
    d.n_tasks = len(w.parent)
    d.parent = ctypes.cast(keep[0], ctypes.POINTER(ctypes.c_int32))
    d.fanout_milli = ctypes.cast(keep[1], ctypes.POINTER(ctypes.c_int32))
    d.n_variants = ctypes.cast(keep[2], ctypes.POINTER(ctypes.c_int32))
    d.n_batches = len(w.batch_sizes)
    d.batch_sizes = ctypes.cast(keep[3], ctypes.POINTER(ctypes.c_int32))
    d.accuracy = ctypes.cast(keep[4], ctypes.POINTER(ctypes.c_double))
    d.latency_us = ctypes.cast(keep[5], ctypes.POINTER(ctypes.c_int64))
    d.slo_us = w.slo_us
    d.comm_us = w.comm_us
    d.cluster_size = w.cluster_size
    d.split_mode = w.split_mode
    d.max_demand_mqps = w.max_demand_mqps
    d.max_levels = max_levels if max_levels is not None else max(1, len(w.demand_mqps))
    vfan = getattr(w, "variant_fanout_milli", None)
    if vfan is not None:
        keep.append(_arr(ctypes.c_int32, vfan))
        d.variant_fanout_milli = ctypes.cast(keep[-1], ctypes.POINTER(ctypes.c_int32))
    return d, keep


# ---- one function per C entry point -----------------------------------------

def loki_alloc_strerror(code: int) -> str:
    return load_library().loki_alloc_strerror(code).decode()


def loki_alloc_validate(desc: loki_alloc_desc_t) -> int:
    return load_library().loki_alloc_validate(ctypes.byref(desc))


def loki_alloc_plan_selfcheck(desc: loki_alloc_desc_t):
    """Returns ``(rc, direct_ok, n_checked, n_mismatch)``."""
    ok, nc, nm = ctypes.c_int32(), ctypes.c_int64(), ctypes.c_int64()
    rc = load_library().loki_alloc_plan_selfcheck(ctypes.byref(desc), ctypes.byref(ok),
                                                  ctypes.byref(nc), ctypes.byref(nm))
    return rc, ok.value, nc.value, nm.value


def loki_alloc_create(desc: loki_alloc_desc_t) -> ctypes.c_void_p:
    h = ctypes.c_void_p()
    rc = load_library().loki_alloc_create(ctypes.byref(desc), ctypes.byref(h))
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_create")
    return h


def loki_alloc_solve(h, d_demand_ptr: int, n_levels: int, stream_ptr: int, d_out_ptr: int) -> None:
    rc = load_library().loki_alloc_solve(h, d_demand_ptr, n_levels, stream_ptr, d_out_ptr)
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_solve")


def loki_alloc_solve_host(h, h_demand_ptr: int, n_levels: int, stream_ptr: int, h_out_ptr: int) -> None:
    rc = load_library().loki_alloc_solve_host(h, h_demand_ptr, n_levels, stream_ptr, h_out_ptr)
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_solve_host")


def loki_alloc_solve_static(h, d_demand_ptr: int, n_levels: int, stream_ptr: int, d_out_ptr: int) -> int:
    """Allocation-free solve (at most 64 levels); returns the C return code."""
    return load_library().loki_alloc_solve_static(h, d_demand_ptr, n_levels, stream_ptr, d_out_ptr)


def loki_alloc_solve_slos(h, d_demand_ptr: int, n_levels: int, slos_us: Sequence[int], stream_ptr: int,
                          d_out_ptr: int) -> None:
    arr = _arr(ctypes.c_int64, list(slos_us))
    rc = load_library().loki_alloc_solve_slos(h, d_demand_ptr, n_levels, arr, len(slos_us), stream_ptr, d_out_ptr)
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_solve_slos")


def loki_alloc_route(h, d_demand_ptr: int, d_plans_ptr: int, n_levels: int, max_workers: int,
                     max_entries: int, stream_ptr: int, d_headers_ptr: int, d_workers_ptr: int,
                     d_entries_ptr: int) -> None:
    rc = load_library().loki_alloc_route(h, d_demand_ptr, d_plans_ptr, n_levels, max_workers, max_entries,
                                         stream_ptr, d_headers_ptr, d_workers_ptr, d_entries_ptr)
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_route")


def loki_alloc_destroy(h) -> None:
    load_library().loki_alloc_destroy(h)


def loki_alloc_set_path(h, path: int) -> None:
    rc = load_library().loki_alloc_set_path(h, path)
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_set_path")


def loki_alloc_set_slo(h, slo_us: int, comm_us: int = 0) -> None:
    rc = load_library().loki_alloc_set_slo(h, slo_us, comm_us)
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_set_slo")


def loki_alloc_set_timing(h, enable: bool) -> None:
    rc = load_library().loki_alloc_set_timing(h, 1 if enable else 0)
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_set_timing")


def loki_alloc_last_score_ms(h):
    """Returns ``(total_ms, n_launches)`` of the last solve's scoring launches."""
    ms, n = ctypes.c_float(), ctypes.c_int32()
    rc = load_library().loki_alloc_last_score_ms(h, ctypes.byref(ms), ctypes.byref(n))
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_last_score_ms")
    return ms.value, n.value


def loki_alloc_last_fma_count(h) -> int:
    """FP64 fused multiply-adds the DIRECT kernel executed in the last solve (0 for other kernels)."""
    n = ctypes.c_int64()
    rc = load_library().loki_alloc_last_fma_count(h, ctypes.byref(n))
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_last_fma_count")
    return n.value


def loki_alloc_debug_status(h):
    """Returns ``(checked_build, site_mask, n_violations)`` of the bounds-checked build's status words."""
    cb, mask, n = ctypes.c_int32(), ctypes.c_uint32(), ctypes.c_uint32()
    rc = load_library().loki_alloc_debug_status(h, ctypes.byref(cb), ctypes.byref(mask), ctypes.byref(n))
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_debug_status")
    return cb.value, mask.value, n.value


def loki_alloc_num_candidates(h) -> int:
    n = ctypes.c_int64()
    rc = load_library().loki_alloc_num_candidates(h, ctypes.byref(n))
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_num_candidates")
    return n.value


def loki_alloc_get_info(h) -> loki_alloc_info_t:
    info = loki_alloc_info_t()
    rc = load_library().loki_alloc_get_info(h, ctypes.byref(info))
    if rc != LOKI_OK:
        raise LokiError(rc, "loki_alloc_get_info")
    return info


def config_to_dict(c: loki_config_t, n_tasks: int) -> dict:
    return {
        "cand_index": int(c.cand_index), "accuracy": float(c.accuracy),
        "total_workers": int(c.total_workers), "status": int(c.status),
        "variant": [[int(c.variant[i][s]) for s in range(2)] for i in range(n_tasks)],
        "batch": [[int(c.batch[i][s]) for s in range(2)] for i in range(n_tasks)],
        "workers": [[int(c.workers[i][s]) for s in range(2)] for i in range(n_tasks)],
        "split_k": [int(c.split_k[i]) for i in range(n_tasks)],
        "latency_budget_us": [int(c.latency_budget_us[i]) for i in range(n_tasks)],
    }


class Allocator:
    """A handle plus device and pinned host buffers sized for ``max_levels`` levels."""

    def __init__(self, w, max_levels: int | None = None, device: str = "cuda:0"):
        import torch
        if not torch.cuda.is_available():
            raise RuntimeError("libloki_alloc needs a CUDA device; there is no CPU fallback")
        self.torch = torch
        self.device = torch.device(device)
        self.n_tasks = len(w.parent)
        desc, self._keep = make_desc(w, max_levels)
        self.max_levels = desc.max_levels
        self.handle = None
        with torch.cuda.device(self.device):
            self.handle = loki_alloc_create(desc)
        self.d_demand = torch.empty(self.max_levels, dtype=torch.int64, device=self.device)
        self.d_out = torch.empty(self.max_levels * CONFIG_SIZE, dtype=torch.uint8, device=self.device)
        self.h_demand = torch.empty(self.max_levels, dtype=torch.int64).pin_memory()
        self.h_out = torch.empty(self.max_levels * CONFIG_SIZE, dtype=torch.uint8).pin_memory()

    def close(self):
        if self.handle is not None:
            loki_alloc_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_path(self, path: int):
        loki_alloc_set_path(self.handle, path)

    def info(self) -> loki_alloc_info_t:
        return loki_alloc_get_info(self.handle)

    def num_candidates(self) -> int:
        return loki_alloc_num_candidates(self.handle)

    def upload(self, demand_mqps: Sequence[int]) -> int:
        n = len(demand_mqps)
        self.h_demand[:n] = self.torch.tensor(list(demand_mqps), dtype=self.torch.int64)
        self.d_demand[:n].copy_(self.h_demand[:n], non_blocking=True)
        return n

    def solve_device(self, n_levels: int) -> None:
        """Enqueue one solve on torch's current stream over ``d_demand[:n_levels]``."""
        with self.torch.cuda.device(self.device):
            stream = self.torch.cuda.current_stream(self.device).cuda_stream
            loki_alloc_solve(self.handle, self.d_demand.data_ptr(), n_levels, stream,
                             self.d_out.data_ptr())

    def solve_host(self, n_levels: int) -> None:
        """``h_demand[:n_levels]`` -> plans in ``h_out``; copies in and out, synchronises."""
        with self.torch.cuda.device(self.device):
            stream = self.torch.cuda.current_stream(self.device).cuda_stream
            loki_alloc_solve_host(self.handle, self.h_demand.data_ptr(), n_levels, stream,
                                  self.h_out.data_ptr())

    def read_device(self, n_levels: int):
        self.torch.cuda.synchronize(self.device)
        raw = self.d_out[: n_levels * CONFIG_SIZE].cpu().numpy().tobytes()
        return _parse(raw, n_levels)

    def read_host(self, n_levels: int):
        raw = self.h_out[: n_levels * CONFIG_SIZE].numpy().tobytes()
        return _parse(raw, n_levels)

    def solve(self, demand_mqps: Sequence[int]):
        """Convenience: upload, solve on the device, read the plans back."""
        n = self.upload(demand_mqps)
        self.solve_device(n)
        return self.read_device(n)


def route_device(alloc: "Allocator", n_levels: int, max_workers: int, max_entries: int):
    """Marshalling helper: runs loki_alloc_route on the plans in ``alloc.d_out`` (demands in
    ``alloc.d_demand``) and returns per level ``(header, workers, entries)`` as ctypes values."""
    torch = alloc.torch
    hs, ws, es = (ctypes.sizeof(loki_route_header_t), ctypes.sizeof(loki_route_worker_t),
                  ctypes.sizeof(loki_route_entry_t))
    d_h = torch.empty(n_levels * hs, dtype=torch.uint8, device=alloc.device)
    d_w = torch.empty(n_levels * max_workers * ws, dtype=torch.uint8, device=alloc.device)
    d_e = torch.empty(n_levels * max_entries * es, dtype=torch.uint8, device=alloc.device)
    with torch.cuda.device(alloc.device):
        stream = torch.cuda.current_stream(alloc.device).cuda_stream
        loki_alloc_route(alloc.handle, alloc.d_demand.data_ptr(), alloc.d_out.data_ptr(), n_levels,
                         max_workers, max_entries, stream, d_h.data_ptr(), d_w.data_ptr(), d_e.data_ptr())
    torch.cuda.synchronize(alloc.device)
    H = (loki_route_header_t * n_levels).from_buffer_copy(d_h.cpu().numpy().tobytes())
    Wk = (loki_route_worker_t * (n_levels * max_workers)).from_buffer_copy(d_w.cpu().numpy().tobytes())
    En = (loki_route_entry_t * (n_levels * max_entries)).from_buffer_copy(d_e.cpu().numpy().tobytes())
    out = []
    for l in range(n_levels):
        h = H[l]
        out.append((h, [Wk[l * max_workers + k] for k in range(min(h.n_workers, max_workers))],
                    [En[l * max_entries + k] for k in range(h.n_entries)]))
    return out


def _parse(raw: bytes, n_levels: int):
    arr = (loki_config_t * n_levels).from_buffer_copy(raw)
    return [arr[i] for i in range(n_levels)]
