"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every symbol the header declares, validates its inputs, and its planner's
fixed-point worker arithmetic is exact where it claims to be."""
import ctypes
import os
import re

import pytest

from paper_2407_03583_b200 import binding as B
from paper_2407_03583_b200 import workloads as W
from helpers import h1_workload

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = B.load_library()
    header = open(os.path.join(ROOT, "include", "loki_alloc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(loki_alloc_[a-z_0-9]+)\s*\(", header))
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert getattr(lib, name) is not None, name
    assert declared == set(B.EXPORTS)
    assert lib.loki_alloc_config_size() == ctypes.sizeof(B.loki_config_t) == 312


def test_binding_constants_match_the_header():
    # every LOKI_PATH_* / LOKI_ERR_* / LOKI_LEVEL_* enumerator of the header has the same value in the binding
    header = open(os.path.join(ROOT, "include", "loki_alloc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    found = dict(re.findall(r"\b(LOKI_(?:PATH|ERR|LEVEL|ROUTE)_[A-Z_0-9]+)\s*=\s*(-?\d+)", header))
    assert "LOKI_PATH_PREFIX" in found and "LOKI_PATH_AUTO" in found
    for name, value in found.items():
        assert getattr(B, name) == int(value), name


def test_checked_build_exports_the_same_interface():
    # the bounds-checked build of the same sources (built by __graft_entry__.build) is a drop-in replacement
    from paper_2407_03583_b200 import build as lib_build
    path = lib_build.DEBUG_LIB_PATH
    if not os.path.exists(path):
        pytest.skip("libloki_alloc_debug.so is not built")
    lib = ctypes.CDLL(path)
    for name in B.EXPORTS:
        assert getattr(lib, name) is not None, name
    lib.loki_alloc_config_size.restype = ctypes.c_int32
    assert lib.loki_alloc_config_size() == ctypes.sizeof(B.loki_config_t)


def test_strerror_is_total():
    for code in range(-7, 2):
        assert B.loki_alloc_strerror(code)


def _desc(w, **kw):
    d, keep = B.make_desc(w)
    for k, v in kw.items():
        setattr(d, k, v)
    return d, keep


def test_validate_accepts_the_named_workloads():
    for name in W.WORKLOAD_NAMES:
        d, _k = _desc(W.make_workload(name))
        assert B.loki_alloc_validate(d) == B.LOKI_OK


@pytest.mark.parametrize("mutate,code", [
    (lambda w: setattr(w, "parent", [-1, 1]), B.LOKI_ERR_INVALID_GRAPH),       # parent >= i
    (lambda w: setattr(w, "parent", [0, 0]), B.LOKI_ERR_INVALID_GRAPH),        # no root
    (lambda w: setattr(w, "parent", [-1, -1]), B.LOKI_ERR_INVALID_GRAPH),      # two roots
    (lambda w: setattr(w, "batch_sizes", [1, 2, 2, 8]), B.LOKI_ERR_INVALID_ARG),
    (lambda w: setattr(w, "batch_sizes", [0, 2, 4, 8]), B.LOKI_ERR_INVALID_ARG),
    (lambda w: w.accuracy.__setitem__(0, 0.0), B.LOKI_ERR_INVALID_ARG),
    (lambda w: w.accuracy.__setitem__(1, 1.5), B.LOKI_ERR_INVALID_ARG),
    (lambda w: w.accuracy.__setitem__(1, float("nan")), B.LOKI_ERR_INVALID_ARG),
    (lambda w: w.latency_us.__setitem__(3, 0), B.LOKI_ERR_INVALID_ARG),
    (lambda w: w.fanout_milli.__setitem__(1, 0), B.LOKI_ERR_INVALID_ARG),
    (lambda w: setattr(w, "slo_us", -1), B.LOKI_ERR_INVALID_ARG),
    (lambda w: setattr(w, "cluster_size", 1 << 24), B.LOKI_ERR_INVALID_ARG),
    (lambda w: setattr(w, "split_mode", 2), B.LOKI_ERR_INVALID_ARG),
    (lambda w: setattr(w, "max_demand_mqps", 1 << 61), B.LOKI_ERR_RANGE),      # overflow proof
])
def test_validate_rejects(mutate, code):
    w = W.make_workload("C1")
    mutate(w)
    d, _k = _desc(w)
    assert B.loki_alloc_validate(d) == code


def test_validate_rejects_counts_and_nulls():
    w = W.make_workload("C1")
    d, _k = _desc(w, n_tasks=0)
    assert B.loki_alloc_validate(d) == B.LOKI_ERR_INVALID_ARG
    d, _k = _desc(w, n_tasks=9)
    assert B.loki_alloc_validate(d) == B.LOKI_ERR_INVALID_ARG
    d, _k = _desc(w, max_levels=0)
    assert B.loki_alloc_validate(d) == B.LOKI_ERR_INVALID_ARG
    d, _k = _desc(w)
    d.accuracy = ctypes.POINTER(ctypes.c_double)()
    assert B.loki_alloc_validate(d) == B.LOKI_ERR_INVALID_ARG
    assert B.load_library().loki_alloc_validate(None) == B.LOKI_ERR_INVALID_ARG


def test_search_space_limit():
    # 8 tasks x 40 variants x 7 batches = 280^8 candidates: far beyond 2^40
    w = W.random_workload(1, n_tasks=8, n_variants=40, batch_sizes=[1, 2, 4, 8, 16, 32, 64], chain=True)
    d, _k = _desc(w)
    assert B.loki_alloc_validate(d) == B.LOKI_ERR_RANGE


def test_entry_points_reject_null_handles_without_a_gpu():
    lib = B.load_library()
    assert lib.loki_alloc_destroy(None) == B.LOKI_OK
    assert lib.loki_alloc_solve(None, None, 1, None, None) == B.LOKI_ERR_INVALID_ARG
    assert lib.loki_alloc_solve_host(None, None, 1, None, None) == B.LOKI_ERR_INVALID_ARG
    assert lib.loki_alloc_set_path(None, 0) == B.LOKI_ERR_INVALID_ARG
    assert lib.loki_alloc_set_timing(None, 1) == B.LOKI_ERR_INVALID_ARG
    assert lib.loki_alloc_get_info(None, None) == B.LOKI_ERR_INVALID_ARG
    assert lib.loki_alloc_create(None, None) == B.LOKI_ERR_INVALID_ARG


@pytest.mark.parametrize("name", W.WORKLOAD_NAMES)
def test_direct_path_arithmetic_is_exact_on_named_workloads(name):
    d, _k = _desc(W.make_workload(name))
    rc, ok, n_checked, n_bad = B.loki_alloc_plan_selfcheck(d)
    assert rc == B.LOKI_OK and ok == 1
    assert n_checked > 100 and n_bad == 0


def test_direct_path_arithmetic_on_random_and_awkward_problems():
    n_direct = 0
    for seed in range(60):
        w = W.random_workload(seed, n_tasks=1 + seed % 4, n_variants=2 + seed % 3,
                              batch_sizes=[1, 3, 8] if seed % 2 else [2, 5], split_mode=int(seed % 3 == 0),
                              fan_fractional=seed % 4 == 1)
        w.max_demand_mqps = 10 ** (4 + seed % 8)
        d, _k = _desc(w)
        rc, ok, n_checked, n_bad = B.loki_alloc_plan_selfcheck(d)
        assert rc == B.LOKI_OK and n_bad == 0
        n_direct += ok
    assert n_direct > 30
    # exact-quotient demands of the hand-worked example
    d, _k = _desc(h1_workload(1))
    rc, ok, n_checked, n_bad = B.loki_alloc_plan_selfcheck(d)
    assert (rc, ok, n_bad) == (0, 1, 0)


def test_direct_path_declines_when_its_conditions_fail():
    # latencies near 12 days at batch 1 make lat / (b * 1e9) >= 1: no 64-bit reciprocal
    w = W.make_workload("C1")
    w.latency_us = [min(x * 10 ** 8, 1 << 40) for x in w.latency_us]
    w.slo_us = 1 << 59
    w.max_demand_mqps = 1000
    d, _k = _desc(w)
    rc, ok, _n, n_bad = B.loki_alloc_plan_selfcheck(d)
    assert rc == B.LOKI_OK and ok == 0 and n_bad == 0


def test_variant_factors_are_validated_and_switch_off_the_direct_path():
    w = W.make_workload("C2", v=3, n_levels=8)
    w.variant_fanout_milli = [1000] * 9
    d, _k = _desc(w)
    assert B.loki_alloc_validate(d) == B.LOKI_OK
    assert B.loki_alloc_plan_selfcheck(d)[1] == 1          # all factors 1: direct path still applies
    w.variant_fanout_milli = [800, 1000, 1700] * 3
    d, _k = _desc(w)
    assert B.loki_alloc_validate(d) == B.LOKI_OK
    assert B.loki_alloc_plan_selfcheck(d)[:2] == (B.LOKI_OK, 0)
    w.variant_fanout_milli = [0] + [1000] * 8
    d, _k = _desc(w)
    assert B.loki_alloc_validate(d) == B.LOKI_ERR_INVALID_ARG


def test_stage_demand_ratios_of_the_root_first_kernel_are_exact():
    """With per-variant factors (Eq. 1) a child's stage demand is ceil(dem * ratio), ratio = edge factor x
    option factor, possibly above 1; the planner's one-fma form is replayed in integers at the demands
    where that ceiling steps."""
    n_with_ratios = 0
    for seed in range(40):
        w = W.random_workload(seed, n_tasks=2 + seed % 3, n_variants=2 + seed % 3,
                              batch_sizes=[1, 3, 8] if seed % 2 else [2, 5], split_mode=int(seed % 3 == 0),
                              fan_fractional=seed % 4 == 1)
        w.max_demand_mqps = 10 ** (4 + seed % 6)
        d, _k = _desc(w)
        rc, _ok, n_plain, n_bad = B.loki_alloc_plan_selfcheck(d)
        assert rc == B.LOKI_OK and n_bad == 0
        rng = W.SplitMix64(1000 + seed)
        awkward = [333, 1001, 2999, 7, 1 << 12, 999, 1700, 125]
        w.variant_fanout_milli = [awkward[int(rng.randint(0, len(awkward) - 1))] for _ in range(sum(w.n_variants))]
        d, _k = _desc(w)
        rc, ok, n_checked, n_bad = B.loki_alloc_plan_selfcheck(d)
        if rc == B.LOKI_ERR_RANGE:          # the factors grow a stage demand out of the 64-bit range
            continue
        assert (rc, ok, n_bad) == (B.LOKI_OK, 0, 0)
        n_with_ratios += n_checked >= n_plain > 100
    assert n_with_ratios > 20
