"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times (direct path, all levels in one solve).  Where the oracle cannot finish
all levels in seconds it computes a sample of levels one by one; properties
that hold at any size are checked on every level."""
import os

import pytest

import oracle
from helpers import check_plan
from paper_2407_03583_b200 import binding as B
from paper_2407_03583_b200 import workloads as W
from test_gpu_parity import assert_same

pytestmark = pytest.mark.gpu
NCPU = max(1, os.cpu_count() or 1)


def _solve_all(w):
    a = B.Allocator(w)
    try:
        assert a.info().direct_ok == 1 and a.info().path_current == B.LOKI_PATH_DIRECT
        return [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
    finally:
        a.close()


def _sweep_invariants(w, got):
    order = sorted(range(w.n_levels), key=lambda j: w.demand_mqps[j])
    prev_acc, infeasible_seen = None, False
    for j in order:
        g = got[j]
        assert g["status"] in (0, 1)
        if g["status"] == 1:
            infeasible_seen = True
            continue
        assert not infeasible_seen
        assert prev_acc is None or g["accuracy"] <= prev_acc
        prev_acc = g["accuracy"]
        check_plan(w, w.demand_mqps[j], g)


def test_c4_full_every_level():
    w = W.make_workload("C4")
    got = _solve_all(w)
    ref = oracle.solve(w, n_threads=NCPU)
    assert_same(w, got, ref, w.demand_mqps)
    _sweep_invariants(w, got)


@pytest.mark.parametrize("name,n_sample", [("C3", 12), ("C5", 12)])
def test_full_size_sampled_levels(name, n_sample):
    w = W.make_workload(name)
    got = _solve_all(w)
    _sweep_invariants(w, got)
    order = sorted(range(w.n_levels), key=lambda j: w.demand_mqps[j])
    # spread the sample over the sweep and include both ends
    picks = sorted({order[int(round(k * (w.n_levels - 1) / (n_sample - 1)))] for k in range(n_sample)})
    dem = [w.demand_mqps[j] for j in picks]
    ref = oracle.solve(w, demand_mqps=dem, n_threads=NCPU)
    assert_same(w, [got[j] for j in picks], ref, dem)


@pytest.mark.parametrize("name,n_sample", [("C4", 8), ("C5", 8)])
def test_full_size_with_per_variant_factors(name, n_sample):
    """The sweeps `bench.py --variant-factors` times (same seeded factors 1.0 .. 2.0 per variant): the
    root-first kernel must be the one that runs -- C5's 94-member classes included -- and agree with
    the oracle on levels spread over the sweep."""
    w = W.make_workload(name)
    frng = W.SplitMix64(99)
    w.variant_fanout_milli = [1000 + int(frng.randint(0, 8)) * 125 for _ in range(sum(w.n_variants))]
    a = B.Allocator(w)
    try:
        assert a.info().direct_ok == 0 and a.info().path_current == B.LOKI_PATH_UNIFORM
        got = [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
    finally:
        a.close()
    _sweep_invariants(w, got)
    order = sorted(range(w.n_levels), key=lambda j: w.demand_mqps[j])
    picks = sorted({order[int(round(k * (w.n_levels - 1) / (n_sample - 1)))] for k in range(n_sample)})
    dem = [w.demand_mqps[j] for j in picks]
    ref = oracle.solve(w, demand_mqps=dem, n_threads=NCPU)
    assert_same(w, [got[j] for j in picks], ref, dem)
