"""Parity at the benchmark's full sizes, on every demand level and for every scoring
kernel a timing is quoted for, in the launch configuration bench.py times (all
levels of the sweep in one solve call).

The oracle enumerates all candidates for all levels once per workload (seconds for
C4, under a minute for C5, a few minutes for C3's 9.8e10 pairs on a multi-core
host); `oracle_cache.winners` keeps its plans per input checksum, so the one run
serves every kernel compared here.  Properties that hold at any size (monotone
accuracy, monotone feasibility, every constraint of the returned plan re-derived
from the raw tables) are checked on every level as well."""
import pytest

from helpers import check_plan
from oracle_cache import full_workload, winners
from paper_2407_03583_b200 import binding as B
from test_gpu_parity import assert_same

pytestmark = pytest.mark.gpu

PATH_NAMES = {B.LOKI_PATH_AUTO: "auto", B.LOKI_PATH_GENERIC: "generic", B.LOKI_PATH_DIRECT: "direct",
              B.LOKI_PATH_HOISTED: "hoisted", B.LOKI_PATH_UNIFORM: "uniform", B.LOKI_PATH_FASTEST: "fastest",
              B.LOKI_PATH_PREFIX: "prefix", B.LOKI_PATH_SHARED: "shared"}


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


def _solve(w, path):
    """All levels in one solve call on `path`; returns (plans, kernel that ran)."""
    a = B.Allocator(w)
    try:
        a.set_path(path)
        got = [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
        return got, a.info().path_last
    finally:
        a.close()


# (workload, path asked for, kernel that must have run)
CASES = [
    ("C4", B.LOKI_PATH_DIRECT, B.LOKI_PATH_DIRECT),
    ("C4", B.LOKI_PATH_HOISTED, B.LOKI_PATH_HOISTED),
    ("C4", B.LOKI_PATH_UNIFORM, B.LOKI_PATH_UNIFORM),
    ("C4", B.LOKI_PATH_GENERIC, B.LOKI_PATH_GENERIC),
    ("C4", B.LOKI_PATH_PREFIX, B.LOKI_PATH_PREFIX),
    ("C4", B.LOKI_PATH_SHARED, B.LOKI_PATH_SHARED),
    ("C4", B.LOKI_PATH_FASTEST, B.LOKI_PATH_PREFIX),
    ("C5", B.LOKI_PATH_DIRECT, B.LOKI_PATH_DIRECT),
    ("C5", B.LOKI_PATH_UNIFORM, B.LOKI_PATH_UNIFORM),
    ("C5", B.LOKI_PATH_HOISTED, B.LOKI_PATH_HOISTED),
    ("C5", B.LOKI_PATH_GENERIC, B.LOKI_PATH_GENERIC),
    ("C5", B.LOKI_PATH_PREFIX, B.LOKI_PATH_PREFIX),
    ("C5", B.LOKI_PATH_SHARED, B.LOKI_PATH_SHARED),
    ("C5", B.LOKI_PATH_FASTEST, B.LOKI_PATH_PREFIX),
    ("C3", B.LOKI_PATH_DIRECT, B.LOKI_PATH_DIRECT),
    ("C3", B.LOKI_PATH_HOISTED, B.LOKI_PATH_HOISTED),
    ("C3", B.LOKI_PATH_UNIFORM, B.LOKI_PATH_UNIFORM),
    ("C3", B.LOKI_PATH_GENERIC, B.LOKI_PATH_GENERIC),
    ("C3", B.LOKI_PATH_PREFIX, B.LOKI_PATH_PREFIX),
    ("C3", B.LOKI_PATH_SHARED, B.LOKI_PATH_SHARED),
    ("C3", B.LOKI_PATH_FASTEST, B.LOKI_PATH_PREFIX),
]


@pytest.mark.parametrize("spec,path,ran", CASES,
                         ids=["%s-%s" % (s, PATH_NAMES[p]) for s, p, _r in CASES])
def test_full_size_every_level(spec, path, ran):
    w = full_workload(spec)
    ref = winners(w)
    got, path_last = _solve(w, path)
    assert path_last == ran
    assert_same(w, got, ref, w.demand_mqps, check=False)


@pytest.mark.parametrize("spec", ["C4", "C5", "C3"])
def test_full_size_default_path_and_sweep_invariants(spec):
    w = full_workload(spec)
    got, path_last = _solve(w, B.LOKI_PATH_AUTO)
    assert path_last == B.LOKI_PATH_PREFIX
    assert_same(w, got, winners(w), w.demand_mqps, check=False)
    _sweep_invariants(w, got)


@pytest.mark.parametrize("spec", ["C4+factors", "C5+factors"])
def test_full_size_with_per_variant_factors(spec):
    """The sweeps `bench.py --variant-factors` times (same seeded factors 1.0 .. 2.0 per variant): the
    root-first kernel must be the one that runs -- C5's 94-member classes included -- and agree with
    the oracle on every level, and so must the generic kernel."""
    w = full_workload(spec)
    ref = winners(w)
    got, path_last = _solve(w, B.LOKI_PATH_AUTO)
    assert path_last == B.LOKI_PATH_UNIFORM
    assert_same(w, got, ref, w.demand_mqps, check=False)
    _sweep_invariants(w, got)
    got, path_last = _solve(w, B.LOKI_PATH_GENERIC)
    assert path_last == B.LOKI_PATH_GENERIC
    assert_same(w, got, ref, w.demand_mqps, check=False)
