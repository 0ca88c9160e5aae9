"""Parity of loki_alloc_route (through the C-ABI) with the routing oracle:
worker lists, routing-table entries (source, destination, probability), routed
and leftover requests per worker, all bit-exact -- both sides run the same IEEE
double operations in the order Algorithm 1 states; the 1e-12 relative bar of the
allocation search is asserted as well."""
import random

import pytest

import oracle
from oracle import route_oracle as R
from helpers import h1_workload
from paper_2407_03583_b200 import binding as B
from paper_2407_03583_b200 import workloads as W
from test_route_oracle import check_properties

pytestmark = pytest.mark.gpu


def gpu_plans_and_routes(w, demands=None, max_workers=None, max_entries=None):
    dem = list(w.demand_mqps if demands is None else demands)
    a = B.Allocator(w, max_levels=len(dem))
    try:
        plans = [B.config_to_dict(c, w.n_tasks) for c in a.solve(dem)]
        mw = max_workers or max(1, w.cluster_size)
        me = max_entries or 2 * w.cluster_size + w.n_tasks
        return plans, B.route_device(a, len(dem), mw, me)
    finally:
        a.close()


def assert_same_routes(w, dem, plans, routes):
    for dm, plan, (h, ws, es) in zip(dem, plans, routes):
        ref = R.route(w, dm, plan)
        if ref.status != 0:
            assert h.status == B.LOKI_ROUTE_NO_PLAN and h.n_workers == 0 and h.n_entries == 0
            continue
        assert h.status == B.LOKI_ROUTE_OK
        assert h.n_workers == len(ref.workers) and h.n_entries == len(ref.entries)
        for g, r in zip(ws, ref.workers):
            assert (g.task, g.variant, g.batch) == (r.task, r.variant, r.batch)
            assert (g.capacity_qps, g.incoming_qps, g.leftover_qps) == (r.capacity_qps, r.incoming_qps, r.leftover_qps)
            assert abs(g.incoming_qps - r.incoming_qps) <= 1e-12 * max(1.0, abs(r.incoming_qps))
        for g, (s, d, pr) in zip(es, ref.entries):
            assert (g.src_worker, g.dst_worker, g.probability) == (s, d, pr)
        assert h.unrouted_qps == ref.unrouted_qps


def test_hand_worked_level():
    w = h1_workload(0, [10, 200, 400, 800, 2000])
    plans, routes = gpu_plans_and_routes(w)
    assert_same_routes(w, w.demand_mqps, plans, routes)
    h, ws, es = routes[1]                       # 200 QPS: the table worked by hand in tests/golden
    assert [(e.src_worker, e.dst_worker, e.probability) for e in es] == \
           [(-1, 0, .5), (-1, 1, .5), (0, 2, .5), (0, 3, .5), (1, 4, .5), (1, 5, .5)]
    assert all(x.incoming_qps == 100.0 and x.leftover_qps == 0.0 for x in ws)
    assert routes[4][0].status == B.LOKI_ROUTE_NO_PLAN


@pytest.mark.parametrize("name,v,m", [("C2", None, None), ("C3", 3, 300), ("C4", 3, 64), ("C5", 2, 200), ("SM", None, 256)])
def test_named_workloads(name, v, m):
    w = W.make_workload(name, v=v, n_levels=m)
    plans, routes = gpu_plans_and_routes(w)
    assert_same_routes(w, w.demand_mqps, plans, routes)
    for dm, plan, (h, ws, es) in list(zip(w.demand_mqps, plans, routes))[:: max(1, w.n_levels // 16)]:
        if plan["status"] == 0 and dm > 0:
            check_properties(w, dm, plan, R.route(w, dm, plan), exact=False)


def test_random_problems_with_split_plans_and_variant_factors():
    n = 0
    for seed in range(24):
        rnd = random.Random(4000 + seed)
        T = rnd.randint(1, 4)
        split = seed % 2
        w = W.random_workload(4100 + seed, n_tasks=min(T, 3) if split else T,
                              n_variants=[rnd.randint(1, 3) for _ in range(T)][: min(T, 3) if split else T],
                              batch_sizes=sorted(rnd.sample([1, 2, 4, 8, 16], rnd.randint(1, 3))),
                              split_mode=split, n_levels=rnd.choice([1, 7, 65]), fan_fractional=seed % 3 == 0)
        if seed % 4 == 1:
            w.variant_fanout_milli = [1000 + 125 * ((seed + k) % 5) for k in range(sum(w.n_variants))]
        w.demand_mqps[0] = 0
        plans, routes = gpu_plans_and_routes(w)
        assert_same_routes(w, w.demand_mqps, plans, routes)
        n += sum(1 for p in plans if p["status"] == 0)
    assert n >= 100


def test_tables_too_small_are_reported():
    w = h1_workload(0, [200, 400])
    plans, routes = gpu_plans_and_routes(w, max_workers=4, max_entries=64)
    assert [r[0].status for r in routes] == [B.LOKI_ROUTE_TABLE_FULL] * 2      # 6 and 12 workers
    plans, routes = gpu_plans_and_routes(w, max_workers=12, max_entries=3)
    assert routes[0][0].status == B.LOKI_ROUTE_TABLE_FULL and routes[0][0].n_entries == 3


def test_argument_errors():
    w = h1_workload(0, [200])
    a = B.Allocator(w)
    try:
        lib = B.load_library()
        assert lib.loki_alloc_route(a.handle, None, a.d_out.data_ptr(), 1, 8, 8, None, 1, 1, 1) == B.LOKI_ERR_INVALID_ARG
        assert lib.loki_alloc_route(a.handle, a.d_demand.data_ptr(), a.d_out.data_ptr(), 0, 8, 8, None, 1, 1, 1) == B.LOKI_ERR_INVALID_ARG
        assert lib.loki_alloc_route(a.handle, a.d_demand.data_ptr(), a.d_out.data_ptr(), 1, 0, 8, None, 1, 1, 1) == B.LOKI_ERR_INVALID_ARG
    finally:
        a.close()
