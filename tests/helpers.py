"""Shared test helpers: the hand-worked H1 problem, golden-file parsing and an
independent feasibility checker that re-derives every constraint of a returned
plan from the raw tables with exact rationals."""
from __future__ import annotations

import os
from fractions import Fraction

from paper_2407_03583_b200.workloads import Workload

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def h1_workload(split_mode: int = 0, demands_qps=(10, 200, 400, 800, 2000)) -> Workload:
    return Workload(
        name="H1", parent=[-1, 0], fanout_milli=[1000, 2000], n_variants=[2, 2],
        batch_sizes=[1, 2], accuracy=[0.8, 0.9, 0.7, 0.95],
        latency_us=[5000, 8000, 10000, 16000, 4000, 6000, 12000, 20000],
        slo_us=60000, comm_us=0, cluster_size=12, split_mode=split_mode,
        demand_mqps=[q * 1000 for q in demands_qps], max_demand_mqps=10_000_000)


def golden_rows(fname: str):
    rows = []
    with open(os.path.join(GOLDEN, fname)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            rows.append(line.split())
    return rows


def ceil_frac(x: Fraction) -> int:
    return -((-x.numerator) // x.denominator)


def check_plan(w: Workload, demand_mqps: int, plan: dict) -> None:
    """Assert that a feasible plan (variant/batch/split_k/workers per task, as
    returned by either implementation) satisfies Eqs. 1-7 of Section 4.1 and
    that its reported worker counts and accuracy follow from the raw tables."""
    T = w.n_tasks
    nb = len(w.batch_sizes)
    first = [sum(w.n_variants[:i]) for i in range(T)]
    vfan = getattr(w, "variant_fanout_milli", None)

    def factor(i):          # share-weighted multiplicative factor of task i's chosen option
        k = plan["split_k"][i]
        f = [1000 if vfan is None else vfan[first[i] + plan["variant"][i][s]] for s in range(1 if k == 16 else 2)]
        return Fraction(f[0], 1000) if k == 16 else Fraction(k * f[0] + (16 - k) * f[1], 16000)

    dem = [0] * T
    dem[0] = demand_mqps
    for i in range(1, T):
        u = w.parent[i]
        dem[i] = ceil_frac(dem[u] * Fraction(w.fanout_milli[i], 1000) * factor(u))
    total = 0
    lat_task = [0] * T
    acc_task = [0.0] * T
    for i in range(T):
        k = plan["split_k"][i]
        parts = 1 if k == 16 else 2
        assert 1 <= k <= 16
        lats, accs = [], []
        for s in range(parts):
            v = plan["variant"][i][s]
            b = plan["batch"][i][s]
            assert 0 <= v < w.n_variants[i] and b in w.batch_sizes
            lat = w.latency_us[(first[i] + v) * nb + w.batch_sizes.index(b)]
            share = k if s == 0 else 16 - k
            if parts == 1:
                share = 16
            need = ceil_frac(Fraction(dem[i] * share * lat, 16 * b * 10 ** 9))
            assert plan["workers"][i][s] == need, (i, s, plan["workers"][i][s], need)
            # Eq. 2: demand routed to this part <= replicas * throughput (b / lat)
            assert Fraction(dem[i] * share, 16 * 1000) <= need * Fraction(b * 10 ** 6, lat)
            total += need
            lats.append(lat)
            accs.append(w.accuracy[first[i] + v])
        if parts == 1:
            assert plan["variant"][i][1] == -1
            acc_task[i] = accs[0]
        else:
            acc_task[i] = accs[1] + (k * 0.0625) * (accs[0] - accs[1])
        lat_task[i] = max(lats)
        assert plan["latency_budget_us"][i] == lat_task[i]
    assert total == plan["total_workers"] <= w.cluster_size          # Eq. 3
    children = [[j for j in range(T) if w.parent[j] == i] for i in range(T)]
    leaves = [i for i in range(T) if not children[i]]
    prod = [0.0] * T
    for i in range(T):
        prod[i] = acc_task[i] if i == 0 else prod[w.parent[i]] * acc_task[i]
    s = None
    for leaf in leaves:
        s = prod[leaf] if s is None else s + prod[leaf]
        tot, hops, j = 0, 0, leaf
        while j != -1:
            tot += lat_task[j]
            hops += 1
            j = w.parent[j]
        assert 2 * tot <= w.slo_us - hops * w.comm_us                # Eqs. 6-7, halved SLO
    assert plan["accuracy"] == s / float(len(leaves))
