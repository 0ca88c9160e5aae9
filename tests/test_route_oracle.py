"""Pins of the routing oracle (MostAccurateFirst, Algorithm 1 of Section 5.1):
hand-worked routing tables, an independent exact-rational replay, and the
properties the paper states for the algorithm -- workers are saturated in
non-increasing order of single-model accuracy, requests are conserved, no
worker exceeds its capacity (Eq. 5), and the routed accuracy is never below
the accuracy the allocation promised."""
import random
from fractions import Fraction

import pytest

import oracle
from oracle import route_oracle as R
from helpers import golden_rows, h1_workload
from paper_2407_03583_b200 import workloads as W
from paper_2407_03583_b200.workloads import Workload


def example_a():
    w = h1_workload(0, [200])
    plan = oracle.result_to_dict(oracle.solve(w)[0], 2)
    assert plan["cand_index"] == 14
    return w, 200_000, plan


def example_b():
    w = Workload(
        name="RB", parent=[-1, 0], fanout_milli=[1000, 1500], n_variants=[2, 2],
        batch_sizes=[1, 2, 4], accuracy=[0.8, 0.9, 0.7, 0.95],
        #            v0: b=1      2      4    v1: b=1     2      4
        latency_us=[5000, 12000, 20000, 10000, 17000, 30000,
                    6000, 11000, 20000, 9000, 16000, 31000],
        slo_us=200000, comm_us=0, cluster_size=16, split_mode=1,
        demand_mqps=[300_000], max_demand_mqps=10_000_000)
    w.variant_fanout_milli = [1000, 2000, 1000, 1000]
    plan = {"status": 0, "split_k": [8, 8],
            "variant": [[0, 1], [1, 0]], "batch": [[4, 1], [2, 4]], "workers": [[1, 2], [4, 2]]}
    return w, 300_000, plan


def test_hand_worked_routing_tables():
    rows = golden_rows("r1_route_two_stage.txt")
    for name, (w, dem, plan) in (("A", example_a()), ("B", example_b())):
        res = R.route(w, dem, plan)
        assert res.status == 0 and res.unrouted_qps == 0.0
        want_e = [(int(r[2]), int(r[3]), float(r[4]) / float(r[5])) for r in rows if r[0] == "E" and r[1] == name]
        want_w = {int(r[2]): (float(r[3]), float(r[4])) for r in rows if r[0] == "W" and r[1] == name}
        assert res.entries == want_e
        assert len(res.workers) == len(want_w)
        for k, wk in enumerate(res.workers):
            assert (wk.incoming_qps, wk.leftover_qps) == want_w[k]


def exact_route(w, demand_mqps, plan):
    """The same greedy in exact rationals, written independently: per edge, walk the
    parent's and the child's sorted workers as two queues."""
    T = w.n_tasks
    nb = len(w.batch_sizes)
    first = [sum(w.n_variants[:i]) for i in range(T)]
    vfan = getattr(w, "variant_fanout_milli", None)
    ws = []          # (task, variant, capacity)
    ids = [[] for _ in range(T)]
    for i in range(T):
        groups = []
        for s in range(1 if plan["split_k"][i] == 16 else 2):
            v, b, n = plan["variant"][i][s], plan["batch"][i][s], plan["workers"][i][s]
            groups.append((-w.accuracy[first[i] + v], s, v, b, n))
        for _na, _s, v, b, n in sorted(groups, key=lambda g: (g[0], g[1])):
            lat = w.latency_us[(first[i] + v) * nb + w.batch_sizes.index(b)]
            for _ in range(n):
                ids[i].append(len(ws))
                ws.append((i, v, Fraction(b * 10 ** 6, lat)))
    inc = [Fraction(0)] * len(ws)
    left = [x[2] for x in ws]
    flows = {}
    lost = Fraction(0)
    order = [(-1, 0)] + [(p, c) for p in range(T) for c in range(T) if w.parent[c] == p]
    for p, c in order:
        srcs = [-1] if p < 0 else ids[p]
        for u in srcs:
            if u < 0:
                out = Fraction(demand_mqps, 1000)
            else:
                f = Fraction(1) if vfan is None else Fraction(vfan[first[p] + ws[u][1]], 1000)
                out = inc[u] * f * Fraction(w.fanout_milli[c], 1000)
            total = out
            for v in ids[c]:
                if out > 0 and left[v] > 0:
                    x = min(out, left[v])
                    flows[(u, v)] = x / total
                    out -= x
                    left[v] -= x
                    inc[v] += x
            lost += out
    return ws, inc, left, flows, lost


def check_properties(w, demand_mqps, plan, res, exact=True):
    T = w.n_tasks
    first = [sum(w.n_variants[:i]) for i in range(T)]
    scale = max(1.0, demand_mqps / 1000.0) * 64
    by_task = [[k for k, x in enumerate(res.workers) if x.task == i] for i in range(T)]
    # the plan's workers, all of them, most accurate first
    for i in range(T):
        n_plan = sum(plan["workers"][i][s] for s in range(1 if plan["split_k"][i] == 16 else 2))
        assert len(by_task[i]) == n_plan
        accs = [w.accuracy[first[i] + res.workers[k].variant] for k in by_task[i]]
        assert accs == sorted(accs, reverse=True)
    for k, x in enumerate(res.workers):
        assert 0.0 <= x.incoming_qps <= x.capacity_qps * (1 + 1e-12)
        assert abs(x.capacity_qps - x.incoming_qps - x.leftover_qps) <= 1e-9 * scale
    # saturation order: within a task, nobody receives requests while a more accurate worker has room
    for i in range(T):
        seen_room = False
        for k in by_task[i]:
            x = res.workers[k]
            if seen_room:
                assert x.incoming_qps <= 1e-9 * scale
            if x.leftover_qps > 1e-9 * scale:
                seen_room = True
    # conservation: the probabilities of one source towards one child task sum to one
    sums = {}
    for s, d, pr in res.entries:
        assert 0.0 < pr <= 1.0 + 1e-12
        sums[(s, res.workers[d].task)] = sums.get((s, res.workers[d].task), 0.0) + pr
    if res.unrouted_qps <= 1e-9 * scale:
        for v in sums.values():
            assert abs(v - 1.0) <= 1e-9
    assert abs(sum(res.workers[k].incoming_qps for k in by_task[0]) + 0.0 - demand_mqps / 1000.0) <= 1e-9 * scale \
        or res.unrouted_qps > 0
    if exact:
        ws, inc, left, flows, lost = exact_route(w, demand_mqps, plan)
        assert len(ws) == len(res.workers)
        for k, x in enumerate(res.workers):
            assert (x.task, x.variant) == ws[k][:2]
            assert abs(x.capacity_qps - float(ws[k][2])) <= 1e-12 * x.capacity_qps
            assert abs(x.incoming_qps - float(inc[k])) <= 1e-9 * scale
            assert abs(x.leftover_qps - float(left[k])) <= 1e-9 * scale
        assert abs(res.unrouted_qps - float(lost)) <= 1e-9 * scale
        got = {(s, d): pr for s, d, pr in res.entries if pr > 1e-9}
        want = {k: float(v) for k, v in flows.items() if v > Fraction(1, 10 ** 9)}
        assert set(got) == set(want)
        for k in got:
            assert abs(got[k] - want[k]) <= 1e-9


def routed_accuracy(w, res):
    """End-to-end accuracy of the routed traffic under independent routing: per
    task the request-weighted mean accuracy, multiplied along each path, averaged
    over the leaves (the accuracy model of Section 2.1)."""
    T = w.n_tasks
    first = [sum(w.n_variants[:i]) for i in range(T)]
    mean = []
    for i in range(T):
        xs = [x for x in res.workers if x.task == i]
        tot = sum(x.incoming_qps for x in xs)
        mean.append(sum(x.incoming_qps * w.accuracy[first[i] + x.variant] for x in xs) / tot)
    pp = [0.0] * T
    for i in range(T):
        pp[i] = mean[i] if i == 0 else pp[w.parent[i]] * mean[i]
    leaves = [i for i in range(T) if i not in w.parent]
    return sum(pp[i] for i in leaves) / len(leaves)


@pytest.mark.parametrize("split", [0, 1])
def test_properties_on_allocator_plans(split):
    n_checked = 0
    for seed in range(24):
        rnd = random.Random(500 + seed)
        T = rnd.randint(1, 3 if split else 4)
        w = W.random_workload(700 + seed, n_tasks=T, n_variants=[rnd.randint(1, 3) for _ in range(T)],
                              batch_sizes=sorted(rnd.sample([1, 2, 4, 8], rnd.randint(1, 3))),
                              split_mode=split, n_levels=6, fan_fractional=seed % 2 == 1)
        for dem, r in zip(w.demand_mqps, oracle.solve(w, n_threads=2)):
            plan = oracle.result_to_dict(r, T)
            res = R.route(w, dem, plan)
            if plan["status"] != 0:
                assert res.status == 1 and not res.entries and not res.workers
                continue
            if dem == 0:
                continue
            check_properties(w, dem, plan, res)
            # the allocation provisions every stage for its demand: nothing is left unrouted
            assert res.unrouted_qps <= 1e-9 * max(1.0, dem / 1000.0) * 64
            # "MostAccurateFirst maximizes the end-to-end pipeline accuracy": never below the plan's
            assert routed_accuracy(w, res) >= plan["accuracy"] * (1 - 1e-12)
            n_checked += 1
    assert n_checked >= 40


def test_per_variant_factors_conserve_requests():
    # with per-variant multiplicative factors the children's demand follows the variants that
    # actually serve the traffic; requests are conserved and the surplus, if any, is reported
    for seed in range(8):
        w = W.random_workload(900 + seed, n_tasks=3, n_variants=[2, 3, 2], batch_sizes=[1, 4],
                              split_mode=1 if seed % 2 else 0, n_levels=5)
        w.variant_fanout_milli = [1000 + 250 * ((seed + k) % 4) for k in range(sum(w.n_variants))]
        for dem, r in zip(w.demand_mqps, oracle.solve(w, n_threads=2)):
            plan = oracle.result_to_dict(r, 3)
            if plan["status"] != 0 or dem == 0:
                continue
            check_properties(w, dem, plan, R.route(w, dem, plan))


def test_demand_above_the_plan_is_reported_not_dropped_silently():
    w, dem, plan = example_a()
    res = R.route(w, 3 * dem, plan)          # three times the demand the plan was made for
    assert res.unrouted_qps == 400.0         # root workers take 200 of 600
    assert all(x.leftover_qps == 0.0 for x in res.workers)
    check_properties(w, 3 * dem, plan, res)


def test_planted_mistake_least_accurate_first_is_caught():
    # sorting the workers the wrong way round breaks the saturation order on example B
    w, dem, plan = example_b()
    bad = {**plan, "variant": [p[::-1] for p in plan["variant"]], "batch": [p[::-1] for p in plan["batch"]],
           "workers": [p[::-1] for p in plan["workers"]]}
    good = R.route(w, dem, plan)
    same = R.route(w, dem, bad)              # group order in the plan must not matter
    assert [(x.task, x.variant, x.incoming_qps) for x in good.workers] == \
           [(x.task, x.variant, x.incoming_qps) for x in same.workers]
    w2 = Workload(**{**w.__dict__})
    w2.accuracy = [0.9, 0.8, 0.95, 0.7]      # swap the accuracies: now v0 is the accurate one
    w2.variant_fanout_milli = w.variant_fanout_milli
    other = R.route(w2, dem, plan)
    assert [x.variant for x in other.workers if x.task == 0] == [0, 1, 1]
