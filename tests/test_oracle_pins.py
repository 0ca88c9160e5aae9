"""Pins of the CPU oracle against things other than itself: hand-worked
examples (tests/golden), an independent brute force, closed forms, special
cases and invariants that follow from the paper's constraint set."""
import itertools
import random
from fractions import Fraction

import pytest

import brute
import oracle
from helpers import check_plan, golden_rows, h1_workload, ceil_frac
from paper_2407_03583_b200 import workloads as W


def _d(r, w):
    return oracle.result_to_dict(r, w.n_tasks)


# ---------------------------------------------------------------- hand-worked

def test_h1_golden_table():
    rows = golden_rows("h1_two_stage_chain.txt")
    w = h1_workload(0, [int(r[0]) for r in rows])
    res = oracle.solve(w)
    for row, r in zip(rows, res):
        d = _d(r, w)
        assert d["cand_index"] == int(row[1]), row
        assert d["total_workers"] == int(row[2]), row
        assert float.fromhex(row[5]) == d["accuracy"], row
        if int(row[1]) >= 0:
            assert d["status"] == 0
            assert [d["workers"][0][0], d["workers"][1][0]] == [int(row[3]), int(row[4])]
            check_plan(w, w.demand_mqps[rows.index(row)], d)
        else:
            assert d["status"] == 1 and d["accuracy"] == 0.0


def test_h1_per_option_worker_tables():
    """Worker counts of every option at D = 200, 400, 800 (hand table in the
    golden file's derivation), read off by restricting the search to one candidate."""
    w = h1_workload(0, [200, 400, 800])
    w.cluster_size = 1000
    w.slo_us = 10 ** 9
    expect0 = {200: [1, 1, 2, 2], 400: [2, 2, 4, 4], 800: [4, 4, 8, 7]}
    expect1 = {200: [2, 2, 5, 4], 400: [4, 3, 10, 8], 800: [7, 5, 20, 16]}
    for o0 in range(4):
        for o1 in range(4):
            c = o0 + 4 * o1
            res = oracle.solve(w, cand_range=(c, c + 1))
            for q, r in zip((200, 400, 800), res):
                d = _d(r, w)
                assert d["cand_index"] == c
                assert d["workers"][0][0] == expect0[q][o0]
                assert d["workers"][1][0] == expect1[q][o1]


def test_h2_single_split_candidate():
    w = h1_workload(1, [400])
    w.cluster_size = 1000
    # task 0 option 22 = pair (o1=0, o2=2), k=4; task 1 option 0
    c = 22 + 94 * 0
    d = _d(oracle.solve(w, cand_range=(c, c + 1))[0], w)
    assert d["cand_index"] == c
    assert d["variant"][0] == [0, 1] and d["batch"][0] == [1, 1] and d["split_k"][0] == 4
    assert d["workers"][0] == [1, 3]
    assert d["latency_budget_us"][0] == 10000
    # accuracy = 0.875 * 0.7
    assert d["accuracy"] == 0.875 * 0.7


def test_h3_split_sweep_golden():
    rows = golden_rows("h3_two_stage_split.txt")
    w = h1_workload(1, [int(r[0]) for r in rows])
    assert w.n_candidates() == 8836
    res = oracle.solve(w, n_threads=3)
    for row, r, dm in zip(rows, res, w.demand_mqps):
        d = _d(r, w)
        assert d["cand_index"] == int(row[1]), row
        assert d["total_workers"] == int(row[2]), row
        assert float.fromhex(row[3]) == d["accuracy"], row
        if d["status"] == 0:
            check_plan(w, dm, d)
    d600 = _d(res[3], w)
    assert d600["variant"] == [[1, -1], [0, 1]] and d600["batch"] == [[2, 0], [2, 1]]
    assert d600["split_k"] == [16, 12] and d600["workers"] == [[5, 0], [3, 4]]


def test_h3_brute_force_agrees_and_naive_split_formula_is_caught():
    """The brute force reproduces H3; with the naive split mean
    (k*A1 + (16-k)*A2)/16 planted into a copy of it, D = 10 would pick c = 269
    with 3 workers -- the spurious 1-ulp gain the three-operation form avoids."""
    w = h1_workload(1, [10, 600])
    got = brute.solve(w)
    assert (got[0]["cand_index"], got[0]["total_workers"]) == (190, 2)
    assert (got[1]["cand_index"], got[1]["total_workers"]) == (5643, 12)
    orig = brute.task_options

    def naive(w_, task):
        opts = orig(w_, task)
        nb = len(w_.batch_sizes)
        first = sum(w_.n_variants[:task])
        singles = [(v, bi) for v in range(w_.n_variants[task]) for bi in range(nb)]
        idx = len(singles)
        for (v1, _), (v2, _) in itertools.combinations(singles, 2):
            for k in range(1, 16):
                a1, a2 = w_.accuracy[first + v1], w_.accuracy[first + v2]
                opts[idx] = ((k * a1 + (16 - k) * a2) / 16.0,) + opts[idx][1:]
                idx += 1
        return opts

    brute.task_options = naive
    try:
        bad = brute.solve_level(w, 10_000)
    finally:
        brute.task_options = orig
    assert (bad["cand_index"], bad["total_workers"]) == (269, 3)


# ---------------------------------------------------------------- brute force

def _random_cases():
    cases = []
    seed = 0
    for split in (0, 1):
        for T in (1, 2, 3):
            for rep in range(40 if not split else 12):
                seed += 1
                rnd = random.Random(seed)
                if split:
                    V = [rnd.randint(1, 2) for _ in range(T)]
                    nb = rnd.randint(1, 2) if T < 3 else 1
                    if T == 3:
                        V = [rnd.randint(1, 2), 1, rnd.randint(1, 2)]
                else:
                    V = [rnd.randint(1, 3) for _ in range(T)]
                    nb = rnd.randint(1, 3)
                bs = sorted(rnd.sample([1, 2, 3, 4, 6, 8, 16], nb))
                cases.append((seed, T, V, bs, split, rep % 3 == 0))
    return cases


@pytest.mark.parametrize("seed,T,V,bs,split,frac", _random_cases())
def test_oracle_matches_brute_force(seed, T, V, bs, split, frac):
    w = W.random_workload(seed, n_tasks=T, n_variants=V, batch_sizes=bs, split_mode=split,
                          n_levels=5, fan_fractional=frac)
    res = oracle.solve(w, n_threads=1 + seed % 3)
    ref = brute.solve(w)
    for r, b, dm in zip(res, ref, w.demand_mqps):
        d = _d(r, w)
        if b is None:
            assert d["status"] == 1 and d["cand_index"] == -1
        else:
            assert d["status"] == 0
            assert d["cand_index"] == b["cand_index"]
            assert d["total_workers"] == b["total_workers"]
            assert d["accuracy"] == b["accuracy"]
            assert [x[:len(p)] for x, p in zip(d["workers"], b["workers"])] == b["workers"]
            check_plan(w, dm, d)


def test_brute_force_with_comm_latency():
    w = W.random_workload(777, n_tasks=3, n_variants=2, batch_sizes=[1, 4], n_levels=4)
    w.comm_us = 1500
    res = oracle.solve(w)
    ref = brute.solve(w)
    for r, b in zip(res, ref):
        assert r.cand_index == (b["cand_index"] if b else -1)


# ---------------------------------------------------------------- closed forms

def test_single_task_is_a_table_scan():
    w = W.random_workload(5, n_tasks=1, n_variants=4, batch_sizes=[1, 2, 4], n_levels=12)
    nb = 3
    for r, dm in zip(oracle.solve(w), w.demand_mqps):
        best = None
        for v in range(4):
            for bi, b in enumerate(w.batch_sizes):
                lat = w.latency_us[v * nb + bi]
                if 2 * lat > w.slo_us:
                    continue
                x = ceil_frac(Fraction(dm * lat, b * 10 ** 9))
                if x > w.cluster_size:
                    continue
                key = (w.accuracy[v], -x, -(v * nb + bi))
                if best is None or key > best:
                    best = key
        if best is None:
            assert r.status == 1
        else:
            assert (r.accuracy, -r.total_workers, -r.cand_index) == best


def test_loose_slo_decouples_tasks():
    """With the SLO out of the way, for a fixed variant tuple the fewest workers
    is the sum over tasks of the per-task minimum over batch sizes; the winner is
    the best variant tuple under that bound."""
    w = W.make_workload("C2", v=4, n_levels=24)
    w.slo_us = 10 ** 12
    nb = len(w.batch_sizes)
    T = w.n_tasks
    res = oracle.solve(w, n_threads=4)
    for r, dm in zip(res, w.demand_mqps):
        dem = [dm]
        for i in range(1, T):
            dem.append(ceil_frac(Fraction(dem[w.parent[i]] * w.fanout_milli[i], 1000)))
        best = None
        for vt in itertools.product(range(4), repeat=T):
            tot = 0
            for i, v in enumerate(vt):
                tot += min(ceil_frac(Fraction(dem[i] * w.latency_us[(4 * i + v) * nb + bi], b * 10 ** 9))
                           for bi, b in enumerate(w.batch_sizes))
            if tot > w.cluster_size:
                continue
            acc = w.accuracy[vt[0]]
            for i in range(1, T):
                acc = acc * w.accuracy[4 * i + vt[i]]
            if best is None or (acc, -tot) > best:
                best = (acc, -tot)
        if best is None:
            assert r.status == 1
        else:
            assert (r.accuracy, -r.total_workers) == best


def test_hardware_scaling_step_when_max_accuracy_fits():
    """Step 1 of the paper (Eqs. 8-11): while the most accurate variant of every
    task fits in the cluster the winner uses exactly those variants and the
    fewest workers over all batch tuples."""
    w = W.make_workload("C2", v=3, n_levels=40)
    nb = len(w.batch_sizes)
    T = w.n_tasks
    res = oracle.solve(w, n_threads=4)
    n_step1 = 0
    for r, dm in zip(res, w.demand_mqps):
        dem = [dm]
        for i in range(1, T):
            dem.append(ceil_frac(Fraction(dem[w.parent[i]] * w.fanout_milli[i], 1000)))
        fewest = None
        for bt in itertools.product(range(nb), repeat=T):
            lat = [w.latency_us[(3 * i + 2) * nb + bt[i]] for i in range(T)]
            if 2 * sum(lat) > w.slo_us:
                continue
            tot = sum(ceil_frac(Fraction(dem[i] * lat[i], w.batch_sizes[bt[i]] * 10 ** 9)) for i in range(T))
            if tot <= w.cluster_size and (fewest is None or tot < fewest):
                fewest = tot
        if fewest is not None:
            n_step1 += 1
            d = _d(r, w)
            assert [d["variant"][i][0] for i in range(T)] == [2] * T
            assert d["total_workers"] == fewest
            acc = w.accuracy[2]
            for i in range(1, T):
                acc = acc * w.accuracy[3 * i + 2]
            assert d["accuracy"] == acc
    assert 0 < n_step1 < len(res)


# ---------------------------------------------------------------- invariants

def _sorted_levels(w, res):
    order = sorted(range(w.n_levels), key=lambda j: w.demand_mqps[j])
    return [(w.demand_mqps[j], res[j]) for j in order]


@pytest.mark.parametrize("name,v,m", [("C2", 8, 256), ("C3", 3, 64), ("C4", 3, 32), ("C5", 2, 48)])
def test_invariants_along_a_demand_sweep(name, v, m):
    w = W.make_workload(name, v=v, n_levels=m)
    res = oracle.solve(w, n_threads=8)
    top = None
    seq = _sorted_levels(w, res)
    prev_acc, prev_w, seen_infeasible = None, None, False
    max_acc = max(r.accuracy for _, r in seq)
    for dm, r in seq:
        if r.status == 1:
            seen_infeasible = True
            continue
        assert not seen_infeasible, "feasibility must be monotone in demand"
        d = _d(r, w)
        check_plan(w, dm, d)
        if prev_acc is not None:
            assert r.accuracy <= prev_acc, "accuracy can only fall as demand rises"
        if r.accuracy == max_acc and prev_w is not None and prev_acc == max_acc:
            assert r.total_workers >= prev_w, "phase 1: workers grow while accuracy holds"
        prev_acc, prev_w = r.accuracy, r.total_workers
    assert any(r.status == 0 for _, r in seq)


def test_split_mode_never_loses_to_single_mode():
    w1 = W.make_workload("C5", v=2, n_levels=40)
    w0 = W.make_workload("C5", v=2, n_levels=40)
    w0.split_mode = 0
    r1 = oracle.solve(w1, n_threads=8)
    r0 = oracle.solve(w0, n_threads=2)
    gains = 0
    for a, b in zip(r1, r0):
        if b.status == 0:
            assert a.status == 0 and a.accuracy >= b.accuracy
            gains += a.accuracy > b.accuracy
        else:
            gains += a.status == 0
    assert gains > 0


def test_looser_slo_or_bigger_cluster_never_hurts():
    base = W.make_workload("C2", v=4, n_levels=32)
    r0 = oracle.solve(base, n_threads=4)
    for field, factor in (("slo_us", 1.5), ("cluster_size", 2)):
        w = W.make_workload("C2", v=4, n_levels=32)
        setattr(w, field, int(getattr(w, field) * factor))
        r1 = oracle.solve(w, n_threads=4)
        for a, b in zip(r1, r0):
            if b.status == 0:
                assert a.status == 0 and a.accuracy >= b.accuracy


def test_slo_below_twice_the_fastest_path_is_infeasible():
    w = W.make_workload("C2", v=4, n_levels=8)
    nb = len(w.batch_sizes)
    fastest = sum(min(w.latency_us[(4 * i + v) * nb] for v in range(4)) for i in range(3))
    w.slo_us = 2 * fastest - 1
    assert all(r.status == 1 for r in oracle.solve(w))
    w.slo_us = 2 * fastest
    assert oracle.solve(w)[0].status == 0


# ---------------------------------------------------------------- metamorphic

def test_time_scaling_and_level_permutation():
    w = W.make_workload("C2", v=4, n_levels=20)
    w.demand_mqps = [2 * (d // 2) for d in w.demand_mqps]
    r0 = oracle.solve(w, n_threads=2)
    w2 = W.make_workload("C2", v=4, n_levels=20)
    w2.latency_us = [2 * x for x in w.latency_us]
    w2.slo_us = 2 * w.slo_us
    w2.demand_mqps = [d // 2 for d in w.demand_mqps]
    # fan-outs are whole, so halving the root demand halves every stage demand
    r2 = oracle.solve(w2, n_threads=2)
    for a, b in zip(r0, r2):
        assert (a.cand_index, a.total_workers, a.accuracy) == (b.cand_index, b.total_workers, b.accuracy)
    perm = list(range(20))
    random.Random(3).shuffle(perm)
    w3 = w.with_demands([w.demand_mqps[j] for j in perm])
    r3 = oracle.solve(w3)
    for k, j in enumerate(perm):
        assert r3[k].cand_index == r0[j].cand_index


def test_bad_demand_and_thread_count_independence():
    w = W.make_workload("C2", v=3, n_levels=6)
    w.demand_mqps[2] = -5
    w.demand_mqps[4] = w.max_demand_mqps + 1
    a = oracle.solve(w, n_threads=1)
    b = oracle.solve(w, n_threads=7)
    assert a[2].status == 2 and a[4].status == 2 and a[2].cand_index == -1
    for x, y in zip(a, b):
        assert (x.cand_index, x.total_workers, x.accuracy, x.status) == \
               (y.cand_index, y.total_workers, y.accuracy, y.status)


def test_zero_demand_needs_no_workers():
    w = h1_workload(0, [0])
    r = oracle.solve(w)[0]
    # every candidate needs 0 workers; best accuracy with the lowest index: (2,2) -> c = 10
    assert (r.cand_index, r.total_workers, r.status) == (10, 0, 0)


# ---------------------------------------------------------------- per-variant multiplicative factors

def test_variant_factor_hand_example():
    """H1 with r(0, v1) = 1.5 (the more accurate detector emits more requests).
    D = 200 QPS: dem0 = 2e5.  With task 0 on v1 the classifier sees
    2e5 * 2.0 * 1.5 = 6e5 mQPS; its option (v1, b=2) then needs
    ceil(6e5 * 20000 / 2e9) = 6 workers, (v1, b=1) needs ceil(7.2) = 8.
    Best accuracy 0.9 * 0.95: (2,3) costs 2 + 6 = 8, (2,2) and (3,2) cost 2 + 8 = 10 -> c = 14, W = 8.
    With task 0 on v0 (factor 1.0) nothing changes from H1."""
    w = h1_workload(0, [200])
    w.variant_fanout_milli = [1000, 1500, 1000, 1000]
    d = _d(oracle.solve(w)[0], w)
    assert (d["cand_index"], d["total_workers"]) == (14, 8)
    assert d["workers"] == [[2, 0], [6, 0]] and d["stage_demand_mqps"] == [200000, 600000]
    check_plan(w, 200000, d)
    # restricted to task 0 = v0: H1's numbers
    w.cluster_size = 1000
    w.slo_us = 10 ** 9
    d = _d(oracle.solve(w, cand_range=(0 + 4 * 3, 0 + 4 * 3 + 1))[0], w)
    assert d["workers"] == [[1, 0], [4, 0]] and d["stage_demand_mqps"] == [200000, 400000]


def test_variant_factor_split_parent_mixes_the_two_factors():
    """A split parent (k/16 of v0, the rest of v1) passes on the share-weighted factor:
    k = 4, factors 1.0 and 1.5 -> (4*1000 + 12*1500)/16000 = 1.375; child demand
    = ceil(4e5 * 2.0 * 1.375) = 1.1e6 mQPS."""
    w = h1_workload(1, [400])
    w.variant_fanout_milli = [1000, 1500, 1000, 1000]
    w.cluster_size = 1000
    c = 22 + 94 * 0                     # task 0: pair (v0,b1)/(v1,b1) with k = 4; task 1: option 0
    d = _d(oracle.solve(w, cand_range=(c, c + 1))[0], w)
    assert d["stage_demand_mqps"] == [400000, 1100000]
    assert d["workers"][1] == [5, 0]    # ceil(1.1e6 * 4000 / 1e9) = ceil(4.4)


def _vf_cases():
    out = []
    for seed in range(60):
        rnd = random.Random(500 + seed)
        split = seed % 3 == 0
        T = rnd.randint(2, 3)
        V = [rnd.randint(1, 2) for _ in range(T)] if split else [rnd.randint(1, 3) for _ in range(T)]
        if split and T == 3:
            V[1] = 1
        nb = 1 if (split and T == 3) else rnd.randint(1, 2)
        out.append((seed, T, V, sorted(rnd.sample([1, 2, 4, 8], nb)), int(split)))
    return out


@pytest.mark.parametrize("seed,T,V,bs,split", _vf_cases())
def test_oracle_matches_brute_force_with_variant_factors(seed, T, V, bs, split):
    w = W.random_workload(900 + seed, n_tasks=T, n_variants=V, batch_sizes=bs, split_mode=split,
                          n_levels=5, fan_fractional=seed % 2 == 0, variant_fan=True)
    res = oracle.solve(w, n_threads=1 + seed % 2)
    ref = brute.solve(w)
    for r, b, dm in zip(res, ref, w.demand_mqps):
        d = _d(r, w)
        if b is None:
            assert d["status"] == 1
        else:
            assert (d["cand_index"], d["total_workers"], d["accuracy"]) == \
                   (b["cand_index"], b["total_workers"], b["accuracy"])
            check_plan(w, dm, d)


def test_unit_variant_factors_change_nothing():
    w = W.make_workload("C2", v=4, n_levels=24)
    a = oracle.solve(w, n_threads=4)
    w.variant_fanout_milli = [1000] * sum(w.n_variants)
    b = oracle.solve(w, n_threads=4)
    for x, y in zip(a, b):
        assert (x.cand_index, x.total_workers, x.accuracy, x.status) == \
               (y.cand_index, y.total_workers, y.accuracy, y.status)


def test_products_beyond_63_bits_take_the_wide_division():
    """demand x latency above 2^63: the oracle's ceiling division must go through its 128-bit
    branch.  One task, one huge batch size; the expected worker counts are Python big integers."""
    batch = 1 << 20
    lats = [5_000_000, 7_000_001]
    w = W.Workload(name="wide", parent=[-1], fanout_milli=[1000], n_variants=[2], batch_sizes=[batch],
                   accuracy=[0.7, 0.9], latency_us=lats, slo_us=10 ** 8, comm_us=0, cluster_size=30000,
                   split_mode=0, demand_mqps=[4 * 10 ** 12, 4 * 10 ** 12 + 1, 10 ** 13],
                   max_demand_mqps=2 * 10 ** 13)
    for r, d in zip(oracle.solve(w), w.demand_mqps):
        o = oracle.result_to_dict(r, 1)
        assert d * lats[1] > 2 ** 63
        need = [-(-d * lat // (batch * 10 ** 9)) for lat in lats]
        # the more accurate variant wins while it fits the cluster, else the other one, else nothing
        if need[1] <= w.cluster_size:
            assert (o["status"], o["cand_index"], o["total_workers"]) == (0, 1, need[1])
        elif need[0] <= w.cluster_size:
            assert (o["status"], o["cand_index"], o["total_workers"]) == (0, 0, need[0])
        else:
            assert o["status"] == 1
