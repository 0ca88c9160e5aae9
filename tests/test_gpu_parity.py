"""Parity of the CUDA path (through the C-ABI) with the CPU oracle: chosen
candidates, worker counts and plans bit-exact, accuracies bit-exact (the stated
bar is 1e-12 relative; both sides run the same IEEE operations in the same
order, so equality is asserted and the tolerance is checked as well)."""
import os
import random

import pytest

import oracle
from helpers import check_plan, golden_rows, h1_workload
from paper_2407_03583_b200 import binding as B
from paper_2407_03583_b200 import workloads as W

pytestmark = pytest.mark.gpu
NCPU = max(1, os.cpu_count() or 1)
PATHS = [B.LOKI_PATH_GENERIC, B.LOKI_PATH_DIRECT, B.LOKI_PATH_HOISTED, B.LOKI_PATH_UNIFORM, B.LOKI_PATH_PREFIX,
         B.LOKI_PATH_SHARED]


def shared_tables_ok(a):
    """Whether the handle has the tables shared by all class tuples (two tasks or more, no per-variant factors)."""
    return B.load_library().loki_alloc_set_path(a.handle, B.LOKI_PATH_SHARED) == B.LOKI_OK


def gpu_solve(w, path, demands=None, max_levels=None, host=False):
    dem = list(w.demand_mqps if demands is None else demands)
    a = B.Allocator(w, max_levels=max_levels or max(1, len(dem)))
    try:
        info = a.info()
        if path == B.LOKI_PATH_DIRECT and not info.direct_ok:
            pytest.skip("direct path not applicable to this problem")
        if path == B.LOKI_PATH_UNIFORM and not info.uniform_ok:
            pytest.skip("level-lane path not applicable to this problem")
        if path in (B.LOKI_PATH_HOISTED, B.LOKI_PATH_PREFIX) and not info.hoisted_ok:
            pytest.skip("hoisted path not applicable to this problem")
        if path == B.LOKI_PATH_SHARED and not shared_tables_ok(a):
            pytest.skip("shared tables not applicable to this problem")
        a.set_path(path)
        if host:
            a.h_demand[:len(dem)] = a.torch.tensor(dem, dtype=a.torch.int64)
            a.solve_host(len(dem))
            res = a.read_host(len(dem))
        else:
            res = a.solve(dem)
        return [B.config_to_dict(c, w.n_tasks) for c in res]
    finally:
        a.close()


def assert_same(w, got, ref, demands, check=True):
    assert len(got) == len(ref)
    for g, r, dm in zip(got, ref, demands):
        o = r if isinstance(r, dict) else oracle.result_to_dict(r, w.n_tasks)
        assert g["status"] == o["status"], (dm, g, o)
        assert g["cand_index"] == o["cand_index"], (dm, g, o)
        assert g["total_workers"] == o["total_workers"], (dm, g, o)
        assert g["accuracy"] == o["accuracy"], (dm, g["accuracy"].hex(), o["accuracy"].hex())
        assert abs(g["accuracy"] - o["accuracy"]) <= 1e-12 * abs(o["accuracy"])
        if o["status"] == 0:
            assert g["variant"] == o["variant"] and g["batch"] == o["batch"]
            assert g["workers"] == o["workers"] and g["split_k"] == o["split_k"]
            assert g["latency_budget_us"] == o["latency_budget_us"]
            if check:
                check_plan(w, dm, g)
        else:
            assert g["cand_index"] == -1 and g["accuracy"] == 0.0 and g["total_workers"] == 0


@pytest.mark.parametrize("path", PATHS)
def test_hand_worked_examples(path):
    for split, fname, acc_col in ((0, "h1_two_stage_chain.txt", 5), (1, "h3_two_stage_split.txt", 3)):
        rows = golden_rows(fname)
        w = h1_workload(split, [int(r[0]) for r in rows])
        got = gpu_solve(w, path)
        for row, g in zip(rows, got):
            assert g["cand_index"] == int(row[1]) and g["total_workers"] == int(row[2])
            assert g["accuracy"] == float.fromhex(row[acc_col])
        assert_same(w, got, oracle.solve(w), w.demand_mqps)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name,v,m", [
    ("C1", None, None), ("C2", None, None), ("C3", 3, 4096), ("C4", 3, 64), ("C5", 2, 1024),
    ("C3", 4, 70), ("C4", 4, 9), ("C5", 3, 130), ("SM", None, None),
])
def test_named_workloads_small_enough_for_full_oracle(path, name, v, m):
    w = W.make_workload(name, v=v, n_levels=m)
    got = gpu_solve(w, path)
    ref = oracle.solve(w, n_threads=NCPU)
    assert_same(w, got, ref, w.demand_mqps, check=w.n_levels <= 300)


@pytest.mark.parametrize("name,v,group", [("C4", 2, 6), ("C3", 2, 7), ("C2", 3, 10), ("C5", 2, 15)])
def test_direct_tiles_end_in_every_admitted_group_size(name, v, group):
    """The direct kernel scores a tile in groups of `group` levels and lets the last group be about
    one third, two thirds or all of one: sweeps whose lengths leave every remainder 1 .. group, a
    few that split into several tiles, and class tuples with more latency-feasible candidates than
    one pass takes (so partly filled rows wait for the next pass) must all give the oracle's plans."""
    lengths = list(range(1, group + 2)) + [3 * group - 1, 5 * group + 2, 253, 259, 2 * 252 + 5]
    full = W.make_workload(name, v=v, n_levels=max(lengths))
    ref = oracle.solve(full, n_threads=NCPU)
    a = B.Allocator(full, max_levels=max(lengths))
    try:
        assert a.info().direct_ok
        a.set_path(B.LOKI_PATH_DIRECT)
        for m in lengths:
            got = [B.config_to_dict(c, full.n_tasks) for c in a.solve(full.demand_mqps[:m])]
            assert a.info().level_tile_last * ((m + 251) // 252) >= m
            assert_same(full, got, ref[:m], full.demand_mqps[:m], check=False)
    finally:
        a.close()


def _random_cases(n):
    out = []
    for seed in range(n):
        rnd = random.Random(1000 + seed)
        T = rnd.randint(1, 5)
        split = seed % 4 == 0
        if split:
            T = min(T, 3)
            V = [rnd.randint(1, 3) for _ in range(T)]
            bs = sorted(rnd.sample([1, 2, 4, 8, 16], rnd.randint(1, 3)))
        else:
            V = [rnd.randint(1, 5) for _ in range(T)]
            bs = sorted(rnd.sample([1, 2, 3, 4, 6, 8, 16, 32], rnd.randint(1, 4)))
        out.append((seed, T, V, bs, int(split), seed % 3 == 1, rnd.choice([1, 7, 33, 64, 65, 150])))
    return out


@pytest.mark.parametrize("path", PATHS)
def test_random_problems(path):
    n_run = 0
    for seed, T, V, bs, split, frac, m in _random_cases(48):
        w = W.random_workload(seed, n_tasks=T, n_variants=V, batch_sizes=bs, split_mode=split,
                              n_levels=m, fan_fractional=frac)
        if seed % 5 == 0:
            w.comm_us = 700
        # degenerate levels: zero demand, negative, above the declared maximum
        w.demand_mqps[0] = 0
        if m > 3:
            w.demand_mqps[2] = -1
            w.demand_mqps[3] = w.max_demand_mqps + 1
        a = B.Allocator(w)
        try:
            if path == B.LOKI_PATH_DIRECT and not a.info().direct_ok:
                continue
            if path == B.LOKI_PATH_UNIFORM and not a.info().uniform_ok:
                continue
            if path in (B.LOKI_PATH_HOISTED, B.LOKI_PATH_PREFIX) and not a.info().hoisted_ok:
                continue
            if path == B.LOKI_PATH_SHARED and not shared_tables_ok(a):
                continue
            a.set_path(path)
            got = [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
        finally:
            a.close()
        assert_same(w, got, oracle.solve(w, n_threads=2), w.demand_mqps, check=m <= 40)
        n_run += 1
    assert n_run >= 30


@pytest.mark.parametrize("path", PATHS)
def test_degenerate_shapes(path):
    # one task; eight tasks with one option each; no workers at all; nothing feasible
    w = W.random_workload(3, n_tasks=1, n_variants=5, batch_sizes=[1, 2, 4], n_levels=40)
    assert_same(w, gpu_solve(w, path), oracle.solve(w), w.demand_mqps)
    w = W.random_workload(4, n_tasks=8, n_variants=1, batch_sizes=[4], n_levels=10)
    w.slo_us = 10 ** 7
    w.cluster_size = 200
    assert_same(w, gpu_solve(w, path), oracle.solve(w), w.demand_mqps)
    w = W.random_workload(5, n_tasks=8, n_variants=2, batch_sizes=[1, 8], n_levels=12, chain=True)
    w.slo_us = 10 ** 7
    w.cluster_size = 500
    assert_same(w, gpu_solve(w, path), oracle.solve(w, n_threads=NCPU), w.demand_mqps)
    w = W.make_workload("C2", v=3, n_levels=16)
    w.cluster_size = 0
    got = gpu_solve(w, path)
    assert all(g["status"] == 1 for g in got)
    assert_same(w, got, oracle.solve(w), w.demand_mqps)
    w = W.make_workload("C2", v=3, n_levels=16)
    w.slo_us = 1000
    assert all(g["status"] == 1 for g in gpu_solve(w, path))


def test_both_paths_and_host_entry_agree_on_a_ragged_sweep():
    w = W.make_workload("C2", v=5, n_levels=131)
    ref = oracle.solve(w, n_threads=NCPU)
    for path in PATHS:
        assert_same(w, gpu_solve(w, path, max_levels=200), ref, w.demand_mqps)
        assert_same(w, gpu_solve(w, path, host=True), ref, w.demand_mqps)


def test_solve_argument_errors():
    w = W.make_workload("C1")
    a = B.Allocator(w, max_levels=4)
    try:
        lib = B.load_library()
        ptr = a.d_demand.data_ptr()
        assert lib.loki_alloc_solve(a.handle, ptr, 5, None, a.d_out.data_ptr()) == B.LOKI_ERR_INVALID_ARG
        assert lib.loki_alloc_solve(a.handle, ptr, 0, None, a.d_out.data_ptr()) == B.LOKI_ERR_INVALID_ARG
        assert lib.loki_alloc_solve(a.handle, None, 1, None, a.d_out.data_ptr()) == B.LOKI_ERR_INVALID_ARG
        assert lib.loki_alloc_solve(a.handle, ptr, 1, None, None) == B.LOKI_ERR_INVALID_ARG
        assert lib.loki_alloc_set_path(a.handle, 8) == B.LOKI_ERR_INVALID_ARG
        assert lib.loki_alloc_set_path(a.handle, -1) == B.LOKI_ERR_INVALID_ARG
        assert a.num_candidates() == 256
        # the handle still works after the refused calls
        got = [B.config_to_dict(c, 2) for c in a.solve(w.demand_mqps)]
        assert_same(w, got, oracle.solve(w), w.demand_mqps)
    finally:
        a.close()


def test_score_timing_and_launch_counts():
    """What one solve enqueues: per tile (or batch of tiles) the scoring kernel and the finishing
    kernel (cross-block reduction + winner decode in one launch); the generic and the direct
    kernel first run the level kernel, and the direct kernel also refreshes its constant-memory
    demand tile with one device-to-device copy per tile."""
    w = W.make_workload("C2", v=4, n_levels=600)
    a = B.Allocator(w)
    try:
        B.loki_alloc_set_timing(a.handle, True)
        a.set_path(B.LOKI_PATH_DIRECT)
        info = a.info()
        tile_max = info.direct_level_tile               # whole level groups within 256 levels
        assert 240 <= tile_max <= 256
        a.solve(w.demand_mqps)
        ms, n = B.loki_alloc_last_score_ms(a.handle)
        tiles = -(-600 // tile_max)
        assert n == tiles == 3 and ms > 0.0
        assert a.info().n_launches_last == 1 + 3 * tiles
        assert a.info().level_tile_last * tiles >= 600
        fma = B.loki_alloc_last_fma_count(a.handle)
        # at most one fma per (candidate, padded level, task); fewer: only latency-feasible candidates are scored
        assert 0 < fma <= (w.n_candidates() + 32 * 4 ** 3) * a.info().level_tile_last * tiles * 3
        a.solve(w.demand_mqps[:64])                     # a short sweep is one tile
        assert B.loki_alloc_last_score_ms(a.handle)[1] == 1 and a.info().n_launches_last == 4
        a.set_path(B.LOKI_PATH_GENERIC)
        a.solve(w.demand_mqps)
        ms, n = B.loki_alloc_last_score_ms(a.handle)
        assert n == 1 and ms > 0.0 and a.info().n_launches_last == 3
        assert B.loki_alloc_last_fma_count(a.handle) == 0
        a.set_path(B.LOKI_PATH_HOISTED)
        a.solve(w.demand_mqps)                          # five 128-level tiles in one launch; no level kernel
        assert B.loki_alloc_last_score_ms(a.handle)[1] == 1 and a.info().n_launches_last == 2
    finally:
        a.close()


def test_two_handles_on_two_streams():
    import torch
    w1 = W.make_workload("C2", v=4, n_levels=64)
    w2 = W.make_workload("C4", v=3, n_levels=64)
    a1, a2 = B.Allocator(w1), B.Allocator(w2)
    try:
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        n1, n2 = a1.upload(w1.demand_mqps), a2.upload(w2.demand_mqps)
        torch.cuda.synchronize()
        for _ in range(3):
            with torch.cuda.stream(s1):
                a1.solve_device(n1)
            with torch.cuda.stream(s2):
                a2.solve_device(n2)
        torch.cuda.synchronize()
        assert_same(w1, [B.config_to_dict(c, 3) for c in a1.read_device(n1)],
                    oracle.solve(w1, n_threads=NCPU), w1.demand_mqps)
        assert_same(w2, [B.config_to_dict(c, 5) for c in a2.read_device(n2)],
                    oracle.solve(w2, n_threads=NCPU), w2.demand_mqps)
    finally:
        a1.close()
        a2.close()


def test_variant_factors_above_one_and_demands_past_the_caps():
    """Ratios edge factor x variant factor far above 1 (a child sees many times its parent's
    demand) with awkward thousandths, on sweeps that run from one request to demands where every
    stage is past its cap (the kernel clamps there): the root-first kernel's one-fma stage demand
    must agree with the oracle's integer ceiling at every level."""
    awkward = [333, 1001, 2999, 4096, 999, 1700, 125, 7]
    n_fast = n_feasible = n_infeasible = 0
    for seed in range(10):
        split = int(seed % 5 == 0)
        w = W.random_workload(700 + seed, n_tasks=2 + seed % 3, n_variants=2 if split else 3,
                              batch_sizes=[1, 4] if split else [1, 2, 8], split_mode=split,
                              n_levels=64, fan_fractional=seed % 2 == 1, variant_fan=True)
        rng = W.SplitMix64(7000 + seed)
        w.variant_fanout_milli = [awkward[int(rng.randint(0, len(awkward) - 1))] for _ in range(sum(w.n_variants))]
        top = max(w.demand_mqps)
        w.demand_mqps = [1, 2, 3] + [max(1, top * (k + 1) * (k + 1) // 400) for k in range(61)]
        w.max_demand_mqps = max(w.demand_mqps)
        ref = oracle.solve(w, n_threads=NCPU)
        n_feasible += sum(1 for r in ref if oracle.result_to_dict(r, w.n_tasks)["status"] == 0)
        n_infeasible += sum(1 for r in ref if oracle.result_to_dict(r, w.n_tasks)["status"] != 0)
        a = B.Allocator(w)
        try:
            for path in (B.LOKI_PATH_GENERIC, B.LOKI_PATH_AUTO):
                a.set_path(path)
                got = [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
                n_fast += int(a.info().path_last == B.LOKI_PATH_UNIFORM)
                assert_same(w, got, ref, w.demand_mqps, check=False)
        finally:
            a.close()
    assert n_fast >= 8 and n_feasible >= 50 and n_infeasible >= 50


def test_per_variant_multiplicative_factors():
    """The paper's model of Eq. 1: the child's demand depends on the parent's chosen
    variant.  The generic kernel and the root-first level-lane kernel apply (the latter is
    what AUTO picks); hand-worked cases and random problems (trees, split mode, fractional
    edge factors, sweeps longer than one tile) must match the oracle on both."""
    w = h1_workload(0, [10, 200, 400, 800])
    w.variant_fanout_milli = [1000, 1500, 1000, 1000]
    a = B.Allocator(w)
    try:
        assert a.info().direct_ok == 0 and a.info().path_auto == B.LOKI_PATH_UNIFORM
        assert B.load_library().loki_alloc_set_path(a.handle, B.LOKI_PATH_DIRECT) == B.LOKI_ERR_RANGE
        assert B.load_library().loki_alloc_set_path(a.handle, B.LOKI_PATH_HOISTED) == B.LOKI_ERR_RANGE
        assert B.load_library().loki_alloc_set_path(a.handle, B.LOKI_PATH_PREFIX) == B.LOKI_ERR_RANGE
        assert B.load_library().loki_alloc_set_path(a.handle, B.LOKI_PATH_SHARED) == B.LOKI_ERR_RANGE
        got = [B.config_to_dict(c, 2) for c in a.solve(w.demand_mqps)]
        a.set_path(B.LOKI_PATH_GENERIC)
        got_generic = [B.config_to_dict(c, 2) for c in a.solve(w.demand_mqps)]
    finally:
        a.close()
    assert (got[1]["cand_index"], got[1]["total_workers"], got[1]["workers"]) == (14, 8, [[2, 0], [6, 0]])
    assert_same(w, got, oracle.solve(w), w.demand_mqps)
    assert_same(w, got_generic, oracle.solve(w), w.demand_mqps)
    n_fast = 0
    for seed in range(24):
        split = int(seed % 4 == 0)
        w = W.random_workload(300 + seed, n_tasks=2 + seed % 4, n_variants=2 if split else 3,
                              batch_sizes=[1, 4] if split else [1, 2, 8], split_mode=split,
                              n_levels=[5, 64, 70, 200][seed % 4], fan_fractional=seed % 2 == 1, variant_fan=True)
        w.demand_mqps[0] = 0
        ref = oracle.solve(w, n_threads=NCPU)
        a = B.Allocator(w)
        try:
            for path in (B.LOKI_PATH_GENERIC, B.LOKI_PATH_AUTO):
                a.set_path(path)
                got = [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
                n_fast += int(a.info().path_last == B.LOKI_PATH_UNIFORM)
                assert_same(w, got, ref, w.demand_mqps, check=w.n_levels <= 10)
        finally:
            a.close()
    assert n_fast >= 16
    # the allocation-free entry point runs the same kernels
    w = W.random_workload(333, n_tasks=3, n_variants=3, batch_sizes=[1, 2, 8], n_levels=40, variant_fan=True)
    a = B.Allocator(w)
    try:
        import torch
        n = a.upload(w.demand_mqps)
        torch.cuda.synchronize()
        rc = B.loki_alloc_solve_static(a.handle, a.d_demand.data_ptr(), n,
                                       torch.cuda.current_stream().cuda_stream, a.d_out.data_ptr())
        assert rc == B.LOKI_OK
        got = [B.config_to_dict(c, 3) for c in a.read_device(n)]
    finally:
        a.close()
    assert_same(w, got, oracle.solve(w, n_threads=NCPU), w.demand_mqps, check=False)


def test_slo_sweep_on_one_handle():
    """The SLO study of the paper's evaluation: one pipeline solved under a range of
    SLOs.  The handle is re-targeted with loki_alloc_set_slo; every setting must
    match an oracle run with that SLO, and a looser SLO never lowers accuracy."""
    w = W.make_workload("C2", v=4, n_levels=40)
    w.demand_mqps[0] = 0
    nb = len(w.batch_sizes)
    fastest = sum(min(w.latency_us[(4 * i + v) * nb] for v in range(4)) for i in range(3))
    slos = [2 * fastest - 1, 2 * fastest, 120_000, 200_000, 300_000, 450_000]
    a = B.Allocator(w)
    prev = None
    try:
        for slo in slos:
            B.loki_alloc_set_slo(a.handle, slo, 0)
            w.slo_us = slo
            ref = oracle.solve(w, n_threads=NCPU)
            for path in PATHS:
                a.set_path(path)
                got = [B.config_to_dict(c, 3) for c in a.solve(w.demand_mqps)]
                assert_same(w, got, ref, w.demand_mqps, check=False)
            if slo == slos[0]:
                assert all(r.status == 1 for r in ref)
            if prev is not None:
                for x, y in zip(ref, prev):
                    if y.status == 0:
                        assert x.status == 0 and x.accuracy >= y.accuracy
            prev = ref
        # communication latency shrinks the budget like a tighter SLO
        B.loki_alloc_set_slo(a.handle, 300_000, 20_000)
        w.slo_us, w.comm_us = 300_000, 20_000
        a.set_path(B.LOKI_PATH_AUTO)
        assert_same(w, [B.config_to_dict(c, 3) for c in a.solve(w.demand_mqps)],
                    oracle.solve(w, n_threads=NCPU), w.demand_mqps, check=False)
        assert B.load_library().loki_alloc_set_slo(a.handle, -1, 0) == B.LOKI_ERR_INVALID_ARG
    finally:
        a.close()


def test_slo_sweep_in_one_call_matches_the_oracle_per_slo():
    # both axes of the paper's SLO study in one call: plans[s][l]; the handle's own SLO is untouched
    w = W.make_workload("SM", n_levels=96)
    w.demand_mqps[0] = 0
    slos = [20_000, 60_000, 120_000, 200_000, 300_000, 500_000]
    torch = __import__("torch")
    a = B.Allocator(w)
    try:
        n = a.upload(w.demand_mqps)
        d_out = torch.empty(len(slos) * n * B.CONFIG_SIZE, dtype=torch.uint8, device=a.device)
        for path in (B.LOKI_PATH_DIRECT, B.LOKI_PATH_GENERIC, B.LOKI_PATH_UNIFORM, B.LOKI_PATH_HOISTED, B.LOKI_PATH_PREFIX,
                     B.LOKI_PATH_SHARED):
            a.set_path(path)
            d_out.zero_()
            B.loki_alloc_solve_slos(a.handle, a.d_demand.data_ptr(), n, slos,
                                    torch.cuda.current_stream().cuda_stream, d_out.data_ptr())
            torch.cuda.synchronize()
            raw = d_out.cpu().numpy().tobytes()
            arr = (B.loki_config_t * (len(slos) * n)).from_buffer_copy(raw)
            prev = None
            for s, slo in enumerate(slos):
                ws = w.with_demands(w.demand_mqps)
                ws.slo_us = slo
                ref = oracle.solve(ws, n_threads=NCPU)
                got = [B.config_to_dict(arr[s * n + l], 2) for l in range(n)]
                assert_same(ws, got, ref, w.demand_mqps, check=False)
                if prev is not None:       # a looser SLO never lowers accuracy (Section 6.4)
                    assert all(x.accuracy >= y.accuracy for x, y in zip(ref, prev))
                prev = ref
            # the handle still answers for its own SLO
            assert_same(w, [B.config_to_dict(c, 2) for c in a.solve(w.demand_mqps)],
                        oracle.solve(w, n_threads=NCPU), w.demand_mqps, check=False)
        lib = B.load_library()
        import ctypes
        many = (ctypes.c_int64 * 65)(*([100_000] * 65))
        assert lib.loki_alloc_solve_slos(a.handle, a.d_demand.data_ptr(), n, many, 65, None, d_out.data_ptr()) == B.LOKI_ERR_RANGE
    finally:
        a.close()


def test_slo_axis_is_fused_into_the_hoisted_launches():
    """The two axes of the paper's SLO study at full length -- workload SM's 1024 demand levels
    under 16 SLOs -- on the path the library picks (the hoisted kernel): the SLOs are a second
    batched axis of the same launches, so the whole study is one scoring launch, and every plan
    matches an oracle run with that SLO."""
    torch = __import__("torch")
    w = W.make_workload("SM")
    w.demand_mqps[5] = 0
    slos = [15_000 + 25_000 * s for s in range(16)]
    a = B.Allocator(w)
    try:
        n = a.upload(w.demand_mqps)
        d_out = torch.zeros(len(slos) * n * B.CONFIG_SIZE, dtype=torch.uint8, device=a.device)
        a.set_path(B.LOKI_PATH_FASTEST)
        B.loki_alloc_set_timing(a.handle, True)
        B.loki_alloc_solve_slos(a.handle, a.d_demand.data_ptr(), n, slos,
                                torch.cuda.current_stream().cuda_stream, d_out.data_ptr())
        torch.cuda.synchronize()
        assert a.info().path_last == B.LOKI_PATH_PREFIX
        ms, n_score = B.loki_alloc_last_score_ms(a.handle)
        assert n_score == 1 and ms > 0.0
        # limits copy; zero-demand answers: memset, scoring, finishing; sweep: scoring, finishing
        assert a.info().n_launches_last == 6
        arr = (B.loki_config_t * (len(slos) * n)).from_buffer_copy(d_out.cpu().numpy().tobytes())
        prev = None
        for s, slo in enumerate(slos):
            ws = w.with_demands(w.demand_mqps)
            ws.slo_us = slo
            ref = oracle.solve(ws, n_threads=NCPU)
            assert_same(ws, [B.config_to_dict(arr[s * n + l], 2) for l in range(n)], ref, w.demand_mqps, check=False)
            if prev is not None:       # a looser SLO never lowers accuracy (Section 6.4)
                assert all(x.accuracy >= y.accuracy for x, y in zip(ref, prev))
            prev = ref
        # a big problem: the scratch holds a few (SLO, tile) pairs per launch, the plans are the same
        w4 = W.make_workload("C4", v=4, n_levels=200)
        a4 = B.Allocator(w4)
        try:
            n4 = a4.upload(w4.demand_mqps)
            slos4 = [260_000, 380_000, 500_000]
            out4 = torch.zeros(len(slos4) * n4 * B.CONFIG_SIZE, dtype=torch.uint8, device=a4.device)
            a4.set_path(B.LOKI_PATH_HOISTED)
            B.loki_alloc_solve_slos(a4.handle, a4.d_demand.data_ptr(), n4, slos4,
                                    torch.cuda.current_stream().cuda_stream, out4.data_ptr())
            torch.cuda.synchronize()
            arr4 = (B.loki_config_t * (len(slos4) * n4)).from_buffer_copy(out4.cpu().numpy().tobytes())
            for s, slo in enumerate(slos4):
                ws = w4.with_demands(w4.demand_mqps)
                ws.slo_us = slo
                assert_same(ws, [B.config_to_dict(arr4[s * n4 + l], 5) for l in range(n4)],
                            oracle.solve(ws, n_threads=NCPU), w4.demand_mqps, check=False)
        finally:
            a4.close()
    finally:
        a.close()


def test_default_path_resolution():
    # decided per solve: the hoisted kernel wherever its class tables fit, except short sweeps of a big
    # candidate space, which take the direct kernel; LOKI_PATH_FASTEST is the older name of the same rule
    cases = (("C2", None, 256, B.LOKI_PATH_PREFIX), ("C2", None, 8, B.LOKI_PATH_PREFIX),
             ("SM", None, 1024, B.LOKI_PATH_PREFIX), ("C5", 2, 300, B.LOKI_PATH_PREFIX),
             ("C1", None, 1, B.LOKI_PATH_PREFIX))
    for name, v, m, want in cases:
        w = W.make_workload(name, v=v, n_levels=m)
        a = B.Allocator(w)
        try:
            assert a.info().path_current == B.LOKI_PATH_AUTO and a.info().path_auto == B.LOKI_PATH_DIRECT
            got = [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
            assert a.info().path_last == want
            # tiles: the hoisted kernel takes 128 levels where the sweep has them and the table fits
            if m >= 128:
                assert a.info().level_tile_last == (128 if name != "C5" else 64)
            assert_same(w, got, oracle.solve(w, n_threads=NCPU), w.demand_mqps, check=False)
            a.set_path(B.LOKI_PATH_FASTEST)
            a.solve(w.demand_mqps)
            assert a.info().path_current == B.LOKI_PATH_FASTEST and a.info().path_last == want
        finally:
            a.close()
    w = W.make_workload("C4", n_levels=64)
    a = B.Allocator(w)
    try:
        a.solve(w.demand_mqps)
        assert a.info().path_last == B.LOKI_PATH_PREFIX
        a.solve(w.demand_mqps[:8])
        assert a.info().path_last == B.LOKI_PATH_DIRECT
        a.set_path(B.LOKI_PATH_DIRECT)
        a.solve(w.demand_mqps)
        assert a.info().path_last == B.LOKI_PATH_DIRECT and a.info().path_current == B.LOKI_PATH_DIRECT
    finally:
        a.close()


def test_random_chains_and_trees_on_the_level_lane_kernels():
    # three and more tasks take the hoisted kernel's joint inner loop (trees: with the check of the
    # paths that bypass task 1); sweeps of 20, 64, 100 and 300 levels take its 32-, 64- and 128-level
    # tiles (the root-first kernel's: 32 and 64), the last one with a ragged final tile
    n_run = 0
    for seed in range(24):
        rnd = random.Random(7000 + seed)
        T = rnd.randint(3, 6)
        split = seed % 5 == 4
        if split:
            T = 3
        w = W.random_workload(7100 + seed, n_tasks=T, n_variants=[rnd.randint(1, 2 if split else 4) for _ in range(T)],
                              batch_sizes=sorted(rnd.sample([1, 2, 4, 8, 16], rnd.randint(1, 2 if split else 3))),
                              split_mode=int(split), n_levels=[20, 64, 100, 300][seed % 4], chain=seed < 16,
                              fan_fractional=seed % 2 == 0)
        w.demand_mqps[0] = 0
        ref = oracle.solve(w, n_threads=NCPU)
        a = B.Allocator(w)
        try:
            info = a.info()
            for path in (B.LOKI_PATH_HOISTED, B.LOKI_PATH_PREFIX, B.LOKI_PATH_SHARED, B.LOKI_PATH_UNIFORM):
                if path == B.LOKI_PATH_SHARED and not shared_tables_ok(a):
                    continue
                if (not info.direct_ok or (path in (B.LOKI_PATH_HOISTED, B.LOKI_PATH_PREFIX) and not info.hoisted_ok)
                        or (path == B.LOKI_PATH_UNIFORM and not info.uniform_ok)):
                    continue
                a.set_path(path)
                got = [B.config_to_dict(c, w.n_tasks) for c in a.solve(w.demand_mqps)]
                assert_same(w, got, ref, w.demand_mqps, check=False)
                n_run += 1
        finally:
            a.close()
    assert n_run >= 36
