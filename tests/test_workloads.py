"""Input generators: the PRNG against its published test vector, and the five
named workloads against the sizes the benchmark definition states."""
from paper_2407_03583_b200 import workloads as W


def test_splitmix64_reference_vector():
    # first outputs for seed 1234567 of the public-domain reference implementation
    rng = W.SplitMix64(1234567)
    assert [rng.next_u64() for _ in range(5)] == [
        6457827717110365317, 3203168211198807973, 9817491932198370423,
        4593380528125082431, 16408922859458223821]


def test_named_workload_sizes():
    expect = {"C1": (256, 1), "C2": (110592, 256), "C3": (24010000, 4096),
              "C4": (24300000, 64), "C5": (17338896, 1024)}
    for name, (n, m) in expect.items():
        w = W.make_workload(name)
        assert (w.n_candidates(), w.n_levels) == (n, m)
        assert w.options_per_task()[0] == {"C1": 16, "C2": 48, "C3": 70, "C4": 30, "C5": 4164}[name]
        assert all(d >= 1 for d in w.demand_mqps)
        assert w.parent[0] == -1 and all(0 <= w.parent[i] < i for i in range(1, w.n_tasks))


def test_profiles_are_sorted_and_co_monotone():
    for name in W.WORKLOAD_NAMES:
        w = W.make_workload(name)
        nb = len(w.batch_sizes)
        off = 0
        for v in w.n_variants:
            acc = w.accuracy[off:off + v]
            assert acc == sorted(acc) and len(set(acc)) == v
            assert all(0.60 <= a <= 0.95 for a in acc)
            for bi in range(nb):
                col = [w.latency_us[(off + k) * nb + bi] for k in range(v)]
                assert col == sorted(col)
            off += v
        assert max(w.latency_us) <= 20000 + 8000 * 64


def test_demand_shapes():
    c2 = W.make_workload("C2")
    assert c2.demand_mqps[0] == 50_000 and c2.demand_mqps[-1] == 5_000_000
    c4 = W.make_workload("C4")
    assert c4.demand_mqps[0] == 100_000 and c4.demand_mqps[-1] == 20_000_000
    c3 = W.make_workload("C3")
    assert min(c3.demand_mqps) < 130_000 and 7_500_000 < max(c3.demand_mqps) < 9_700_000
    c5 = W.make_workload("C5")
    assert c5.demand_mqps[0] == 100_000 and c5.demand_mqps[-1] == 10_000_000


def test_generation_is_deterministic():
    a = W.make_workload("C3", n_levels=128)
    b = W.make_workload("C3", n_levels=128)
    assert a.checksum() == b.checksum()
    assert a.checksum() != W.make_workload("C3", n_levels=127).checksum()


def test_social_media_shaped_workload():
    w = W.make_workload("SM")
    assert (w.parent, w.n_variants, w.fanout_milli) == ([-1, 0], [5, 4], [1000, 1000])
    assert (w.n_candidates(), w.n_levels) == (25 * 20, 1024)
    # bursts stand out of the diurnal curve
    assert max(w.demand_mqps[96::97]) > 1.2 * max(w.demand_mqps[95::97])
    assert 50_000 < min(w.demand_mqps) < 600_000 and 4_000_000 < max(w.demand_mqps) < 9_000_000
