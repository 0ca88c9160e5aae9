"""Seeded synthetic allocation problems (inputs only).

This module produces the *inputs* of the allocation search: a pipeline tree,
per-variant accuracy and per-(variant, batch) latency profiles, an SLO, a
cluster size and a demand sweep.  It contains none of the method's arithmetic
(no accuracy products, no worker counts, no argmax) and is the one module that
both the CPU oracle's tests and the CUDA path's tests/bench may import.

The paper evaluates on production demand traces and profiled model families
(Section 6.1, "Pipelines" and "Datasets"); neither is available, so the five
named workloads below stand in for their *shape*: profiles where a more
accurate variant is slower (cf. the accuracy/throughput figure of Section 2.1),
integer fan-out per edge (the multiplicative factors of Section 4.1), and demand
sweeps that are linear, log-uniform, or a noisy diurnal sine.

Random numbers: one SplitMix64 stream per workload, seeded with the workload's
seed.  Draw order: for each task in index order its accuracies, then its
latency intercepts, then its latency slopes; then one fan-out per edge in task
order; then the demand noise.  A uniform double is ``(x >> 11) * 2**-53``; a
uniform integer in ``[lo, hi]`` is ``lo + x % (hi - lo + 1)``; a standard
normal is Box-Muller on two uniforms.
"""
from __future__ import annotations

import math
import struct
from dataclasses import dataclass, field
from typing import List, Sequence

MASK64 = (1 << 64) - 1


class SplitMix64:
    """SplitMix64 (Steele, Lea, Flood 2014): a 64-bit counter-based generator."""

    def __init__(self, seed: int):
        self.state = seed & MASK64

    def next_u64(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & MASK64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
        return z ^ (z >> 31)

    def uniform(self) -> float:
        """Uniform double in [0, 1)."""
        return (self.next_u64() >> 11) * (2.0 ** -53)

    def randint(self, lo: int, hi: int) -> int:
        """Uniform integer in [lo, hi] (modulo reduction)."""
        return lo + self.next_u64() % (hi - lo + 1)

    def normal(self) -> float:
        """Standard normal by Box-Muller (cosine branch)."""
        u1 = ((self.next_u64() >> 11) + 1) * (2.0 ** -53)  # (0, 1]
        u2 = self.uniform()
        return math.sqrt(-2.0 * math.log(u1)) * math.cos(2.0 * math.pi * u2)


@dataclass
class Workload:
    """One allocation problem plus a demand sweep.

    ``accuracy`` is task-major (all variants of task 0, then task 1, ...);
    ``latency_us`` is ``[sum(n_variants)][len(batch_sizes)]`` flattened
    row-major.  ``demand_mqps`` is in milli-queries per second.
    """

    name: str
    parent: List[int]
    fanout_milli: List[int]
    n_variants: List[int]
    batch_sizes: List[int]
    accuracy: List[float]
    latency_us: List[int]
    slo_us: int
    comm_us: int
    cluster_size: int
    split_mode: int
    demand_mqps: List[int]
    max_demand_mqps: int = 0
    seed: int = 0
    note: str = ""
    # optional per-variant multiplicative factor r(i,k) in thousandths (task-major,
    # like ``accuracy``); None means 1000 for every variant
    variant_fanout_milli: List[int] | None = None
    _checksum: int = field(default=0, repr=False)

    def __post_init__(self):
        if self.max_demand_mqps <= 0:
            self.max_demand_mqps = max(self.demand_mqps) if self.demand_mqps else 1

    @property
    def n_tasks(self) -> int:
        return len(self.parent)

    @property
    def n_levels(self) -> int:
        return len(self.demand_mqps)

    def options_per_task(self) -> List[int]:
        """Number of options of each task (single options, plus 15 splits per
        unordered pair of distinct single options in split mode)."""
        out = []
        nb = len(self.batch_sizes)
        for v in self.n_variants:
            ns = v * nb
            out.append(ns + (ns * (ns - 1) // 2) * 15 if self.split_mode else ns)
        return out

    def n_candidates(self) -> int:
        n = 1
        for o in self.options_per_task():
            n *= o
        return n

    def with_demands(self, demand_mqps: Sequence[int], name: str | None = None) -> "Workload":
        w = Workload(**{k: getattr(self, k) for k in (
            "name", "parent", "fanout_milli", "n_variants", "batch_sizes", "accuracy",
            "latency_us", "slo_us", "comm_us", "cluster_size", "split_mode")},
            demand_mqps=list(demand_mqps), max_demand_mqps=self.max_demand_mqps,
            seed=self.seed, note=self.note,
            variant_fanout_milli=None if self.variant_fanout_milli is None else list(self.variant_fanout_milli))
        if name:
            w.name = name
        return w

    def checksum(self) -> int:
        """FNV-1a (64-bit) over a canonical little-endian serialisation."""
        if self._checksum:
            return self._checksum
        h = 0xCBF29CE484222325

        def feed(b: bytes):
            nonlocal h
            for byte in b:
                h ^= byte
                h = (h * 0x100000001B3) & MASK64

        def ints(xs, fmt):
            feed(struct.pack("<q", len(xs)))
            feed(struct.pack("<%d%s" % (len(xs), fmt), *xs))

        ints(self.parent, "i")
        ints(self.fanout_milli, "i")
        ints(self.n_variants, "i")
        ints(self.batch_sizes, "i")
        ints(self.accuracy, "d")
        ints(self.latency_us, "q")
        ints([self.slo_us, self.comm_us, self.cluster_size, self.split_mode], "q")
        ints(self.demand_mqps, "q")
        if self.variant_fanout_milli is not None:
            ints(self.variant_fanout_milli, "i")
        self._checksum = h
        return h


def _profiles(rng: SplitMix64, n_variants: Sequence[int], batch_sizes: Sequence[int]):
    """Accuracies U[0.60, 0.95] sorted ascending (bit-equal draws are redrawn);
    latency ``a_v + c_v * b`` microseconds with ``a ~ U{2000..20000}`` and
    ``c ~ U{500..8000}``, each sorted ascending and assigned in accuracy order
    so that a more accurate variant is never faster."""
    accuracy: List[float] = []
    latency: List[int] = []
    for v in n_variants:
        accs: List[float] = []
        while len(accs) < v:
            a = 0.60 + 0.35 * rng.uniform()
            if a not in accs:
                accs.append(a)
        accs.sort()
        a0 = sorted(rng.randint(2000, 20000) for _ in range(v))
        c0 = sorted(rng.randint(500, 8000) for _ in range(v))
        accuracy.extend(accs)
        for k in range(v):
            for b in batch_sizes:
                latency.append(a0[k] + c0[k] * b)
    return accuracy, latency


def _fanouts(rng: SplitMix64, parent: Sequence[int], choices: Sequence[int]) -> List[int]:
    out = [1000]
    for _ in range(1, len(parent)):
        out.append(1000 * choices[rng.next_u64() % len(choices)])
    return out


def _to_mqps(qps: float) -> int:
    return max(1, int(math.floor(qps * 1000.0 + 0.5)))


def _linear(lo: float, hi: float, n: int) -> List[int]:
    if n == 1:
        return [_to_mqps(lo)]
    return [_to_mqps(lo + (hi - lo) * j / (n - 1)) for j in range(n)]


def make_workload(name: str, *, v: int | None = None, n_levels: int | None = None) -> Workload:
    """Build one of the named workloads ``C1`` .. ``C5`` or ``SM``.

    ``v`` overrides the number of variants per task and ``n_levels`` the length
    of the demand sweep (reduced-size parity cases keep everything else).
    """
    name = name.upper()
    if name == "C1":      # tiny 2-stage chain
        seed, parent, vv, bs = 0, [-1, 0], v or 4, [1, 2, 4, 8]
        rng = SplitMix64(seed)
        acc, lat = _profiles(rng, [vv] * 2, bs)
        fan = [1000, 1000]
        dem = _linear(200.0, 200.0, n_levels or 1)
        return Workload("C1", parent, fan, [vv] * 2, bs, acc, lat, 200_000, 0, 8, 0, dem,
                        seed=seed, note="2-stage chain, 1 level at 200 QPS")
    if name == "C2":      # 3-stage chain
        seed, parent, vv, bs = 1, [-1, 0, 1], v or 8, [1, 2, 4, 8, 16, 32]
        rng = SplitMix64(seed)
        acc, lat = _profiles(rng, [vv] * 3, bs)
        fan = _fanouts(rng, parent, [1, 2, 3])
        dem = _linear(50.0, 5000.0, n_levels or 256)
        return Workload("C2", parent, fan, [vv] * 3, bs, acc, lat, 300_000, 0, 64, 0, dem,
                        seed=seed, note="3-stage chain, linear sweep 50..5000 QPS")
    if name == "C3":      # 4-task tree, diurnal trace
        seed, parent, vv = 2, [-1, 0, 0, 1], v or 10
        bs = [1, 2, 4, 8, 16, 32, 64]
        rng = SplitMix64(seed)
        acc, lat = _profiles(rng, [vv] * 4, bs)
        fan = _fanouts(rng, parent, [2, 3, 4])
        m = n_levels or 4096
        dem = []
        for j in range(m):
            q = 4050.0 + 3950.0 * math.sin(2.0 * math.pi * j / m - math.pi / 2.0)
            q *= 1.0 + 0.05 * rng.normal()
            dem.append(_to_mqps(max(q, 0.001)))
        return Workload("C3", parent, fan, [vv] * 4, bs, acc, lat, 400_000, 0, 128, 0, dem,
                        seed=seed, note="detector -> {classifier -> leaf, recognizer}; noisy diurnal sine 100..8000 QPS")
    if name == "C4":      # 5-stage chain, log-uniform sweep
        seed, parent, vv, bs = 3, [-1, 0, 1, 2, 3], v or 6, [1, 2, 4, 8, 16]
        rng = SplitMix64(seed)
        acc, lat = _profiles(rng, [vv] * 5, bs)
        fan = _fanouts(rng, parent, [1, 2])
        m = n_levels or 64
        dem = [_to_mqps(100.0 * 200.0 ** (j / (m - 1) if m > 1 else 0.0)) for j in range(m)]
        return Workload("C4", parent, fan, [vv] * 5, bs, acc, lat, 500_000, 0, 256, 0, dem,
                        seed=seed, note="5-stage chain, log-uniform sweep 100..20000 QPS")
    if name == "C5":      # 2-stage chain, split mode
        seed, parent, vv, bs = 4, [-1, 0], v or 6, [1, 2, 4, 8]
        rng = SplitMix64(seed)
        acc, lat = _profiles(rng, [vv] * 2, bs)
        fan = _fanouts(rng, parent, [1, 2, 3])
        dem = _linear(100.0, 10000.0, n_levels or 1024)
        return Workload("C5", parent, fan, [vv] * 2, bs, acc, lat, 250_000, 0, 96, 1, dem,
                        seed=seed, note="2-stage chain, k/16 traffic splits, linear sweep 100..10000 QPS")
    if name == "SM":      # the paper's second pipeline shape: classify, then caption
        # Two tasks in a chain with model families of different sizes (the paper names a
        # ResNet family for classification and a CLIP-ViT family for captioning), every
        # image is captioned once (factor 1), and a bursty demand trace: a diurnal sine
        # with 10 % multiplicative noise and a 1.6x burst every 97th step, standing in for
        # the shape of the public tweet-arrival trace the paper replays.
        seed, parent, bs = 5, [-1, 0], [1, 2, 4, 8, 16]
        nv = [v or 5, max(1, (v or 5) - 1)]
        rng = SplitMix64(seed)
        acc, lat = _profiles(rng, nv, bs)
        fan = [1000, 1000]
        m = n_levels or 1024
        dem = []
        for j in range(m):
            q = 2100.0 + 1900.0 * math.sin(2.0 * math.pi * j / m - math.pi / 2.0)
            q *= 1.0 + 0.10 * rng.normal()
            if j % 97 == 96:
                q *= 1.6
            dem.append(_to_mqps(max(q, 0.001)))
        return Workload("SM", parent, fan, nv, bs, acc, lat, 300_000, 0, 48, 0, dem,
                        seed=seed, note="classifier -> captioner, bursty diurnal trace 200..4000 QPS")
    raise ValueError("unknown workload %r" % name)


# C1..C5 are the five benchmark configurations; SM is the second pipeline shape of the
# paper's evaluation (Section 6.1, "Pipelines").
WORKLOAD_NAMES = ("C1", "C2", "C3", "C4", "C5", "SM")


def shard_sweep(name: str, rank: int, world: int) -> Workload:
    """Rank ``rank``'s problem when ``world`` processes share the work by demand
    level: the sweep is drawn ``world`` times as long and dealt out round-robin,
    so every rank solves a sweep of the workload's own length over the same range
    (per-rank work is fixed: weak scaling, no data exchanged between ranks)."""
    base = make_workload(name)
    if world <= 1:
        return base
    big = make_workload(name, n_levels=base.n_levels * world)
    w = base.with_demands(big.demand_mqps[rank::world])
    w.max_demand_mqps = max(big.demand_mqps)
    return w


def random_workload(seed: int, *, n_tasks: int, n_variants: Sequence[int] | int,
                    batch_sizes: Sequence[int], split_mode: int = 0, n_levels: int = 4,
                    chain: bool = False, fan_choices: Sequence[int] = (1, 2, 3),
                    fan_fractional: bool = False, variant_fan: bool = False) -> Workload:
    """A small random instance: random rooted tree (``parent[i] < i``), random
    profiles, and SLO / cluster size / demands drawn so that sweeps cross from
    "everything feasible" to "nothing feasible".  ``fan_fractional`` draws
    fan-outs that are not whole multiples of 1000 milli-units."""
    rng = SplitMix64(0xA5A5_0000 + seed)
    parent = [-1]
    for i in range(1, n_tasks):
        parent.append(i - 1 if chain else int(rng.next_u64() % i))
    if isinstance(n_variants, int):
        n_variants = [n_variants] * n_tasks
    acc, lat = _profiles(rng, n_variants, batch_sizes)
    if fan_fractional:
        fan = [1000] + [int(rng.randint(300, 3500)) for _ in range(1, n_tasks)]
    else:
        fan = _fanouts(rng, parent, list(fan_choices))
    # depth of the deepest path decides a sensible SLO range
    depth = [1] * n_tasks
    for i in range(1, n_tasks):
        depth[i] = depth[parent[i]] + 1
    d = max(depth)
    slo = int(rng.randint(2 * 6000 * d, 2 * 45000 * d))
    cluster = int(rng.randint(2, 40))
    dem = []
    for _ in range(n_levels):
        e = rng.uniform() * 3.7          # 10**0 .. 10**3.7 QPS
        dem.append(_to_mqps(10.0 ** e))
    vfan = None
    if variant_fan:
        # a more accurate variant emits more downstream requests (Section 2.2.1, "workload multiplication")
        vfan = []
        for v in n_variants:
            vfan.extend(sorted(int(rng.randint(400, 2600)) for _ in range(v)))
    return Workload("R%d" % seed, parent, fan, list(n_variants), list(batch_sizes), acc, lat,
                    slo, 0, cluster, split_mode, dem, seed=seed, note="random small instance",
                    variant_fanout_milli=vfan)
