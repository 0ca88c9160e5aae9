"""Independent brute-force search for tiny allocation problems (pure Python).

Written separately from ``oracle/`` and in a different shape -- explicit option
lists built with ``itertools.combinations``, a recursive walk over the tasks,
exact rationals for every ceiling -- so that a mistake in the oracle's index
arithmetic, option numbering, rounding or tie-breaking does not repeat here.
Python floats are IEEE doubles and ``a * b`` is a single rounded multiply, so
accuracies agree with the oracle bit for bit.

Follows Section 4.1 of the paper: Eq. 1 (stage demand), Eq. 2 with Eq. 5
(workers), Eq. 3 (cluster), Eqs. 6-7 with the halved SLO (latency), the
objective of Eqs. 8-12 as one lexicographic order.
"""
from __future__ import annotations

import itertools
from fractions import Fraction
from typing import List, Optional, Tuple


def ceil_frac(x: Fraction) -> int:
    return -((-x.numerator) // x.denominator)


def task_options(w, task: int) -> List[Tuple]:
    """Every option of a task in index order:
    ``(accuracy, latency, [(share_16ths, lat_us, batch, variant), ...], factor)``."""
    nb = len(w.batch_sizes)
    first = sum(w.n_variants[:task])
    vfan = getattr(w, "variant_fanout_milli", None)
    singles = []
    for v in range(w.n_variants[task]):
        for bi in range(nb):
            singles.append((v, w.batch_sizes[bi], w.latency_us[(first + v) * nb + bi],
                            w.accuracy[first + v], 1000 if vfan is None else vfan[first + v]))
    # fourth entry: the option's multiplicative factor as a rational (share-weighted mean)
    opts = [(s[3], s[2], [(16, s[2], s[1], s[0])], Fraction(s[4], 1000)) for s in singles]
    if w.split_mode:
        for s1, s2 in itertools.combinations(singles, 2):      # lexicographic pairs
            for k in range(1, 16):
                a = s2[3] + (k * 0.0625) * (s1[3] - s2[3])
                opts.append((a, max(s1[2], s2[2]),
                             [(k, s1[2], s1[1], s1[0]), (16 - k, s2[2], s2[1], s2[0])],
                             Fraction(k * s1[4] + (16 - k) * s2[4], 16000)))
    return opts


def solve_level(w, demand_mqps: int) -> Optional[dict]:
    """Best plan for one demand level, or ``None`` if nothing is feasible."""
    T = w.n_tasks
    children = [[j for j in range(T) if w.parent[j] == i] for i in range(T)]
    leaves = [i for i in range(T) if not children[i]]
    opts = [task_options(w, i) for i in range(T)]
    stride = [1] * T
    for i in range(1, T):
        stride[i] = stride[i - 1] * len(opts[i - 1])
    def stage_demands(chosen):
        # exact, ceiling on every edge; the parent's option contributes its factor
        dem = [0] * T
        dem[0] = demand_mqps
        for i in range(1, T):
            u = w.parent[i]
            dem[i] = ceil_frac(dem[u] * Fraction(w.fanout_milli[i], 1000) * opts[u][chosen[u]][3])
        return dem

    best = None  # (accuracy, -workers, -index)
    best_plan = None

    def walk(i: int, chosen: List[int]):
        nonlocal best, best_plan
        if i == T:
            # latency on every root-to-leaf path
            for leaf in leaves:
                tot, hops, j = 0, 0, leaf
                while j != -1:
                    tot += opts[j][chosen[j]][1]
                    hops += 1
                    j = w.parent[j]
                if 2 * tot > w.slo_us - hops * w.comm_us:
                    return
            dem = stage_demands(chosen)
            workers = []
            for j in range(T):
                per = []
                for share, lat, b, _v in opts[j][chosen[j]][2]:
                    per.append(ceil_frac(Fraction(dem[j] * share * lat, 16 * b * 10 ** 9)))
                workers.append(per)
            total = sum(sum(p) for p in workers)
            if total > w.cluster_size:
                return
            prod = [0.0] * T
            for j in range(T):
                aj = opts[j][chosen[j]][0]
                prod[j] = aj if j == 0 else prod[w.parent[j]] * aj
            s = None
            for leaf in leaves:
                s = prod[leaf] if s is None else s + prod[leaf]
            acc = s / float(len(leaves))
            index = sum(chosen[j] * stride[j] for j in range(T))
            key = (acc, -total, -index)
            if best is None or key > best:
                best = key
                best_plan = {"cand_index": index, "accuracy": acc, "total_workers": total,
                             "workers": workers, "choice": list(chosen)}
            return
        for o in range(len(opts[i])):
            chosen.append(o)
            walk(i + 1, chosen)
            chosen.pop()

    walk(0, [])
    return best_plan


def solve(w, demands=None) -> List[Optional[dict]]:
    return [solve_level(w, d) for d in (w.demand_mqps if demands is None else demands)]
