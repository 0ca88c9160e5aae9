"""CPU oracle of the Load Balancer's request routing (MostAccurateFirst,
Algorithm 1 of Section 5.1).  Test infrastructure only: imported by ``tests/``
and by ``__graft_entry__.smoke``; never by the product package.  It shares no
code with the CUDA path.

Input: the pipeline tree and profiles of a workload, one demand level (root QPS)
and the allocation plan of that level (per task one or two groups of identical
workers, each group hosting one (variant, batch size)).  Output: the routing
tables -- for the Frontend and for every worker, per child task the list of
(child worker, routing probability) -- plus, per worker, its capacity, the
requests routed to it and its leftover capacity (the list the paper hands to
upstream workers for opportunistic rerouting).

The steps follow Algorithm 1 in the paper's order, in IEEE double arithmetic
(Python floats: no fused multiply-add), one rounded operation per line:

* tasks in topological order (task index order: ``parent[i] < i``);
* the workers of a task in non-increasing order of single-model accuracy
  (reading: equal accuracies -- the two groups of a same-variant split -- keep
  the plan's group order; workers of one group are interchangeable and keep
  their index order);
* the Frontend is the parent of the root task: one virtual worker (id -1) whose
  outgoing requests are the level's demand in queries per second;
* for worker ``u`` of task ``i`` and child ``c``:
  ``outgoing = u.incoming * multFactor * branchRatio`` where ``branchRatio`` is
  the per-edge factor ``fanout_milli[c] / 1000`` and ``multFactor`` the
  per-variant factor ``variant_fanout_milli / 1000`` of the variant ``u`` hosts
  (1 when the workload has none);
* the child's workers in sorted order: while ``capacity > 0`` and
  ``outgoing > 0`` route ``min(outgoing, capacity)`` with probability
  ``routed / totalChildDemand``;
* capacity of a worker hosting (variant v, batch b): its peak throughput
  ``q = b / l`` (Eq. 5) in queries per second, ``b * 1e6 / lat_us(v, b)``.

Requests that find no capacity (possible only by rounding, or when the plan was
made for a lower demand) are summed in ``unrouted_qps``.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List


@dataclass
class RouteWorker:
    task: int
    variant: int
    batch: int
    capacity_qps: float        # Eq. 5
    incoming_qps: float = 0.0
    leftover_qps: float = 0.0  # capacity not used by the routing


@dataclass
class RouteResult:
    status: int                                  # 0 routed, 1 the level has no plan
    workers: List[RouteWorker] = field(default_factory=list)
    entries: List[tuple] = field(default_factory=list)   # (src worker or -1, dst worker, probability)
    unrouted_qps: float = 0.0


def _sorted_groups(w, plan: dict, task: int):
    """Worker groups of a task in non-increasing accuracy of the hosted variant."""
    first = sum(w.n_variants[:task])
    groups = []
    n_groups = 1 if plan["split_k"][task] == 16 else 2
    for s in range(n_groups):
        v = plan["variant"][task][s]
        groups.append((s, v, plan["batch"][task][s], plan["workers"][task][s], w.accuracy[first + v]))
    # stable sort: equal accuracies keep the plan's order
    groups.sort(key=lambda g: -g[4])
    return groups


def route(w, demand_mqps: int, plan: dict) -> RouteResult:
    """MostAccurateFirst for one demand level.  ``plan`` is the dictionary view of
    an allocation (``variant``, ``batch``, ``workers``, ``split_k`` per task,
    ``status``) as produced by either implementation of the allocation search."""
    if plan["status"] != 0:
        return RouteResult(status=1)
    T = w.n_tasks
    nb = len(w.batch_sizes)
    first = [sum(w.n_variants[:i]) for i in range(T)]
    vfan = getattr(w, "variant_fanout_milli", None)
    res = RouteResult(status=0)
    task_workers: List[List[int]] = [[] for _ in range(T)]     # sorted worker ids per task
    remaining: List[float] = []                                # capacity left per worker
    for i in range(T):
        for (_s, v, b, n, _a) in _sorted_groups(w, plan, i):
            bi = w.batch_sizes.index(b)
            lat = w.latency_us[(first[i] + v) * nb + bi]
            cap = (float(b) * 1e6) / float(lat)
            for _ in range(n):
                task_workers[i].append(len(res.workers))
                res.workers.append(RouteWorker(task=i, variant=v, batch=b, capacity_qps=cap))
                remaining.append(cap)
    children: List[List[int]] = [[] for _ in range(T)]
    for i in range(1, T):
        children[w.parent[i]].append(i)

    def fill(src: int, child: int, outgoing: float):
        total = outgoing
        for cw in task_workers[child]:
            if remaining[cw] > 0.0 and outgoing > 0.0:
                routed = min(outgoing, remaining[cw])
                res.entries.append((src, cw, routed / total))
                outgoing = outgoing - routed
                remaining[cw] = remaining[cw] - routed
                res.workers[cw].incoming_qps = res.workers[cw].incoming_qps + routed
        if outgoing > 0.0:
            res.unrouted_qps = res.unrouted_qps + outgoing

    fill(-1, 0, float(demand_mqps) / 1000.0)                   # the Frontend's table
    for i in range(T):
        for u in task_workers[i]:
            wk = res.workers[u]
            mult = 1.0 if vfan is None else float(vfan[first[i] + wk.variant]) / 1000.0
            for c in children[i]:
                branch = float(w.fanout_milli[c]) / 1000.0
                outgoing = (wk.incoming_qps * mult) * branch
                fill(u, c, outgoing)
    for k, wk in enumerate(res.workers):
        wk.leftover_qps = remaining[k]
    return res
