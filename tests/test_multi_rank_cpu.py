"""The N > 1 path of the benchmark on CPU: two gloo ranks shard a demand sweep by
level (no data-path collective) and agree on the slowest rank's time."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2407_03583_b200 import workloads as W


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.shard_sweep("C2", rank, world)
        mine = torch.tensor(w.demand_mqps, dtype=torch.int64)
        gathered = [torch.empty_like(mine) for _ in range(world)]
        dist.all_gather(gathered, mine)
        t = torch.tensor([10.0 + 5.0 * rank], dtype=torch.float64)     # pretend step times
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        if rank == 0:
            out.put(([g.tolist() for g in gathered], float(t), w.max_demand_mqps, w.n_levels))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_the_sweep_and_take_the_max_time():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    shards, t_max, max_dem, n_levels = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    base = W.make_workload("C2")
    big = W.make_workload("C2", n_levels=base.n_levels * world)
    assert n_levels == base.n_levels and all(len(s) == base.n_levels for s in shards)
    # the shards are disjoint and together are exactly the longer sweep
    merged = [None] * len(big.demand_mqps)
    for r, s in enumerate(shards):
        merged[r::world] = s
    assert merged == big.demand_mqps
    assert max_dem == max(big.demand_mqps)
    assert t_max == 15.0


def test_single_rank_is_the_named_workload():
    assert W.shard_sweep("C4", 0, 1).checksum() == W.make_workload("C4").checksum()
