"""Multi-rank plumbing of the benchmark on CPU (gloo, world size 2): ranks draw
disjoint batches, the job time is the slowest rank's, the aggregate counts every
rank's updates.  Agents are independent, so there is no data-path collective to
test: only this bookkeeping."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    sys.path.insert(0, ROOT)
    import bench
    from biwl import make_config
    import oracle
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = make_config(bench.HEADLINE, N=6, T=3, seed=bench.rank_seed(rank))
    q, _, _ = oracle.run_workload(w)           # the rank's own shard, computed independently
    mine = 0.010 * (rank + 1)                   # pretend device time: rank 1 is the slow one
    sec = bench.max_over_ranks(dist, mine, "cpu")
    value = bench.aggregate_throughput(w.updates, world, sec)
    sums = torch.tensor([float(q.sum()), float(w.obs.sum())], dtype=torch.float64)
    gathered = [torch.zeros_like(sums) for _ in range(world)]
    dist.all_gather(gathered, sums)
    if rank == 0:
        out.put((sec, value, w.updates, [g.tolist() for g in gathered]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_sharding_and_aggregation():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    sec, value, updates, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert abs(sec - 0.020) < 1e-12                      # max over ranks, not rank 0's own time
    assert abs(value - updates * 2 / 0.020) < 1e-6       # whole-job aggregate
    assert gathered[0][1] != gathered[1][1]              # ranks drew different batches
    # every belief block sums to one: N*T*F per rank
    assert all(abs(g[0] - 6 * 3 * 3) < 1e-9 for g in gathered)
