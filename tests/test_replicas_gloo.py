"""The N > 1 path of the benchmark is N independent replicas: no collective on the data path, only the
aggregation of the per-rank figures.  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seeds = [bench.rank_seed(rank, s) for s in range(5)]
    ms, moved = bench.aggregate_over_ranks(dist, 10.0 + 5.0 * rank, 1000 * (rank + 1), "cpu")
    gathered = [None] * world
    dist.all_gather_object(gathered, seeds)
    if rank == 0:
        out.put((ms, moved, gathered))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_total_bytes():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, moved, seeds = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 15.0 and moved == 3000
    assert not set(seeds[0]) & set(seeds[1])


def test_replica_batches_differ_between_ranks():
    sys.path.insert(0, ROOT)
    import argparse
    import numpy as np
    import bench
    args = argparse.Namespace(requests=128, hbm_gb=1.0, host_gb=1.0)
    a = bench.make_batch(args, bench.rank_seed(0, 0))
    b = bench.make_batch(args, bench.rank_seed(1, 0))
    assert not np.array_equal(a.reqs["prompt"], b.reqs["prompt"])
