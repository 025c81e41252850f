"""The benchmark's multi-rank bookkeeping with two gloo ranks on CPU: independent batches per rank, the
slowest rank's time decides, the value counts every rank's tokens.  (The data path has no collective.)"""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)

    def rmax(x):
        t = torch.tensor([x], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    local_ms = 10.0 if rank == 0 else 25.0          # rank 1 is the slow one
    total_ms, value = bench.aggregate_over_ranks(local_ms, tokens_per_rank_step=1000, steps=5, world=world, reduce_max=rmax)
    seeds = [None] * world
    dist.all_gather_object(seeds, bench.rank_seed(2024, rank))
    out[rank] = (total_ms, value, seeds)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, 29581, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        total_ms, value, seeds = res[rank]
        assert total_ms == 25.0
        assert abs(value - 1000 * 2 * 5 / 0.025) < 1e-6
        assert seeds == [2024, 2025]
