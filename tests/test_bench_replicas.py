"""bench.py with N > 1 runs N independent replicas (the path has no exchange step): the only
multi-rank logic is the max-over-ranks timing and the aggregate.  Checked here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench

    def reduce_max(v):
        t = torch.tensor([v], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    local = 0.010 if rank == 0 else 0.025  # the slow rank sets the job's time
    value, elapsed = bench.aggregate_replicas(ops_per_step=1e12, steps=5, elapsed_local_s=local, world=world,
                                              reduce_max=reduce_max)
    dist.barrier()
    out[rank] = (value, elapsed)
    dist.destroy_process_group()


def test_two_replicas_aggregate_over_the_slowest_rank():
    world, port = 2, 29611
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    value, elapsed = res[0]
    assert elapsed == 0.025
    assert abs(value - 2 * 1e12 * 5 / 0.025 / 1e12) < 1e-9
