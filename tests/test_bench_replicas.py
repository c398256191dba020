"""bench.py's multi-GPU figure: N independent replicas (the path does not shard), MAX over ranks, value = time / N.
Run as two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    total_ms = 100.0 if rank == 0 else 160.0           # rank 1 is the slower replica
    e2e_ms = 12.0 if rank == 0 else 11.0
    ms_per_step, value, e2e = bench.aggregate(total_ms, e2e_ms, 10, world, "cpu")
    out[rank] = (ms_per_step, value, e2e)
    dist.destroy_process_group()


def test_replica_aggregation_takes_the_slowest_rank_and_divides_by_world():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            ms_per_step, value, e2e = out[rank]
            assert ms_per_step == 16.0 and value == 8.0 and e2e == 6.0


def test_single_rank_aggregation_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate(50.0, 7.0, 5, 1, "cpu") == (10.0, 10.0, 7.0)
