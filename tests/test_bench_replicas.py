"""Multi-GPU runs are independent replicas (batch-1 decode does not shard): the only cross-rank logic is the
MAX-over-ranks timing of bench.py.  Exercised here with two gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    # rank 1 is the slow replica: the job's time is its time, the job's tokens are both ranks' tokens
    value, e2e, ms = bench.replica_throughput(512, 1000.0 * (1 + rank), 1.5 * (1 + rank), dist, "cpu")
    out[rank] = (value, e2e, ms)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_throughput_takes_the_max_over_ranks():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29500 + os.getpid() % 2000, out), nprocs=world, join=True)
    for r in range(world):
        value, e2e, ms = out[r]
        assert ms == 2000.0
        assert abs(value - 2 * 512 / 2.0) < 1e-9 and abs(e2e - 2 * 512 / 3.0) < 1e-9


def test_single_rank_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.replica_throughput(100, 500.0, 1.0) == (200.0, 100.0, 500.0)
