"""bench.py runs N independent replicas (the drafting step has no collective): the job's
throughput is the units of all ranks over the slowest rank's time.  Checked here with two
gloo ranks on CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    seconds = 2.0 if rank == 0 else 5.0            # rank 1 is the slow one
    value, t = bench.replica_throughput(dist, torch.device("cpu"), 1000, seconds)
    out[rank] = (value, t)
    dist.destroy_process_group()


def test_replica_throughput_uses_the_slowest_rank():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank, args=(world, port, out), nprocs=world, join=True)
        for r in range(world):
            value, t = out[r]
            assert t == 5.0
            assert abs(value - 2 * 1000 / 5.0) < 1e-9


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    value, t = bench.replica_throughput(None, torch.device("cpu"), 12, 0.5)
    assert value == 24.0 and t == 0.5
