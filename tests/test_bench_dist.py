"""The multi-rank part of bench.py on CPU: two gloo ranks reduce their step time
to the maximum and report whole-job throughput over replicas."""
import os
import sys

import pytest
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
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    max_ms = bench.reduce_max(local_ms, world)
    value = bench.aggregate_value(1000.0, world, max_ms)
    out[rank] = (max_ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregation():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        for rank in range(world):
            max_ms, value = out[rank]
            assert max_ms == pytest.approx(15.0)
            assert value == pytest.approx(1000.0 * 2 / 15e-3)


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5, 1) == 3.5
    assert bench.aggregate_value(10.0, 1, 2.0) == pytest.approx(5000.0)
    assert bench.dist_env() == (int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)),
                                int(os.environ.get("WORLD_SIZE", 1)))
