"""The multi-GPU path of bench.py is "replicas only": every rank runs the same workload, no collective touches the
data, and the reported time is the slowest rank's.  The reduction and the aggregate are exercised here with two
CPU processes over gloo."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    total_ms, e2e_ms = bench.max_over_ranks([10.0 + 5.0 * rank, 30.0 - 2.0 * rank])
    value = bench.aggregate_value(2.0e9, 4, total_ms, world)
    out[rank] = (total_ms, e2e_ms, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_timing_is_the_slowest_ranks_and_value_sums_replicas():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        total_ms, e2e_ms, value = res[rank]
        assert total_ms == 15.0 and e2e_ms == 30.0  # max over ranks, element-wise
        assert value == pytest.approx(2 * 2.0e9 * 4 / 15.0e-3 / 1e9)


def test_single_process_reduction_is_the_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
