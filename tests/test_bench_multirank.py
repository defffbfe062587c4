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


def test_rotation_sets_cover_l2_or_fall_back_to_flushing():
    """Timed steps rotate through operand sets so that a set has left L2 before its next use: the sets touched in
    between must exceed the L2 size; a working set too small for a reasonable number of copies is flushed instead."""
    sys.path.insert(0, ROOT)
    import bench
    assert bench.rotation_sets(84e6) == 3            # the 8192 x 8192 4x GEMV: two other sets = 168 MB > L2
    assert bench.rotation_sets(400e6) == 2           # larger than L2 by itself: one other set is enough
    assert bench.rotation_sets(1e6) == 1             # would need > 12 copies: timed one launch at a time after a flush
    for ws in (15e6, 30e6, 60e6, 100e6, 200e6):
        n = bench.rotation_sets(ws)
        assert n == 1 or (n - 1) * ws >= bench.L2_BYTES, (ws, n)
