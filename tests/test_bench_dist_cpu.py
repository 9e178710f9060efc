"""The multi-GPU plumbing of bench.py on CPU: two gloo ranks, replicas only.

The path has no exchange step, so N ranks are N independent replicas; the only
cross-rank logic is the timing rule (max of the elapsed time over ranks, sum of the
events served).  That helper is exercised here with world_size 2."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank: int, world: int, port: int, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        elapsed = 0.010 * (rank + 1)            # rank 1 is the slow one
        t, n = bench.reduce_max_time(elapsed, 100 + rank, dist)
        out[rank] = (t, n)
    finally:
        dist.destroy_process_group()


def test_max_time_and_total_events_over_two_ranks():
    port = 29500 + (os.getpid() % 2000)
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        assert dict(out) == {0: (0.020, 201), 1: (0.020, 201)}


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max_time(0.5, 7, None) == (0.5, 7)


def test_algorithmic_bytes_formula():
    sys.path.insert(0, ROOT)
    import bench
    ab = bench.algorithmic_bytes_per_event(25_557_032, 25_558, 25_558, 32)
    assert ab["push"] == 12 * 25_557_032 + 8 * 25_558
    assert ab["apply"] == 8 * 25_558 * 33 + 8 * 25_558
    assert ab["pull"] == 4 * 25_557_032 + 12 * 25_558
    assert abs(ab["total"] - 416.4e6) < 0.1e6
