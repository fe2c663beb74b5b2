"""bench.py with more than one GPU runs independent replicas: the only cross-rank logic is the
max-over-ranks of the timed interval and the aggregation of the value.  Both are exercised here
with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(100.0 + 50.0 * rank, dist, "cpu")      # rank 1 is the slow replica
    dist.barrier()
    out[rank] = (ms, bench.aggregate_value(20, ms, world))
    dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_aggregate_rate():
    world, port = 2, 29000 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1]
        ms, value = out[0]
        assert ms == 150.0
        assert abs(value - 2 * 20 / 0.150) < 1e-9


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(12.5, None, "cpu") == 12.5
    assert abs(bench.aggregate_value(10, 500.0, 1) - 20.0) < 1e-12
