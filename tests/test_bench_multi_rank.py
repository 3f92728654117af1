"""World-size-2 check (gloo, CPU) of the multi-rank arithmetic of bench.py: replicas run
independently, the reported time is the slowest rank's and the value is the whole-job aggregate."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 3.0 + 2.0 * rank                                # rank 1 is the slow one
    ms_max = bench.max_over_ranks(ms, dist, "cpu")
    out[rank] = (ms_max, bench.job_throughput(1000.0, world, ms_max))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate_value():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms_max, value = res[0]
    assert ms_max == 5.0
    assert abs(value - 2 * 1000.0 / 5.0e-3) < 1e-6


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(2.5, None, "cpu") == 2.5
    assert bench.job_throughput(10.0, 1, 2.0) == 5000.0
