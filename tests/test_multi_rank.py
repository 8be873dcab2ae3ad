"""The N > 1 path of bench.py on CPU: two gloo ranks, independent replicas, the
job's step time is the slowest rank's and its throughput counts every replica."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    my_ms = 2.0 + rank          # rank 1 is the slow one
    ms = bench.max_over_ranks(my_ms, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.whole_job_tflops(world, 10**12, ms))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_all_the_work():
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, tflops = res[0]
    assert ms == 3.0
    assert tflops == pytest.approx(2 * 1.0 / 3e-3)


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(1.5, torch.device("cpu")) == 1.5
    assert bench.whole_job_tflops(1, 2 * 10**12, 1.0) == pytest.approx(2000.0)
