"""The multi-GPU contract of the benchmark is "replicas only": every rank runs the same layers, the job is charged
the slowest rank's time and credited the sum of the work.  The two helpers that implement this are exercised here
with two gloo ranks on the CPU (the GPU run uses the same code over NCCL)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))  # rank 1 is the slow one
    dist.barrier()
    out[rank] = (ms, bench.whole_job_tops(world, 2.0e12, ms))
    dist.destroy_process_group()


def test_two_ranks_are_charged_the_slowest_time_and_credited_both_works():
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(2, 29541, out), nprocs=2, join=True)
        assert out[0] == out[1]
        ms, tops = out[0]
        assert ms == 15.0
        assert abs(tops - 2 * 2.0e12 / 15.0e-3 / 1e12) < 1e-9


def test_single_rank_passes_through():
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.whole_job_tops(1, 1.0e12, 1000.0) == 1.0  # 1e12 ops in 1000 ms
