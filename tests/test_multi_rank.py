"""The multi-GPU run is N independent replicas (the path has no exchange step): the only thing ranks share is
the timing reduction of the benchmark. Two gloo ranks on the CPU check that reduction and the whole-job rate."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local = 10.0 + 5.0 * rank                    # rank 1 is the slow one
    slowest = bench.max_over_ranks(local, world)
    rate = bench.whole_job_rate(8192, 4, world, slowest * 1e-3)
    dist.barrier()
    out[rank] = (slowest, rate)
    dist.destroy_process_group()


def test_two_ranks_agree_on_slowest_time_and_whole_job_rate():
    world, port = 2, 29500 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_rank_main, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1]
        slowest, rate = out[0]
        assert slowest == 15.0
        assert rate == 8192 * 4 * 2 / 15e-3


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_rate(100, 2, 1, 0.5) == 400.0
