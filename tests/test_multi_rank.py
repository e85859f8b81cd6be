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


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`python bench.py --gpus 2` with no launcher around it: the script spawns two ranks itself (here the stub step on
    gloo), rank 0 prints the one JSON line, n_gpus is the number of ranks that ran, the time is the slowest rank's."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "stub", "--steps", "5", "--warmup", "1"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["steps"] == 5
    assert out["ms_per_step"] >= 4.0          # rank 1 sleeps 4 ms per step, rank 0 only 2: the slowest rank counts
