"""The N > 1 path on CPU (gloo, world size 2).  The path does not shard and has no data-path
collective: ranks are independent replicas, and the only cross-rank step is the max over ranks of
the device-measured times that the benchmark reports.  These tests run that glue as two real
processes, and check that the reference arm leaves ranks other than 0 without work."""
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + rank, 3.0 - rank, 0.5, 7.0 * (rank + 1), 1.0]
        got = bench.max_over_ranks(mine, dist, "cpu")
        dist.barrier()
        out[rank] = (got, bench.job_throughput(world, 2048, got[0] / 10))
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_job_throughput_with_two_gloo_ranks():
    mgr = mp.Manager()
    out = mgr.dict()
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0][0] == out[1][0] == [11.0, 3.0, 0.5, 14.0, 1.0]  # slowest rank per entry, same on every rank
    # two ranks, 2048 tokens each per step, 1.1 ms per step
    assert abs(out[0][1] - 2 * 2048 / 1.1e-3) < 1e-6 * out[0][1]


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 0 and p.stdout.strip() == ""
