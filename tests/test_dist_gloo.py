"""The multi-rank plumbing of the benchmark on CPU (gloo, world size 2): replicas share nothing on
the data path; only the timings are reduced (slowest rank decides) and rank 0 reports."""
import json
import os
import subprocess
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = [10.0 + 5.0 * rank, 40.0 - 3.0 * rank]      # rank 1 slower on the first, rank 0 on the second
    red = bench.max_over_ranks(mine, "cpu")
    dist.barrier()
    out.put((rank, red, bench.job_throughput(world, 20, red[0])))
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_throughput():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    for rank, red, value in got:
        assert red == [15.0, 40.0]                      # element-wise maximum, identical on both ranks
        assert abs(value - 2 * 20 / 0.015) < 1e-6       # 2 replicas x 20 steps / slowest rank's time


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks([3.5, 1.0], "cpu") == [3.5, 1.0]
    assert bench.job_throughput(1, 10, 20.0) == 500.0


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
