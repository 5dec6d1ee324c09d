"""Host-side logic of bench.py: the multi-rank timing reduction (world_size 2, gloo, CPU) and the
behaviour of the reference arm on ranks other than 0."""

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
    mine = [10.0 + rank, 20.0 - rank, 3.0 * (rank + 1)]
    got = bench.max_over_ranks(mine, world, "cpu")
    out.put((rank, got))
    dist.barrier()
    dist.destroy_process_group()


def test_times_are_reduced_with_max_over_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res[0] == res[1] == [11.0, 20.0, 6.0]


def test_whole_job_value_counts_all_replicas():
    sys.path.insert(0, ROOT)
    import bench
    one = bench.whole_job_tflops(2e12, 10, 1, 1000.0)
    assert abs(one - 20.0) < 1e-12
    assert abs(bench.whole_job_tflops(2e12, 10, 4, 1000.0) - 4 * one) < 1e-12


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
