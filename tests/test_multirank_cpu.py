"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job aggregation,
and the reference arm's "rank 0 only" rule.  (The path itself has no exchange step: replicas only.)"""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(torch, dist, 3.0 + rank, "cpu")        # rank 1 is the slow one
    val = bench.whole_job_value(1000.0, world, ms)
    out[rank] = (ms, val)
    dist.destroy_process_group()


def test_two_ranks_agree_on_the_slowest_time_and_sum_the_bytes():
    ctx = mp.get_context("spawn")
    with ctx.Manager() as m:
        out = m.dict()
        port = 29500 + os.getpid() % 2000
        procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
        for p in procs:
            p.start()
        for p in procs:
            p.join(120)
            assert p.exitcode == 0
        assert out[0] == out[1]
        ms, val = out[0]
        assert ms == 4.0
        assert val == 1000.0 * 2 / 4.0 / 1e6


def test_reference_arm_runs_on_rank_0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0
    assert r.stdout.strip() == ""          # the other ranks exit without work and print nothing


def test_single_rank_passthrough():
    import bench
    assert bench.max_over_ranks(torch, None, 2.5, "cpu") == 2.5
    assert bench.whole_job_value(2e9, 1, 1.0) == 2000.0
