"""The multi-rank host logic of bench.py on CPU: two gloo ranks, max-over-ranks timing, whole-job
throughput, distinct seeds, and the reference arm's "rank 0 only" rule."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 1.0 if rank == 0 else 3.0
    ms = bench.max_over_ranks(local_ms, world)
    dist.barrier()
    # rank 1 asks for more host memory than any machine has: every rank must then hear "no"
    allowed = (bench.host_memory_allows(1 << 20, world), bench.host_memory_allows((1 << 20) if rank == 0 else (1 << 60), world))
    out[rank] = (ms, bench.whole_job_gbps(world, 12_000_000_000, ms), bench.rank_seed(rank), allowed)
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_the_slowest_time_and_the_job_throughput():
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
    assert out[0][0] == out[1][0] == 3.0
    assert out[0][1] == pytest.approx(2 * 12e9 / 3e-3 / 1e9)
    assert out[0][2] != out[1][2]
    assert out[0][3] == out[1][3] == (True, False)


def test_single_rank_needs_no_process_group():
    import bench

    assert bench.max_over_ranks(2.5, 1) == 2.5
    assert bench.whole_job_gbps(1, 10**9, 1.0) == pytest.approx(1000.0)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       capture_output=True, text=True, env=env, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--cpu-sample-units", "8"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
