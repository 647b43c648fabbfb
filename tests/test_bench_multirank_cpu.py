"""The N > 1 path of bench.py (independent replicas: barrier, max-over-ranks time, whole-job value),
exercised with two gloo ranks on CPU; and the reference arm's rank handling."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, device="cpu")  # rank 1 is the slow one
    val = bench.whole_job_value(1e12, 4, world, ms)
    q.put((rank, ms, val))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_the_aggregate_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, val in got:
        assert ms == 15.0  # max over ranks, on every rank
        assert val == pytest.approx(1e12 * 4 * 2 / 15e-3 / 1e12)  # work of both replicas over the slowest rank's time


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                         capture_output=True, text=True, env=env, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_step_flops_and_gradient_offsets_of_the_configurations():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_23536_b200 import inputs

    assert bench.step_flops(inputs.CONFIGS["C2"]) == pytest.approx(5.05e12, rel=2e-3)
    assert bench.step_flops(inputs.CONFIGS["C3"]) == pytest.approx(343e12, rel=2e-3)
    offs, total = inputs.grad_offsets(inputs.CONFIGS["C2"]["linears"])
    assert (offs, total) == ([0, 12582912, 16777216, 39845888], 51380224)
