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


def test_block_summary_and_oracle_sample_choice():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2609_23536_b200 import inputs

    blocks = [{"ms": 30.0, "sm_mhz": 1965.0}, {"ms": 40.0, "sm_mhz": 1500.0}, {"ms": 35.0, "sm_mhz": 1600.0}]
    s = bench.block_summary(blocks, steps=10, flop_per_step=1e12, world=2)
    assert s["blocks"] == 3 and s["timed_region_s"] == pytest.approx(0.105)
    assert s["ms_per_step_median"] == 3.5 and s["ms_per_step_min"] == 3.0 and s["ms_per_step_max"] == 4.0
    assert s["value_median"] == pytest.approx(1e12 * 10 * 2 / 35e-3 / 1e12, rel=1e-3)  # the median block, whole job
    assert s["value_first_block"] > s["value_last_block"] and s["sm_mhz_first_block"] == 1965.0 and s["sm_mhz_last_block"] == 1600.0
    # the oracle's bounded sample: the whole block for config 2, the smallest linear for config 3 or for many samples
    only, text = bench.oracle_sample_choice("C2", inputs.CONFIGS["C2"])
    assert only is None and "all 4 linears" in text
    only, text = bench.oracle_sample_choice("C3", inputs.CONFIGS["C3"])
    assert inputs.CONFIGS["C3"]["linears"][only][0] == "o" and "1/832 of a step" in text
    only, _ = bench.oracle_sample_choice("C2", inputs.CONFIGS["C2"], many=True)
    assert inputs.CONFIGS["C2"]["linears"][only][0] == "o"
    # the stamped DRAM traffic figures name a summary that exists and the launch count they were taken for
    for cfg, (nbytes, launches, summary, commit) in bench.QE_TRAFFIC.items():
        assert os.path.exists(os.path.join(ROOT, "profiles", summary)) and nbytes > 0 and launches > 0 and len(commit) >= 7
