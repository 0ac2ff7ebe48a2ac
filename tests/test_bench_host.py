"""Host-side logic of bench.py, including the multi-rank path on two gloo ranks (CPU)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["BENCH_ROOT"])
import torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world)          # rank 1 is the slow one
val = bench.job_tflops(2.0e12, world, ms)
dist.barrier()
if rank == 0:
    print(json.dumps({"ms": ms, "value": val, "world": world}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_take_the_slowest_time_and_sum_the_work(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, BENCH_ROOT=ROOT)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29531", str(script)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["world"] == 2 and line["ms"] == 15.0                  # max over ranks
    assert line["value"] == pytest.approx(2 * 2.0e12 / 15e-3 / 1e12)  # both ranks' work / slowest time


def test_flop_counts_and_sample_text():
    sys.path.insert(0, ROOT)
    import bench
    f = bench.flops_per_config()
    assert f["C2"] == 2 * 4096 ** 3 and f["C3"] == 4 * 8192 * 4096 * 16384
    assert f["C5"] == pytest.approx(2.750e11, rel=1e-3)               # causal half
    assert "rows" in bench.oracle_sample_text()
    assert bench.job_tflops(1e12, 1, 1.0) == pytest.approx(1000.0)
    assert bench.max_over_ranks(3.5, 1) == 3.5


def test_reference_arm_ranks_other_than_zero_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                         capture_output=True, text=True, env=env, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
