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


PLUMBING = r"""
import os, sys, json
sys.path.insert(0, os.environ["BENCH_ROOT"])
import torch.distributed as dist
import bench
from paper_2511_16964_b200.sharded import vocab_shard_range
# everything bench.run_ours does with the rank environment before it touches a GPU, on both ranks
rank, world, local_rank = bench.rank_env()
dist.init_process_group("gloo")
assert (rank, world) == (dist.get_rank(), dist.get_world_size())
args = bench.parse_args(["--gpus", "2", "--steps", "4", "--warmup", "1", "--only", "X3"])
assert args.only == ("X3",) and args.warmup == 3 and args.steps == 4          # warm-up raised to the minimum of 3
weak = bench.per_rank_flops(bench.ALL, world)
strong = bench.per_rank_flops(args.only, world)
cols = vocab_shard_range(32000, rank, world)
ms = bench.max_over_ranks(2.0 + rank, world)
out = {"rank": rank, "local_rank": local_rank, "weak_job": bench.job_tflops(sum(weak.values()), world, ms),
       "strong_job": bench.job_tflops(sum(strong.values()), world, ms), "cols": cols, "ms": ms}
gathered = [None] * world
dist.all_gather_object(gathered, out)
if rank == 0:
    print(json.dumps(gathered))
dist.destroy_process_group()
"""


def test_rank_plumbing_of_the_cuda_arm_on_two_gloo_ranks(tmp_path):
    """The multi-rank branch of the CUDA arm, up to its first CUDA call: rank environment, arguments, per-rank
    flops for the replicated (weak) and the column-sharded (strong) workloads, column ranges, max over ranks."""
    sys.path.insert(0, ROOT)
    import bench
    script = tmp_path / "plumbing.py"
    script.write_text(PLUMBING)
    env = dict(os.environ, BENCH_ROOT=ROOT)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    ranks = json.loads([l for l in out.stdout.splitlines() if l.startswith("[")][-1])
    assert [r["rank"] for r in ranks] == [0, 1] and [r["local_rank"] for r in ranks] == [0, 1]
    assert all(r["ms"] == 3.0 for r in ranks)                                      # the slower rank's time on both
    f = bench.flops_per_config()
    assert ranks[0]["weak_job"] == pytest.approx(2 * sum(f[k] for k in bench.ALL) / 3e-3 / 1e12)
    assert ranks[0]["strong_job"] == pytest.approx(f["X3"] / 3e-3 / 1e12)           # one problem, split over two ranks
    assert ranks[0]["cols"] == [0, 16000] and ranks[1]["cols"] == [16000, 32000]


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
