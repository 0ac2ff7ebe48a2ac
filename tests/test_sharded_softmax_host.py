"""Column-sharded softmax: the oracle's two-step form pinned to the plain definition, the shard-range
arithmetic, and the exchange between the two steps on two gloo ranks (CPU)."""
import os
import subprocess
import sys

import numpy as np
import pytest

import pike_inputs as G
from oracle import pike_oracle as O

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _load_sharded():
    """paper_2511_16964_b200/sharded.py's range arithmetic without loading the CUDA library."""
    import paper_2511_16964_b200.sharded as S
    return S


@pytest.mark.parametrize("N,world", [(32000, 8), (32000, 3), (8, 1), (16, 4), (1000, 7), (40, 8)])
def test_shard_ranges_partition_the_columns(N, world):
    S = _load_sharded()
    edges = [S.vocab_shard_range(N, r, world) for r in range(world)]
    assert edges[0][0] == 0 and edges[-1][1] == N
    widths = []
    for r, (lo, hi) in enumerate(edges):
        assert lo % 8 == 0 and hi % 8 == 0 and lo <= hi
        if r:
            assert lo == edges[r - 1][1]                       # contiguous, disjoint
        widths.append(hi - lo)
    assert max(widths) - min(widths) <= 8                      # balanced to one block of 8 columns


def test_shard_range_rejections():
    S = _load_sharded()
    with pytest.raises(ValueError):
        S.vocab_shard_range(1001, 0, 2)
    with pytest.raises(ValueError):
        S.vocab_shard_range(1000, 2, 2)


@pytest.mark.parametrize("cuts", [[0, 1000], [0, 504, 1000], [0, 8, 16, 992, 1000], [0, 248, 256, 1000]])
def test_two_step_oracle_equals_the_plain_softmax(cuts):
    """exp(v-m)/l with (m, l) combined from per-slice pairs is the softmax over all columns (exact up to
    fp64 rounding); a wrong combine (forgetting exp(m_r - m), summing maxima) fails this."""
    c = G.config4(M=37, K=64, N=1000, seed=3)
    b = G.uniform((1000,), 0.5, seed=3, tensor_id=77, dtype="bf16")
    want = O.linear_epilogue(c["x"], c["w"], b, act="silu", scale=3.0, reduce="softmax")
    parts = [O.softmax_shard_stats(c["x"], c["w"][:, lo:hi], b[lo:hi], act="silu", scale=3.0)
             for lo, hi in zip(cuts[:-1], cuts[1:])]
    all_stats = np.stack([s for _, s in parts])
    got = np.concatenate([O.softmax_shard_finish(v, all_stats) for v, _ in parts], axis=1)
    assert np.abs(got - want).max() <= 1e-15
    assert np.abs(got.sum(axis=1) - 1).max() <= 1e-13


def test_shard_stats_closed_form():
    """A slice of equal logits c has max c and sum = its width; two such slices (c1 over n1 columns, c2 over
    n2) give probabilities e^{c1}/(n1 e^{c1} + n2 e^{c2}) - the logistic closed form."""
    x = np.ones((2, 8))
    w1, w2 = np.full((8, 16), 0.25), np.full((8, 24), -0.125)          # logits 2 and -1
    v1, s1 = O.softmax_shard_stats(x, w1)
    v2, s2 = O.softmax_shard_stats(x, w2)
    assert np.allclose(s1, [[2.0, 16.0]] * 2, atol=1e-15) and np.allclose(s2, [[-1.0, 24.0]] * 2, atol=1e-15)
    p1 = O.softmax_shard_finish(v1, np.stack([s1, s2]))
    assert np.allclose(p1, 1.0 / (16.0 + 24.0 * np.exp(-3.0)), rtol=1e-15)


WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["PIKE_ROOT"])
import numpy as np, torch, torch.distributed as dist
import pike_inputs as G
from oracle import pike_oracle as O
import paper_2511_16964_b200.sharded as S
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
c = G.config4(M=19, K=64, N=1000, seed=5)
lo, hi = S.vocab_shard_range(1000, rank, world)
v, stats = O.softmax_shard_stats(c["x"], c["w"][:, lo:hi])             # this rank's slice, CPU oracle
all_stats = S.gather_row_stats(torch.from_numpy(stats), None)          # the exchange under test (gloo)
assert tuple(all_stats.shape) == (world, 19, 2)
assert torch.equal(all_stats[rank], torch.from_numpy(stats))           # rank-major layout
mine = O.softmax_shard_finish(v, all_stats.numpy())
want = O.linear_epilogue(c["x"], c["w"], reduce="softmax")[:, lo:hi]
err = float(np.abs(mine - want).max())
errs = [None] * world
dist.all_gather_object(errs, (lo, hi, err))
if rank == 0:
    print(json.dumps({"world": world, "parts": errs}))
dist.destroy_process_group()
"""


def test_exchange_of_row_stats_on_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, PIKE_ROOT=ROOT)
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29533", str(script)],
                         capture_output=True, text=True, env=env, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    import json
    line = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert line["world"] == 2
    (lo0, hi0, e0), (lo1, hi1, e1) = line["parts"]
    assert (lo0, hi0, lo1, hi1) == (0, 504, 504, 1000)
    assert max(e0, e1) <= 1e-15
