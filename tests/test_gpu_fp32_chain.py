"""GPU parity: fp32 Linear + bias + activation + scale + residual + reduction (CUDA-core path).
Bar: max |gpu - oracle| <= 1e-4 (fp32 configs)."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_f32, dev, host64

pytestmark = pytest.mark.gpu
F32 = torch.float32


def _run(c, *, act, reduce, scale=1.0, residual=None, w_is_nk=False, gamma=None, beta=None, eps=1e-5):
    import paper_2511_16964_b200 as P
    w = c["w"].T.copy() if w_is_nk else c["w"]
    out = P.pike_linear_epilogue(dev(c["x"], F32), dev(w, F32), dev(c.get("b"), F32), dev(residual, F32),
                                 dev(gamma, F32), dev(beta, F32), act=act, scale=scale, reduce=reduce, eps=eps,
                                 w_is_nk=w_is_nk)
    torch.cuda.synchronize()
    want = O.linear_epilogue(c["x"], c["w"], c.get("b"), residual, gamma, beta, act=act, scale=scale,
                             reduce=reduce, eps=eps)
    return host64(out), want


def test_config1_full():
    c = G.config1()
    got, want = _run(c, act="gelu_erf", reduce="layernorm", gamma=c["gamma"], beta=c["beta"], eps=c["eps"])
    check_f32(got, want, 1e-4, "config 1")
    # LayerNorm invariants on the GPU output itself
    assert np.abs(got.mean(axis=1)).max() < 1e-5


@pytest.mark.parametrize("act", ["none", "gelu_erf", "gelu_tanh", "silu"])
@pytest.mark.parametrize("reduce", ["none", "layernorm", "softmax"])
def test_ragged_shapes_every_act_and_reduce(act, reduce):
    c = G.config1(M=37, K=100, N=200, seed=3)
    rng = np.random.default_rng(5)
    res = rng.standard_normal((37, 200)).astype(np.float32)
    gamma = rng.uniform(0.5, 1.5, 200).astype(np.float32)
    beta = rng.uniform(-0.1, 0.1, 200).astype(np.float32)
    got, want = _run(c, act=act, reduce=reduce, scale=0.5, residual=res, gamma=gamma, beta=beta)
    check_f32(got, want, 1e-4, f"{act}/{reduce}")


@pytest.mark.parametrize("M,K,N", [(1, 8, 8), (5, 1, 1024), (700, 300, 72), (3, 2500, 40)])
def test_edge_shapes_and_weight_layout(M, K, N):
    c = G.config1(M=M, K=K, N=N, seed=1)
    for nk in (False, True):
        got, want = _run(c, act="gelu_erf", reduce="layernorm", w_is_nk=nk)
        check_f32(got, want, 1e-4, f"{M}x{K}x{N} nk={nk}")


def test_empty_batch_and_rejections():
    import paper_2511_16964_b200 as P
    x = torch.zeros((0, 16), device="cuda")
    w = torch.zeros((16, 8), device="cuda")
    assert P.pike_linear_epilogue(x, w).shape == (0, 8)
    with pytest.raises(P.PikeError) as e:            # N > 1024 on the fp32 path
        P.pike_linear_epilogue(torch.zeros((4, 16), device="cuda"), torch.zeros((16, 1032), device="cuda"))
    assert e.value.code == 6
    with pytest.raises(P.PikeError) as e:            # K mismatch
        P.pike_linear_epilogue(torch.zeros((4, 16), device="cuda"), torch.zeros((24, 8), device="cuda"))
    assert e.value.code == 2
    with pytest.raises(P.PikeError) as e:            # out aliases x
        xx = torch.zeros((8, 8), device="cuda")
        P.pike_linear_epilogue(xx, torch.zeros((8, 8), device="cuda"), out=xx)
    assert e.value.code == 6
    with pytest.raises(P.PikeError) as e:            # misaligned base pointer
        buf = torch.zeros(4 * 16 + 1, device="cuda")
        P.pike_linear_epilogue(buf[1:].view(4, 16), w)
    assert e.value.code == 4


@pytest.mark.parametrize("M,K,N", [(182, 148, 1), (91, 1, 840), (1, 64, 72)])
def test_extent_one_dimensions_with_arbitrary_strides(M, K, N):
    """torch leaves the stride of an extent-1 dimension arbitrary: a [1, K] transpose view of a [K, 1] tensor keeps
    stride 1 for its single row.  Such views are accepted (the binding hands the C ABI canonical strides)."""
    import paper_2511_16964_b200 as P
    c = G.config1(M=M, K=K, N=N, seed=9)
    w_t = dev(c["w"], F32).t()                              # [N, K] view of the [K, N] tensor
    if N == 1 or K == 1:
        assert w_t.is_contiguous() and w_t.stride() != (K, 1)      # the case this test is about
    x = dev(c["x"], F32)
    out = P.pike_linear_epilogue(x, w_t if w_t.is_contiguous() else w_t.contiguous(), dev(c["b"], F32), act="gelu_erf",
                                 reduce="layernorm", eps=c["eps"], w_is_nk=True)
    want = O.linear_epilogue(c["x"], c["w"], c["b"], act="gelu_erf", reduce="layernorm", eps=c["eps"])
    check_f32(host64(out), want, 1e-4, f"{M}x{K}x{N} with an extent-1 stride")


@pytest.mark.parametrize("M,K,N", [(64, 256, 256), (40, 700, 512), (24, 300, 1000), (9, 520, 96), (128, 64, 1024)])
@pytest.mark.parametrize("nk", [False, True])
def test_small_problem_kernel_is_exact_on_integers(M, K, N, nk):
    """Small integers make every product and partial sum exact in fp32 whatever the summation order, so the k slices,
    the 4x4 register tiles, the chunks of k (one, or several of 256) and every ragged edge of the small-problem
    kernel must reproduce the oracle bit for bit, with tiled copies ([K,N] weights, aligned pitches) and without."""
    import paper_2511_16964_b200 as P
    rng = np.random.default_rng(M * 7 + K + N + nk)
    x = rng.integers(-4, 5, (M, K)).astype(np.float32)
    w = rng.integers(-3, 4, (K, N)).astype(np.float32)
    b = rng.integers(-8, 9, N).astype(np.float32)
    r = rng.integers(-8, 9, (M, N)).astype(np.float32)
    want = O.linear_epilogue(x, w, b, r, act="none", scale=2.0)
    wd = dev(w.T.copy() if nk else w, F32)
    got = P.pike_linear_epilogue(dev(x, F32), wd, dev(b, F32), dev(r, F32), act="none", scale=2.0, w_is_nk=nk)
    assert np.array_equal(host64(got), want)
    # the same through row pitches that are not multiples of 16 bytes: per-thread copies instead of tiled ones
    xp = torch.zeros((M, K + 1), device="cuda", dtype=F32)
    xp[:, :K] = dev(x, F32)
    wrows, wcols = wd.shape
    wp = torch.zeros((wrows, wcols + 3), device="cuda", dtype=F32)
    wp[:, :wcols] = wd
    got = P.pike_linear_epilogue(xp[:, :K], wp[:, :wcols], dev(b, F32), dev(r, F32), act="none", scale=2.0, w_is_nk=nk)
    assert np.array_equal(host64(got), want)


@pytest.mark.parametrize("reduce", ["layernorm", "softmax"])
@pytest.mark.parametrize("M,K,N", [(40, 700, 512), (24, 300, 1000), (16, 256, 40)])
def test_small_problem_kernel_reductions_over_wide_and_ragged_rows(M, K, N, reduce):
    c = G.config1(M=M, K=K, N=N, seed=11)
    rng = np.random.default_rng(N)
    gamma = rng.uniform(0.5, 1.5, N).astype(np.float32)
    beta = rng.uniform(-0.1, 0.1, N).astype(np.float32)
    got, want = _run(c, act="silu", reduce=reduce, gamma=gamma, beta=beta)
    check_f32(got, want, 1e-4, f"{M}x{K}x{N} {reduce}")
    if reduce == "softmax":
        assert np.abs(got.sum(axis=1) - 1.0).max() < 1e-5


def test_layernorm_statistics_survive_a_mean_that_dwarfs_the_spread():
    """The one-pass shifted statistics and the pooled merge across the cluster must not lose the variance when
    every value sits near 100 and the row's spread is about 0.4 (a residual of 100 added to each output).  Bar 2e-4:
    an fp32 value near 100 carries a rounding error of up to 3.8e-6, which the division by the spread multiplies by 2.5
    before anything else is counted."""
    c = G.config1(M=32, K=256, N=512, seed=5)
    res = np.full((32, 512), 100.0, np.float32)
    got, want = _run(c, act="gelu_erf", reduce="layernorm", residual=res)
    check_f32(got, want, 2e-4, "mean 100")
