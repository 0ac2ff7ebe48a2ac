"""GPU parity: bf16 tcgen05 GEMM + register epilogue, and the split-row softmax.
Bar: |gpu - oracle| <= 2e-2 + 2e-2*|oracle| (bf16 configs); the softmax chain adds
relative-error, row-sum and arg-max gates because its probabilities are far below atol."""
import functools

import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def _gemm(c, *, act="none", scale=1.0, bias=True, residual=True, w_is_nk=False, out_dtype=BF16, rows=None,
          reduce="none", gamma=None, beta=None, eps=1e-5):
    import paper_2511_16964_b200 as P
    w = np.ascontiguousarray(c["w"].T) if w_is_nk else c["w"]
    b = c["b"] if bias else None
    r = c["r"] if residual else None
    out = P.pike_linear_epilogue(dev(c["x"], BF16), dev(w, BF16), dev(b, BF16), dev(r, BF16), dev(gamma, BF16),
                                 dev(beta, BF16), act=act, scale=scale, reduce=reduce, eps=eps, out_dtype=out_dtype,
                                 w_is_nk=w_is_nk)
    torch.cuda.synchronize()
    st, where = P.pike_get_last_device_status()
    assert st == 0, f"device status {st} at {where:#x}"
    want = O.linear_epilogue(c["x"], c["w"], b, r, gamma, beta, act=act, scale=scale, reduce=reduce, eps=eps, rows=rows)
    got = host64(out)
    return (got if rows is None else got[rows]), want


@pytest.mark.parametrize("w_is_nk", [True, False])
def test_single_tile_plain_gemm(w_is_nk):
    # integer-valued operands: every product and partial sum is exact, so any descriptor,
    # swizzle or transpose mistake shows up as a large error, not as rounding
    rng = np.random.default_rng(0)
    c = dict(x=rng.integers(-3, 4, (128, 64)).astype(np.float32), w=rng.integers(-3, 4, (64, 256)).astype(np.float32))
    got, want = _gemm(c, bias=False, residual=False, w_is_nk=w_is_nk, out_dtype=F32)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("w_is_nk", [True, False])
@pytest.mark.parametrize("M,K,N", [(128, 256, 256), (300, 192, 328), (1, 8, 8), (130, 72, 520)])
def test_small_and_ragged_shapes(M, K, N, w_is_nk):
    c = G.config2(M=M, K=K, N=N, seed=2)
    got, want = _gemm(c, act="silu", scale=0.5, w_is_nk=w_is_nk)
    check_bf16(got, want, what=f"{M}x{K}x{N} nk={w_is_nk}")


@pytest.mark.parametrize("act", ["none", "gelu_erf", "gelu_tanh", "silu"])
@pytest.mark.parametrize("bias,residual,out_dtype", [(True, True, BF16), (False, True, F32), (True, False, F32),
                                                     (False, False, BF16)])
def test_every_epilogue_combination(act, bias, residual, out_dtype):
    c = G.config2(M=200, K=320, N=264, seed=4)
    got, want = _gemm(c, act=act, scale=0.75, bias=bias, residual=residual, out_dtype=out_dtype)
    check_bf16(got, want, what=f"{act} bias={bias} res={residual} {out_dtype}")
    if out_dtype == F32 and act == "none":
        assert np.abs(got - want).max() < 2e-3        # fp32 out: only accumulation-order rounding is left


def test_more_tiles_than_sms_persistent_schedule():
    c = G.config2(M=2560, K=256, N=2312, seed=5)      # 20 x 10 = 200 tiles, ragged last column tile
    got, want = _gemm(c, act="silu", scale=0.5)
    check_bf16(got, want, what="200 tiles")


@functools.lru_cache(maxsize=1)
def _config2_full():
    return G.config2()


def test_config2_full_size_sampled_rows():
    c = _config2_full()
    # one row in every 128-row CTA block (32 blocks), at a different position in each, plus the corners
    rows = np.unique(np.concatenate([[b * 128 + (37 * b + 5) % 128 for b in range(32)], [0, 127, 128, 4095]]))
    got, want = _gemm(c, act="silu", scale=0.5, rows=rows)
    check_bf16(got, want, what="config 2")


def _softmax_gates(got, want, what):
    check_bf16(got, want, what=what)                              # contractual (vacuous for tiny p)
    big = want >= 1e-7
    rel = np.abs(got - want)[big] / want[big]
    assert rel.max() <= 1e-3, f"{what}: max relative error {rel.max():.2e}"
    assert np.abs(got.sum(axis=1) - 1).max() <= 1e-5, f"{what}: row sums"
    assert (got.argmax(axis=1) == want.argmax(axis=1)).all(), f"{what}: argmax"


@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("M,K,N", [(130, 64, 1000), (64, 128, 256), (5, 256, 8)])
def test_split_row_softmax_small(M, K, N, w_is_nk):
    c = G.config4(M=M, K=K, N=N, seed=6)
    got, want = _gemm(c, bias=False, residual=False, out_dtype=F32, reduce="softmax", w_is_nk=w_is_nk)
    _softmax_gates(got, want, f"softmax {M}x{K}x{N}")


def test_config4_full_size_sampled_rows():
    c = G.config4()
    # one row in every 128-row CTA block (16 blocks), at a different position in each, plus the corners
    rows = np.unique(np.concatenate([[b * 128 + (37 * b + 5) % 128 for b in range(16)], [0, 127, 128, 2047]]))
    got, want = _gemm(c, bias=False, residual=False, out_dtype=F32, reduce="softmax", rows=rows)
    _softmax_gates(got, want, "config 4")


@pytest.mark.parametrize("out_dtype", [BF16, F32])
@pytest.mark.parametrize("M,K,N,w_is_nk", [(130, 64, 1000, False), (300, 192, 264, True), (5, 256, 8, False),
                                             (512, 256, 2048, False)])
def test_split_row_layernorm(M, K, N, w_is_nk, out_dtype):
    c = G.config2(M=M, K=K, N=N, seed=7)
    aff = G.config3(M=1, D=N, F=8, seed=7, affine=True)           # bf16 gamma ~ 1 +- 0.5, beta ~ +-0.1
    got, want = _gemm(c, act="gelu_erf", scale=0.5, w_is_nk=w_is_nk, out_dtype=out_dtype, reduce="layernorm",
                      gamma=aff["gamma"], beta=aff["beta"], eps=1e-5)
    check_bf16(got, want, what=f"layernorm {M}x{K}x{N} {out_dtype}")
    if out_dtype == F32:                                           # fp32 out: only fp32 statistics rounding is left
        assert np.abs(got - want).max() < 2e-3


def test_split_row_layernorm_with_a_large_common_offset():
    # rows whose mean is far larger than their spread: a sum-of-squares formula would cancel, the
    # pairwise (mean, M2) merge does not
    c = G.config2(M=64, K=64, N=1024, seed=8)
    c = dict(c, r=(c["r"] * 0.25 + 100.0).astype(np.float32))
    c["r"] = G.round_to_bf16(c["r"])
    got, want = _gemm(c, out_dtype=F32, reduce="layernorm")
    assert np.abs(got - want).max() < 2e-2 and np.abs(got.mean(axis=1)).max() < 1e-3


def test_rejections():
    import paper_2511_16964_b200 as P
    x = torch.zeros((16, 64), device="cuda", dtype=BF16)
    w = torch.zeros((64, 64), device="cuda", dtype=BF16)
    with pytest.raises(P.PikeError) as e:                 # softmax needs fp32 output
        P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=BF16)
    assert e.value.code == 6
    with pytest.raises(P.PikeError) as e:                 # N not a multiple of 8
        P.pike_linear_epilogue(x, torch.zeros((64, 60), device="cuda", dtype=BF16))
    assert e.value.code == 6
    with pytest.raises(P.PikeError) as e:                 # workspace too small for the partials
        P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32,
                               workspace=torch.zeros(64, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 7
    with pytest.raises(P.PikeError) as e:                 # mixed operand dtypes
        P.pike_linear_epilogue(x, w.float())
    assert e.value.code == 3
