"""GPU parity of the IEEE-half (f16) variant of every 16-bit chain: same kernels, f16 operand format,
f16 conversions in the epilogues.

Bar: |gpu - oracle| <= 2.5e-3 + 2.5e-3*|oracle|.  The bf16 bar is 2e-2 for a type whose rounding step is
2^-8; f16's step is 2^-11, eight times finer, hence 2e-2 / 8.  Exact-value cases (integers that need
eleven significant bits, pass-through of full-mantissa values) separate "computed in f16" from "computed
through bf16", which the tolerance alone could not."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
F16, BF16, F32 = torch.float16, torch.bfloat16, torch.float32


def check_f16(got, want, what=""):
    return check_bf16(got, want, atol=2.5e-3, rtol=2.5e-3, what=what)


def _ok():
    import paper_2511_16964_b200 as P
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)


def _gemm(c, *, act="none", scale=1.0, bias=True, residual=True, w_is_nk=False, out_dtype=F16, reduce="none",
          gamma=None, beta=None, eps=1e-5, side=F16):
    import paper_2511_16964_b200 as P
    w = np.ascontiguousarray(c["w"].T) if w_is_nk else c["w"]
    b = c.get("b") if bias else None
    r = c.get("r") if residual else None
    out = P.pike_linear_epilogue(dev(c["x"], F16), dev(w, F16), dev(b, side), dev(r, side), dev(gamma, side),
                                 dev(beta, side), act=act, scale=scale, reduce=reduce, eps=eps, out_dtype=out_dtype,
                                 w_is_nk=w_is_nk)
    _ok()
    want = O.linear_epilogue(c["x"], c["w"], b, r, gamma, beta, act=act, scale=scale, reduce=reduce, eps=eps)
    return host64(out), want


@pytest.mark.parametrize("w_is_nk", [True, False])
def test_integers_that_need_eleven_bits_are_exact(w_is_nk):
    # |x| up to 2047 is exact in f16 but not in bf16 (8 significant bits): a kernel that read or multiplied
    # the operands as bf16 cannot return the exact sums
    rng = np.random.default_rng(1)
    c = dict(x=rng.integers(-2047, 2048, (256, 64)).astype(np.float32),
             w=rng.integers(-3, 4, (64, 256)).astype(np.float32))
    got, want = _gemm(c, bias=False, residual=False, w_is_nk=w_is_nk, out_dtype=F32)
    assert np.array_equal(got, want)


def test_f16_values_pass_through_the_epilogue_unchanged():
    c = G.config2(M=300, K=64, N=264, seed=31, dtype="f16")
    # full-mantissa inputs: most values are not representable in bf16
    assert (G.round_to_bf16(c["x"]) != c["x"]).mean() > 0.5
    # x @ I written as f16 returns x bit for bit (operand format, accumulator read-out and f16 packing)
    eye = dict(x=c["x"], w=np.eye(64, 264, dtype=np.float32))
    got, _ = _gemm(eye, bias=False, residual=False)
    assert np.array_equal(got[:, :64], c["x"].astype(np.float64)) and not got[:, 64:].any()
    # 0 @ w + bias + residual with an fp32 result: the f16 bias and residual are read exactly
    zero = dict(c, x=np.zeros_like(c["x"]))
    got, _ = _gemm(zero, out_dtype=F32)
    want = (c["b"][None, :].astype(np.float32) + c["r"]).astype(np.float64)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("w_is_nk", [True, False])
@pytest.mark.parametrize("M,K,N", [(128, 256, 256), (300, 192, 328), (1, 8, 8), (130, 72, 520)])
def test_small_and_ragged_shapes(M, K, N, w_is_nk):
    c = G.config2(M=M, K=K, N=N, seed=32, dtype="f16")
    got, want = _gemm(c, act="silu", scale=0.5, w_is_nk=w_is_nk)
    check_f16(got, want, what=f"f16 {M}x{K}x{N} nk={w_is_nk}")


@pytest.mark.parametrize("act", ["none", "gelu_erf", "gelu_tanh", "silu"])
@pytest.mark.parametrize("bias,residual,out_dtype,side", [(True, True, F16, F16), (False, True, F32, F32),
                                                          (True, False, F32, F16), (True, True, F16, F32)])
def test_epilogue_combinations(act, bias, residual, out_dtype, side):
    c = G.config2(M=200, K=320, N=264, seed=33, dtype="f16")
    got, want = _gemm(c, act=act, scale=0.75, bias=bias, residual=residual, out_dtype=out_dtype, side=side)
    check_f16(got, want, what=f"f16 {act} bias={bias} res={residual} {out_dtype}")


def test_persistent_schedule_many_tiles():
    c = G.config2(M=2560, K=256, N=2312, seed=34, dtype="f16")
    got, want = _gemm(c, act="silu", scale=0.5)
    check_f16(got, want, what="f16 200 tiles")


def test_split_row_softmax():
    c = G.config4(M=200, K=256, N=2000, seed=35, dtype="f16")
    got, want = _gemm(c, bias=False, residual=False, reduce="softmax", out_dtype=F32)
    assert np.abs(got.sum(axis=1) - 1).max() < 1e-5
    assert np.abs(got / want - 1).max() < 2e-3
    assert np.array_equal(got.argmax(axis=1), want.argmax(axis=1))


@pytest.mark.parametrize("out_dtype", [F16, F32])
def test_split_row_layernorm(out_dtype):
    c = G.config2(M=260, K=192, N=1032, seed=36, dtype="f16")
    gamma = G.round_to((1.0 + G.uniform((1032,), 0.5, seed=36, tensor_id=90, dtype="f16")).astype(np.float32), "f16")
    beta = G.uniform((1032,), 0.1, seed=36, tensor_id=91, dtype="f16")
    got, want = _gemm(c, act="gelu_tanh", reduce="layernorm", gamma=gamma, beta=beta, out_dtype=out_dtype)
    check_f16(got, want, what=f"f16 linear+layernorm {out_dtype}")


@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("M,D,F", [(200, 256, 512), (1, 8, 8), (333, 136, 1032), (40, 4608, 64)])
def test_mlp_block(M, D, F, w_is_nk):
    import paper_2511_16964_b200 as P
    c = G.config3(M=M, D=D, F=F, seed=37, affine=True, dtype="f16")
    w1 = np.ascontiguousarray(c["w1"].T) if w_is_nk else c["w1"]
    w2 = np.ascontiguousarray(c["w2"].T) if w_is_nk else c["w2"]
    out = P.pike_mlp_block(dev(c["x"], F16), dev(c["gamma"], F16), dev(c["beta"], F16), dev(w1, F16),
                           dev(c["b1"], F16), dev(w2, F16), dev(c["b2"], F16), eps=c["eps"], w_is_nk=w_is_nk)
    _ok()
    assert out.dtype == F16
    want = O.mlp_block(c["x"], c["gamma"], c["beta"], c["w1"], c["b1"], c["w2"], c["b2"], act="gelu_tanh", eps=c["eps"])
    check_f16(host64(out), want, what=f"f16 mlp {M}x{D}x{F}")


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("B,H,S,D", [(1, 2, 256, 128), (2, 3, 300, 128), (1, 1, 1, 128), (1, 2, 513, 64), (2, 2, 129, 64)])
def test_attention(B, H, S, D, causal):
    import paper_2511_16964_b200 as P
    c = G.config5(B=B, H=H, S=S, D=D, seed=38, dtype="f16")
    out = P.pike_attention_chain(dev(c["q"], F16), dev(c["k"], F16), dev(c["v"], F16), scale=c["scale"], causal=causal)
    _ok()
    got = host64(out)
    want = O.attention(c["q"], c["k"], c["v"], scale=c["scale"], causal=causal)
    check_f16(got, want, what=f"f16 attention B{B} H{H} S{S} D{D} causal={causal}")
    if causal:      # row 0 sees key 0 only: V[0] passes through bit for bit, full f16 mantissa included
        assert np.array_equal(got[:, :, 0, :], c["v"][:, :, 0, :].astype(np.float64))


def test_cross_attention():
    import paper_2511_16964_b200 as P
    cq = G.config5(B=2, H=2, S=200, seed=39, dtype="f16")
    ck = G.config5(B=2, H=2, S=77, seed=40, dtype="f16")
    out = P.pike_attention_chain(dev(cq["q"], F16), dev(ck["k"], F16), dev(ck["v"], F16), scale=cq["scale"], causal=False)
    _ok()
    check_f16(host64(out), O.attention(cq["q"], ck["k"], ck["v"], scale=cq["scale"], causal=False), what="f16 cross")


@pytest.mark.parametrize("B,S,E,causal,w_is_nk", [(2, 300, 256, True, False), (3, 129, 384, False, True)])
def test_attention_block(B, S, E, causal, w_is_nk):
    import paper_2511_16964_b200 as P
    c = G.attention_block(B=B, S=S, E=E, seed=41, dtype="f16")
    wq = np.ascontiguousarray(c["w_qkv"].T) if w_is_nk else c["w_qkv"]
    wo = np.ascontiguousarray(c["w_o"].T) if w_is_nk else c["w_o"]
    out = P.pike_attention_block(dev(c["x"], F16), dev(c["gamma"], F16), dev(c["beta"], F16), dev(wq, F16),
                                 dev(c["b_qkv"], F16), dev(wo, F16), dev(c["b_o"], F16), scale=float(c["scale"]),
                                 causal=causal, eps=c["eps"], w_is_nk=w_is_nk)
    _ok()
    want = O.attention_block(c["x"], c["gamma"], c["beta"], c["w_qkv"], c["b_qkv"], c["w_o"], c["b_o"],
                             num_heads=c["num_heads"], scale=c["scale"], causal=causal, eps=c["eps"])
    check_f16(host64(out), want, what=f"f16 attention block B{B} S{S} E{E}")


@pytest.mark.parametrize("w_is_nk", [False, True])
def test_grouped_linear(w_is_nk):
    import paper_2511_16964_b200 as P
    c = G.grouped_linear(T=700, K=128, N=264, G=5, seed=42, dtype="f16")
    w = np.ascontiguousarray(c["w"].transpose(0, 2, 1)) if w_is_nk else c["w"]
    off = torch.from_numpy(c["offsets"]).to("cuda")
    out = P.pike_grouped_linear_epilogue(dev(c["x"], F16), dev(w, F16), dev(c["b"], F16), dev(c["r"], F16), off,
                                         act="silu", scale=0.5, w_is_nk=w_is_nk)
    _ok()
    want = O.grouped_linear_epilogue(c["x"], c["w"], c["b"], c["r"], c["offsets"], act="silu", scale=0.5)
    check_f16(host64(out), want, what="f16 grouped")


def test_the_two_16_bit_types_never_mix():
    import paper_2511_16964_b200 as P
    z = lambda shape, dt: torch.zeros(shape, device="cuda", dtype=dt)
    cases = [
        lambda: P.pike_linear_epilogue(z((16, 64), F16), z((64, 64), BF16), None, None, None, None),
        lambda: P.pike_linear_epilogue(z((16, 64), F16), z((64, 64), F16), z((64,), BF16), None, None, None),
        lambda: P.pike_linear_epilogue(z((16, 64), BF16), z((64, 64), BF16), None, z((16, 64), F16), None, None),
        lambda: P.pike_linear_epilogue(z((16, 64), F16), z((64, 64), F16), None, None, None, None, out_dtype=BF16),
        lambda: P.pike_mlp_block(z((16, 64), F16), None, None, z((64, 128), F16), None, z((128, 64), BF16), None),
        lambda: P.pike_mlp_block(z((16, 64), F16), z((64,), BF16), None, z((64, 128), F16), None, z((128, 64), F16), None),
        lambda: P.pike_attention_chain(z((1, 1, 16, 128), F16), z((1, 1, 16, 128), BF16), z((1, 1, 16, 128), F16), scale=1.0),
        lambda: P.pike_attention_chain(z((1, 1, 16, 128), F16), z((1, 1, 16, 128), F16), z((1, 1, 16, 128), F16), scale=1.0,
                                       out=z((1, 1, 16, 128), BF16)),
        lambda: P.pike_grouped_linear_epilogue(z((16, 64), F16), z((2, 64, 64), BF16), None, None,
                                               torch.tensor([0, 8, 16], dtype=torch.int32, device="cuda")),
        lambda: P.pike_attention_block(z((1, 16, 128), F16), None, None, z((128, 384), F16), None, z((128, 128), BF16), None,
                                       scale=1.0),
    ]
    for i, call in enumerate(cases):
        with pytest.raises(P.PikeError) as e:
            call()
        assert e.value.code == 3, f"case {i}: status {e.value.code}"
