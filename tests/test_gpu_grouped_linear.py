"""GPU parity: grouped linear + epilogue (many weight matrices, one launch, device-side group offsets)."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def _run(c, *, act="silu", scale=0.5, bias=True, residual=True, w_is_nk=False, out_dtype=BF16):
    import paper_2511_16964_b200 as P
    w = np.ascontiguousarray(c["w"].transpose(0, 2, 1)) if w_is_nk else c["w"]
    b = c["b"] if bias else None
    r = c["r"] if residual else None
    off = torch.from_numpy(c["offsets"]).to("cuda")
    out = P.pike_grouped_linear_epilogue(dev(c["x"], BF16), dev(w, BF16), dev(b, BF16), dev(r, BF16), off, act=act,
                                         scale=scale, w_is_nk=w_is_nk, out_dtype=out_dtype)
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    want = O.grouped_linear_epilogue(c["x"], c["w"], b, r, c["offsets"], act=act, scale=scale)
    return host64(out), want


@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("T,K,N,Gn", [(700, 128, 264, 5), (64, 64, 64, 8), (1500, 192, 520, 3), (9, 8, 8, 12)])
def test_uneven_groups(T, K, N, Gn, w_is_nk):
    c = G.grouped_linear(T=T, K=K, N=N, G=Gn, seed=18)
    assert (np.diff(c["offsets"]) == 0).any() or Gn <= 2          # the recipe contains an empty group
    got, want = _run(c, w_is_nk=w_is_nk)
    check_bf16(got, want, what=f"grouped {T}x{K}x{N} G={Gn} nk={w_is_nk}")


@pytest.mark.parametrize("act,bias,residual,out_dtype", [("none", False, False, F32), ("gelu_tanh", True, False, BF16),
                                                         ("gelu_erf", False, True, F32)])
def test_epilogue_variants(act, bias, residual, out_dtype):
    c = G.grouped_linear(T=900, K=256, N=328, G=6, seed=19)
    got, want = _run(c, act=act, scale=0.75, bias=bias, residual=residual, out_dtype=out_dtype)
    check_bf16(got, want, what=f"grouped {act}")


def test_single_group_equals_the_plain_chain_bitwise():
    import paper_2511_16964_b200 as P
    c = G.config2(M=600, K=128, N=264, seed=20)
    x, w, b, r = dev(c["x"], BF16), dev(c["w"], BF16), dev(c["b"], BF16), dev(c["r"], BF16)
    off = torch.tensor([0, 600], dtype=torch.int32, device="cuda")
    a = P.pike_grouped_linear_epilogue(x, w[None], b[None], r, off, act="silu", scale=0.5)
    bb = P.pike_linear_epilogue(x, w, b, r, act="silu", scale=0.5)
    torch.cuda.synchronize()
    assert torch.equal(a, bb)


def test_mid_size_mixture_of_experts_shape():
    c = G.grouped_linear(T=4096, K=1024, N=2048, G=16, seed=21)
    got, want = _run(c, act="silu", scale=1.0, residual=False)
    check_bf16(got, want, what="grouped 4096x1024x2048 G=16")


def test_rejections():
    import paper_2511_16964_b200 as P
    x = torch.zeros((16, 64), device="cuda", dtype=BF16)
    w = torch.zeros((2, 64, 64), device="cuda", dtype=BF16)
    off = torch.tensor([0, 8, 16], dtype=torch.int32, device="cuda")
    with pytest.raises(P.PikeError) as e:                 # K mismatch
        P.pike_grouped_linear_epilogue(x, torch.zeros((2, 32, 64), device="cuda", dtype=BF16), None, None, off)
    assert e.value.code == 2
    with pytest.raises(P.PikeError) as e:                 # bias must be [G,N]
        P.pike_grouped_linear_epilogue(x, w, torch.zeros((64,), device="cuda", dtype=BF16), None, off)
    assert e.value.code == 2
    with pytest.raises(TypeError):                        # offsets must be device int32
        P.pike_grouped_linear_epilogue(x, w, None, None, off.long())
