"""GPU parity: pre-LN transformer MLP block (LayerNorm -> GEMM+GELU -> GEMM+residual)."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def _run(c, *, act="gelu_tanh", rows=None, w_is_nk=False):
    import paper_2511_16964_b200 as P
    w1 = np.ascontiguousarray(c["w1"].T) if w_is_nk else c["w1"]
    w2 = np.ascontiguousarray(c["w2"].T) if w_is_nk else c["w2"]
    out = P.pike_mlp_block(dev(c["x"], BF16), dev(c["gamma"], BF16), dev(c["beta"], BF16), dev(w1, BF16),
                           dev(c["b1"], BF16), dev(w2, BF16), dev(c["b2"], BF16), act=act, eps=c["eps"],
                           w_is_nk=w_is_nk)
    torch.cuda.synchronize()
    st, where = P.pike_get_last_device_status()
    assert st == 0, f"device status {st} at {where:#x}"
    want = O.mlp_block(c["x"], c["gamma"], c["beta"], c["w1"], c["b1"], c["w2"], c["b2"], act=act, eps=c["eps"],
                       rows=rows)
    got = host64(out)
    return (got if rows is None else got[rows]), want


@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("M,D,F", [(200, 256, 512), (1, 8, 8), (333, 136, 1032)])
def test_small_blocks_with_affine_layernorm(M, D, F, w_is_nk):
    c = G.config3(M=M, D=D, F=F, seed=7, affine=True)
    got, want = _run(c, w_is_nk=w_is_nk)
    check_bf16(got, want, what=f"mlp {M}x{D}x{F}")


@pytest.mark.parametrize("act", ["gelu_erf", "silu", "none"])
def test_other_activations(act):
    c = G.config3(M=150, D=192, F=384, seed=8, affine=True)
    got, want = _run(c, act=act)
    check_bf16(got, want, what=f"mlp act={act}")


def test_config3_full_size_sampled_rows():
    c = G.config3()
    # one row in every 128-row CTA block (64 blocks), at a different position in each, plus the corners
    rows = np.unique(np.concatenate([[b * 128 + (37 * b + 5) % 128 for b in range(64)], [0, 127, 128, 8191]]))
    got, want = _run(c, rows=rows)
    check_bf16(got, want, what="config 3")


def test_rejections():
    import paper_2511_16964_b200 as P
    x = torch.zeros((16, 64), device="cuda", dtype=BF16)
    w1 = torch.zeros((64, 128), device="cuda", dtype=BF16)
    w2 = torch.zeros((128, 64), device="cuda", dtype=BF16)
    with pytest.raises(P.PikeError) as e:                 # workspace too small
        P.pike_mlp_block(x, None, None, w1, None, w2, None, workspace=torch.zeros(256, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 7
    with pytest.raises(P.PikeError) as e:                 # w2 shape does not chain
        P.pike_mlp_block(x, None, None, w1, None, w1, None)
    assert e.value.code == 2
    assert P.pike_mlp_block_workspace(x, w1) == 2048 + 4096
