"""GPU parity: pre-LN attention block with fused input and output projections."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def _run(c, causal, w_is_nk=False):
    import paper_2511_16964_b200 as P
    wq = np.ascontiguousarray(c["w_qkv"].T) if w_is_nk else c["w_qkv"]
    wo = np.ascontiguousarray(c["w_o"].T) if w_is_nk else c["w_o"]
    out = P.pike_attention_block(dev(c["x"], BF16), dev(c["gamma"], BF16), dev(c["beta"], BF16), dev(wq, BF16),
                                 dev(c["b_qkv"], BF16), dev(wo, BF16), dev(c["b_o"], BF16), scale=float(c["scale"]),
                                 causal=causal, eps=c["eps"], w_is_nk=w_is_nk)
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    want = O.attention_block(c["x"], c["gamma"], c["beta"], c["w_qkv"], c["b_qkv"], c["w_o"], c["b_o"],
                             num_heads=c["num_heads"], scale=c["scale"], causal=causal, eps=c["eps"])
    return host64(out), want


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("B,S,E,w_is_nk", [(1, 128, 128, False), (2, 300, 256, False), (3, 129, 384, True), (1, 1, 128, False)])
def test_small_blocks(B, S, E, w_is_nk, causal):
    c = G.attention_block(B=B, S=S, E=E, seed=13)
    got, want = _run(c, causal, w_is_nk)
    check_bf16(got, want, what=f"attention block B{B} S{S} E{E} causal={causal}")


def test_mid_size_block():
    c = G.attention_block(B=2, S=640, E=1024, seed=14)
    got, want = _run(c, True)
    check_bf16(got, want, what="attention block 2x640x1024")


def test_rejections():
    import paper_2511_16964_b200 as P
    x = torch.zeros((1, 16, 192), device="cuda", dtype=BF16)          # E not a multiple of 128
    w = torch.zeros((192, 576), device="cuda", dtype=BF16)
    wo = torch.zeros((192, 192), device="cuda", dtype=BF16)
    with pytest.raises(P.PikeError) as e:
        P.pike_attention_block(x, None, None, w, None, wo, None, scale=1.0)
    assert e.value.code == 6
    x = torch.zeros((1, 16, 128), device="cuda", dtype=BF16)
    with pytest.raises(P.PikeError) as e:                              # w_qkv has the wrong width
        P.pike_attention_block(x, None, None, torch.zeros((128, 256), device="cuda", dtype=BF16),
                               None, torch.zeros((128, 128), device="cuda", dtype=BF16), None, scale=1.0)
    assert e.value.code == 2
    assert P.pike_attention_block_workspace(x, scale=1.0) == 2 * 4096 + 3 * 4096
