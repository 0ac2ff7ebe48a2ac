"""GPU parity on the edges of the envelope: empty inputs, very long reductions, many row tiles, the half-tile
schedule of the GEMM with a ragged last column tile, extreme logits and scores (rescale path of the online
softmax), long ragged sequences.  Same bars as the other parity tests."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def _status_ok():
    import paper_2511_16964_b200 as P
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)


def test_empty_batches_launch_nothing():
    import paper_2511_16964_b200 as P
    x0 = torch.zeros((0, 64), dtype=BF16, device="cuda")
    w = torch.zeros((64, 72), dtype=BF16, device="cuda")
    assert P.pike_linear_epilogue(x0, w, act="silu").shape == (0, 72)
    assert P.pike_linear_epilogue(x0, w, reduce="softmax", out_dtype=F32).shape == (0, 72)
    w1, w2 = torch.zeros((64, 128), dtype=BF16, device="cuda"), torch.zeros((128, 64), dtype=BF16, device="cuda")
    assert P.pike_mlp_block(x0, None, None, w1, None, w2, None).shape == (0, 64)
    q0 = torch.zeros((0, 2, 16, 128), dtype=BF16, device="cuda")
    assert P.pike_attention_chain(q0, q0, q0, scale=1.0, causal=True).shape == (0, 2, 16, 128)
    _status_ok()


def test_very_long_reduction():
    """K = 32768: 512 k-blocks through the ring, fp32 accumulation of 32768 products per output."""
    c = G.config2(M=72, K=32768, N=80, seed=21)
    import paper_2511_16964_b200 as P
    got = P.pike_linear_epilogue(dev(c["x"], BF16), dev(c["w"], BF16), dev(c["b"], BF16), dev(c["r"], BF16), act="silu",
                                 scale=0.5)
    _status_ok()
    check_bf16(host64(got), O.linear_epilogue(c["x"], c["w"], c["b"], c["r"], act="silu", scale=0.5), what="K=32768")


def test_many_row_tiles_one_narrow_column_tile():
    c = G.config2(M=20000, K=64, N=8, seed=22)
    import paper_2511_16964_b200 as P
    got = P.pike_linear_epilogue(dev(c["x"], BF16), dev(c["w"], BF16), dev(c["b"], BF16), dev(c["r"], BF16),
                                 act="gelu_tanh")
    _status_ok()
    check_bf16(host64(got), O.linear_epilogue(c["x"], c["w"], c["b"], c["r"], act="gelu_tanh"), what="20000x64x8")


@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("out_dtype", [BF16, F32])
def test_half_tile_round_with_a_ragged_last_column_tile(w_is_nk, out_dtype):
    """10 x 8 tiles on 74 clusters: one whole round, then 6 tiles as 12 half tiles; the last column tile holds
    136 columns, so its second half is 8 columns wide."""
    M, K, N = 2560, 64, 1928
    c = G.config2(M=M, K=K, N=N, seed=23)
    import paper_2511_16964_b200 as P
    w = np.ascontiguousarray(c["w"].T) if w_is_nk else c["w"]
    got = P.pike_linear_epilogue(dev(c["x"], BF16), dev(w, BF16), dev(c["b"], BF16), dev(c["r"], BF16), act="silu",
                                 scale=0.5, out_dtype=out_dtype, w_is_nk=w_is_nk)
    _status_ok()
    check_bf16(host64(got), O.linear_epilogue(c["x"], c["w"], c["b"], c["r"], act="silu", scale=0.5),
               what="half-tile round")


def test_softmax_of_extreme_logits():
    """Logits of a few hundred: rows are nearly one-hot, exp(v - max) underflows for most columns."""
    c = G.config4(M=64, K=128, N=1000, seed=24)
    import paper_2511_16964_b200 as P
    got = host64(P.pike_linear_epilogue(dev(c["x"], BF16), dev(c["w"], BF16), scale=400.0, reduce="softmax",
                                        out_dtype=F32))
    _status_ok()
    want = O.linear_epilogue(c["x"], c["w"], scale=400.0, reduce="softmax")
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= 2e-3                     # bf16 products are exact; the scale amplifies fp32 sums
    assert np.abs(got.sum(axis=1) - 1).max() <= 1e-5
    assert (got.argmax(axis=1) == want.argmax(axis=1)).all()


@pytest.mark.parametrize("causal", [True, False])
def test_attention_with_scores_of_several_hundred(causal):
    """scale = 4: scores reach +-200, so the running maximum jumps by far more than the lazy-rescale
    threshold from tile to tile and the accumulator is rescaled many times; masked and underflowed
    probabilities must come out as exact zeros, not NaN."""
    c = G.config5(B=1, H=2, S=700, seed=25)
    import paper_2511_16964_b200 as P
    got = P.pike_attention_chain(dev(c["q"], BF16), dev(c["k"], BF16), dev(c["v"], BF16), scale=4.0, causal=causal)
    _status_ok()
    check_bf16(host64(got), O.attention(c["q"], c["k"], c["v"], scale=4.0, causal=causal), what="scale 4 attention")


def test_attention_growing_scores_force_a_rescale_on_every_tile():
    """Keys whose scores grow with the key index: every KV tile raises the row maximum by more than 2^8."""
    S, D = 640, 128
    q = np.zeros((1, 1, S, D), np.float32)
    q[..., 0] = 1.0
    k = np.zeros((1, 1, S, D), np.float32)
    k[0, 0, :, 0] = G.round_to_bf16(np.arange(S, dtype=np.float32) * 0.125)    # score_j ~ j / 8, a bf16 value
    v = G.config5(B=1, H=1, S=S, seed=26)["v"]
    import paper_2511_16964_b200 as P
    got = P.pike_attention_chain(dev(q, BF16), dev(k, BF16), dev(v, BF16), scale=1.0, causal=False)
    _status_ok()
    check_bf16(host64(got), O.attention(q, k, v, scale=1.0, causal=False), what="growing scores")


def test_long_ragged_sequence_sampled_rows():
    S = 4096 + 77
    c = G.config5(B=1, H=1, S=S, seed=27)
    import paper_2511_16964_b200 as P
    got = host64(P.pike_attention_chain(dev(c["q"], BF16), dev(c["k"], BF16), dev(c["v"], BF16),
                                        scale=float(c["scale"]), causal=True))[0, 0]
    _status_ok()
    rows = np.array([0, 1, 127, 128, 2047, 2048, 4095, 4096, S - 1])
    want = O.attention_head(c["q"][0, 0], c["k"][0, 0], c["v"][0, 0], scale=c["scale"], causal=True, rows=rows)
    check_bf16(got[rows], want, what="S = 4173")
