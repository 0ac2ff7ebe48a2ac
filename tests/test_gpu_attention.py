"""GPU parity: GEMM -> online softmax -> GEMM attention chain (scores never leave the chip)."""
import functools

import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def _run(c, causal):
    import paper_2511_16964_b200 as P
    out = P.pike_attention_chain(dev(c["q"], BF16), dev(c["k"], BF16), dev(c["v"], BF16), scale=c["scale"],
                                 causal=causal)
    torch.cuda.synchronize()
    st, where = P.pike_get_last_device_status()
    assert st == 0, f"device status {st} at {where:#x}"
    return host64(out)


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("B,H,S", [(1, 1, 128), (1, 2, 256), (2, 3, 300), (1, 1, 1), (1, 2, 129), (1, 1, 640)])
def test_small_and_ragged_sequences(B, H, S, causal):
    c = G.config5(B=B, H=H, S=S, seed=9)
    got = _run(c, causal)
    want = O.attention(c["q"], c["k"], c["v"], scale=c["scale"], causal=causal)
    check_bf16(got, want, what=f"attention B{B} H{H} S{S} causal={causal}")


def test_structural_properties_on_the_gpu_output():
    c = G.config5(B=1, H=2, S=384, seed=10)
    got = _run(c, True)
    # causal row 0 attends to key 0 only -> O[0] = V[0] exactly (bf16 values pass through)
    assert np.array_equal(got[:, :, 0, :], c["v"][:, :, 0, :].astype(np.float64))
    # V == 1 -> O == 1
    c1 = dict(c, v=np.ones_like(c["v"]))
    assert np.abs(_run(c1, True) - 1).max() <= 2 ** -7
    # run-to-run bit reproducibility
    assert np.array_equal(got, _run(c, True))


@pytest.mark.parametrize("causal", [True, False])
@pytest.mark.parametrize("B,H,S", [(1, 2, 128), (2, 3, 300), (1, 1, 1), (1, 2, 513)])
def test_head_dimension_64(B, H, S, causal):
    c = G.config5(B=B, H=H, S=S, D=64, seed=15)
    got = _run(c, causal)
    want = O.attention(c["q"], c["k"], c["v"], scale=c["scale"], causal=causal)
    check_bf16(got, want, what=f"attention D=64 B{B} H{H} S{S} causal={causal}")


@pytest.mark.parametrize("D", [128, 64])
@pytest.mark.parametrize("Sq,Sk", [(128, 384), (200, 77), (1, 300), (300, 1)])
def test_cross_attention_keys_of_another_length(Sq, Sk, D):
    import paper_2511_16964_b200 as P
    cq = G.config5(B=2, H=2, S=Sq, D=D, seed=16)
    ck = G.config5(B=2, H=2, S=Sk, D=D, seed=17)
    out = P.pike_attention_chain(dev(cq["q"], BF16), dev(ck["k"], BF16), dev(ck["v"], BF16), scale=cq["scale"],
                                 causal=False)
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    want = O.attention(cq["q"], ck["k"], ck["v"], scale=cq["scale"], causal=False)
    check_bf16(host64(out), want, what=f"cross attention Sq{Sq} Sk{Sk} D{D}")
    with pytest.raises(P.PikeError) as e:                 # no causal alignment is defined for Sq != Sk
        P.pike_attention_chain(dev(cq["q"], BF16), dev(ck["k"], BF16), dev(ck["v"], BF16), scale=1.0, causal=True)
    assert e.value.code == 6


def test_strided_views_of_a_packed_projection_buffer():
    """q, k, v as slices of one [B,S,3,H,D] buffer and the output written as [B,S,H,D]: no copies."""
    import paper_2511_16964_b200 as P
    B, H, S = 2, 3, 200
    c = G.config5(B=B, H=H, S=S, seed=12)
    packed = torch.empty((B, S, 3, H, 128), dtype=BF16, device="cuda")
    for i, name in enumerate("qkv"):
        packed[:, :, i] = dev(c[name], BF16).permute(0, 2, 1, 3)
    q, k, v = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))      # [B,H,S,D] views, row pitch 3*H*128
    out_bshd = torch.zeros((B, S, H, 128), dtype=BF16, device="cuda")
    P.pike_attention_chain(q, k, v, scale=c["scale"], causal=True, out=out_bshd.permute(0, 2, 1, 3))
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    want = O.attention(c["q"], c["k"], c["v"], scale=c["scale"], causal=True)
    check_bf16(host64(out_bshd.permute(0, 2, 1, 3)), want, what="strided attention")


@pytest.mark.parametrize("D", [128, 64])
def test_output_rows_that_are_only_16_byte_aligned(D):
    """Output rows with a pitch of D + 8 elements: every other row starts 16 bytes off a 32-byte boundary, so the
    kernel must fall back from its 32-byte stores; the padding columns stay untouched."""
    import paper_2511_16964_b200 as P
    B, H, S = 1, 2, 200
    c = G.config5(B=B, H=H, S=S, D=D, seed=14)
    padded = torch.full((B, H, S, D + 8), 7.0, dtype=BF16, device="cuda")
    P.pike_attention_chain(dev(c["q"], BF16), dev(c["k"], BF16), dev(c["v"], BF16), scale=c["scale"], causal=True,
                           out=padded[..., :D])
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    check_bf16(host64(padded[..., :D]), O.attention(c["q"], c["k"], c["v"], scale=c["scale"], causal=True),
               what="padded output rows")
    assert (padded[..., D:] == 7.0).all()


@functools.lru_cache(maxsize=1)
def _config5_full():
    return G.config5()


def test_config5_full_size_sampled_rows():
    c = _config5_full()
    got = _run(c, True)
    rng = np.random.default_rng(11)
    worst = 0.0
    # every one of the 256 heads: two rows each, in query tiles that rotate with the head index, so every
    # (head) and every one of the 16 query tiles (both tiles of every CTA's pair) is covered many times over
    for i in range(256):
        b, h = divmod(i, 32)
        rows = np.array([(i % 16) * 128 + (29 * i) % 128, ((i + 7) % 16) * 128 + (53 * i + 11) % 128])
        if i % 64 == 0:
            rows = np.unique(np.concatenate([rows, [0, 127, 128, 2047], rng.integers(0, 2048, 12)]))
        want = O.attention_head(c["q"][b, h], c["k"][b, h], c["v"][b, h], scale=c["scale"], causal=True, rows=rows)
        worst = max(worst, check_bf16(got[b, h][rows], want, what=f"config 5 head ({b},{h})"))
    assert worst < 2e-2


def test_rejections():
    import paper_2511_16964_b200 as P
    q = torch.zeros((1, 1, 16, 96), device="cuda", dtype=BF16)
    with pytest.raises(P.PikeError) as e:                 # head dimension other than 64 or 128
        P.pike_attention_chain(q, q.clone(), q.clone(), scale=1.0)
    assert e.value.code == 6
    q = torch.zeros((1, 1, 16, 128), device="cuda", dtype=BF16)
    with pytest.raises(P.PikeError) as e:                 # v does not have k's sequence length
        P.pike_attention_chain(q, torch.zeros((1, 1, 32, 128), device="cuda", dtype=BF16), q.clone(), scale=1.0,
                               causal=False)
    assert e.value.code == 2
    with pytest.raises(P.PikeError) as e:                 # non-positive scale
        P.pike_attention_chain(q, q.clone(), q.clone(), scale=0.0)
    assert e.value.code == 6
    assert P.pike_attention_chain_workspace(q, scale=1.0) == 0


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("pattern", ["rising", "falling", "late spike", "huge scores"])
def test_row_maxima_that_move_between_key_tiles(pattern, dtype):
    """The accumulator is only rescaled when a row's maximum grows by more than a threshold (lazy rescale): keys
    whose scores rise steadily from tile to tile force a rescale at every step, falling ones none after the first,
    a single late key with a far larger score makes everything before it vanish, and scores in the hundreds leave
    one probability per row.  All four must come out like the plain definition."""
    import paper_2511_16964_b200 as P
    tdt = BF16 if dtype == "bf16" else torch.float16
    S, D = 5 * 128 + 37, 128
    c = G.config5(B=1, H=2, S=S, D=D, seed=77, dtype=dtype)
    k = c["k"].astype(np.float64)
    tile = np.arange(S) // 128
    if pattern == "rising":
        k *= (1.0 + 2.0 * tile)[None, None, :, None]
    elif pattern == "falling":
        k *= (1.0 + 2.0 * tile[::-1])[None, None, :, None]
    elif pattern == "late spike":
        k[:, :, 4 * 128 + 5, :] = 6.0 * np.sign(c["q"][:, :, -1:, :].astype(np.float64).mean(axis=2))
    else:
        k *= 16.0
    k = G.round_to(k.astype(np.float32), dtype)
    scale = 1.0 if pattern == "huge scores" else c["scale"]
    for causal in (False, True):
        got = host64(P.pike_attention_chain(dev(c["q"], tdt), dev(k, tdt), dev(c["v"], tdt), scale=scale, causal=causal))
        assert P.pike_get_last_device_status() == (0, 0)
        want = O.attention(c["q"], k, c["v"], scale=scale, causal=causal)
        check_bf16(got, want, what=f"{pattern} {dtype} causal={causal}")
