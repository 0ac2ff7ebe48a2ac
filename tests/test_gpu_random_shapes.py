"""Randomised sweep: seeded random shapes, types, layouts and epilogue flags through every entry point, each result
compared with the fp64 oracle at the contractual tolerance.  The fixed cases of the other files aim at the tile
boundaries on purpose; this one looks for what nobody aimed at."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, check_f32, dev, host64

pytestmark = pytest.mark.gpu
BF16, F16, F32 = torch.bfloat16, torch.float16, torch.float32


def _pick(rng, *a):
    return a[int(rng.integers(len(a)))]


def _dim(rng, lo, hi, mult=1):
    return max(mult, int(rng.integers(lo, hi + 1)) // mult * mult)


@pytest.mark.parametrize("seed", range(4))
def test_random_16bit_linear_chains(seed):
    import paper_2511_16964_b200 as P
    rng = np.random.default_rng(100 + seed)
    for case in range(30):
        dt = _pick(rng, "bf16", "f16")
        tdt = BF16 if dt == "bf16" else F16
        M, K, N = _dim(rng, 1, 700), _dim(rng, 8, 1100, 8), _dim(rng, 8, 1300, 8)
        c = G.config2(M=M, K=K, N=N, seed=1000 * seed + case, dtype=dt)
        act = _pick(rng, "none", "silu", "gelu_tanh", "gelu_erf")
        red = _pick(rng, "none", "none", "softmax", "layernorm")
        nk, use_b = bool(rng.integers(2)), bool(rng.integers(2))
        use_r = bool(rng.integers(2)) and red != "softmax"
        odt = F32 if (red == "softmax" or rng.integers(3) == 0) else tdt
        scale = float(_pick(rng, 1.0, 0.5, 1.75))
        gam = bet = None
        if red == "layernorm":
            gam = G.round_to((G.uniform((N,), 0.5, seed=seed, tensor_id=90, dtype=dt) + 1.0).astype(np.float32), dt)
            bet = G.uniform((N,), 0.2, seed=seed, tensor_id=91, dtype=dt)
        w = c["w"]
        got = P.pike_linear_epilogue(dev(c["x"], tdt), dev(w.T.copy() if nk else w, tdt), dev(c["b"], tdt) if use_b else None,
                                     dev(c["r"], tdt) if use_r else None, dev(gam, tdt), dev(bet, tdt), act=act, scale=scale,
                                     reduce=red, eps=1e-5, out_dtype=odt, w_is_nk=nk)
        want = O.linear_epilogue(c["x"], w, c["b"] if use_b else None, c["r"] if use_r else None, gam, bet, act=act,
                                 scale=scale, reduce=red, eps=1e-5)
        what = f"{dt} {M}x{K}x{N} act={act} reduce={red} nk={nk} bias={use_b} res={use_r} out={odt} scale={scale}"
        if red == "softmax":
            g = host64(got)
            assert np.abs(g - want).max() <= 1e-3 * want.max() + 1e-7 and np.abs(g.sum(1) - 1).max() <= 1e-5, what
        else:
            check_bf16(host64(got), want, what=what)
    assert P.pike_get_last_device_status() == (0, 0)


@pytest.mark.parametrize("seed", range(4))
def test_random_attention(seed):
    import paper_2511_16964_b200 as P
    rng = np.random.default_rng(200 + seed)
    for case in range(25):
        dt = _pick(rng, "bf16", "f16")
        tdt = BF16 if dt == "bf16" else F16
        D, B, H = _pick(rng, 64, 128), _dim(rng, 1, 2), _dim(rng, 1, 3)
        causal = bool(rng.integers(2))
        S = _dim(rng, 1, 600)
        Sk = S if (causal or rng.integers(2)) else _dim(rng, 1, 700)
        ds = 1000 * seed + case
        q = G.normal((B, H, S, D), seed=ds, tensor_id=41, dtype=dt)
        k = G.normal((B, H, Sk, D), seed=ds, tensor_id=42, dtype=dt)
        v = G.normal((B, H, Sk, D), seed=ds, tensor_id=43, dtype=dt)
        scale = float(_pick(rng, D ** -0.5, 0.3, 1.0))
        bshd = bool(rng.integers(2))          # [B,S,H,D] storage viewed as [B,H,S,D]

        def mk(a):
            t = dev(a, tdt)
            return t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3) if bshd else t

        got = host64(P.pike_attention_chain(mk(q), mk(k), mk(v), scale=scale, causal=causal))
        for b in range(B):
            for h in range(H):
                want = O.attention_head(q[b, h], k[b, h], v[b, h], scale=scale, causal=causal)
                check_bf16(got[b, h], want, what=f"{dt} B{B} H{H} S{S} Sk{Sk} D{D} causal={causal} scale={scale:.3f} bshd={bshd}")
    assert P.pike_get_last_device_status() == (0, 0)


@pytest.mark.parametrize("seed", range(3))
def test_random_blocks_fp32_chains_and_groups(seed):
    import paper_2511_16964_b200 as P
    rng = np.random.default_rng(300 + seed)
    for case in range(12):
        ds = 1000 * seed + case
        # pre-LN MLP block
        dt = _pick(rng, "bf16", "f16")
        tdt = BF16 if dt == "bf16" else F16
        M, D, F = _dim(rng, 1, 500), _dim(rng, 8, 520, 8), _dim(rng, 8, 1100, 8)
        c = G.config3(M=M, D=D, F=F, seed=ds, affine=True, dtype=dt)
        act = _pick(rng, "gelu_tanh", "silu", "gelu_erf")
        got = P.pike_mlp_block(*(dev(c[n], tdt) for n in ("x", "gamma", "beta", "w1", "b1", "w2", "b2")), act=act, eps=c["eps"])
        check_bf16(host64(got), O.mlp_block(c["x"], c["gamma"], c["beta"], c["w1"], c["b1"], c["w2"], c["b2"], act=act, eps=c["eps"]),
                   what=f"mlp {dt} {M}x{D}x{F} {act}")
        # fp32 chain
        M, K, N = _dim(rng, 1, 300), _dim(rng, 1, 400), _dim(rng, 1, 1024)
        c = G.config1(M=M, K=K, N=N, seed=ds)
        red, act, nk = _pick(rng, "none", "layernorm", "softmax"), _pick(rng, "none", "gelu_erf", "silu"), bool(rng.integers(2))
        ln = red == "layernorm"
        got = P.pike_linear_epilogue(dev(c["x"], F32), dev(c["w"].T.copy() if nk else c["w"], F32), dev(c["b"], F32), None,
                                     dev(c["gamma"], F32) if ln else None, dev(c["beta"], F32) if ln else None, act=act,
                                     reduce=red, eps=c["eps"], w_is_nk=nk)
        check_f32(host64(got), O.linear_epilogue(c["x"], c["w"], c["b"], None, c["gamma"] if ln else None,
                                                 c["beta"] if ln else None, act=act, reduce=red, eps=c["eps"]),
                  1e-4, f"fp32 {M}x{K}x{N} {act}/{red} nk={nk}")
        # grouped linear
        T, K, N, ng = _dim(rng, 1, 1500), _dim(rng, 8, 520, 8), _dim(rng, 8, 700, 8), _dim(rng, 1, 9)
        c = G.grouped_linear(T=T, K=K, N=N, G=ng, seed=ds)
        act = _pick(rng, "none", "silu")
        got = host64(P.pike_grouped_linear_epilogue(dev(c["x"], BF16), dev(c["w"], BF16), dev(c["b"], BF16), dev(c["r"], BF16),
                                                    torch.from_numpy(c["offsets"]).cuda(), act=act))
        off = c["offsets"]
        for g in range(ng):
            a, b = int(off[g]), int(off[g + 1])
            if b > a:
                check_bf16(got[a:b], O.linear_epilogue(c["x"][a:b], c["w"][g], c["b"][g], c["r"][a:b], act=act),
                           what=f"grouped T{T} K{K} N{N} G{ng} group {g} {act}")
    assert P.pike_get_last_device_status() == (0, 0)
