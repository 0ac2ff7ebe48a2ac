"""Seeded synthetic inputs for the fused-chain workloads.

This module only *draws numbers*: it holds none of the chains' arithmetic (no
matmul, activation, normalisation or attention).  Both the CPU oracle's tests
and the CUDA path's tests/bench take their inputs from here so that the two
sides see bit-identical tensors without sharing any other code.

Generator (counter based, stateless, so any element can be produced alone):

    r(c)  = mix(mix(seed) ^ (tensor_id << 40) ^ c)        c < 2**40
    mix(z) = splitmix64 output function applied to z + golden-ratio increment
    u0(c) = (r(c) >> 11) * 2**-53            in [0, 1)   (uniform draws)
    u1(c) = ((r(c) >> 11) + 1) * 2**-53      in (0, 1]   (log argument)

    uniform element i  = -a + 2a*u0(i)                     in [-a, a)
    normal  element i  = sqrt(-2 ln u1(2i)) * cos(2 pi u0(2i+1))   (Box-Muller)

Values are computed in fp64, rounded to fp32 (round-to-nearest-even) and, for
16-bit tensors, rounded again to bf16 or to IEEE binary16 ("f16") (RNE).  The
rounded value *is* the input: 16-bit tensors are returned as float32 arrays
holding exactly representable values, so an fp64 consumer can upcast them
exactly.

The paper measures on KernelBench models, whose task files are not reproduced
here; the five workloads below are synthetic stand-ins with the shapes and
value distributions of MLP-, logits- and causal-attention-type inference
chains (dense weights, no sparsity, no structure).
"""
from __future__ import annotations

import numpy as np

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GAMMA = np.uint64(0x9E3779B97F4A7C15)
_CHUNK = 1 << 22


def _mix(z: np.ndarray) -> np.ndarray:
    """splitmix64 output function (Steele, Lea, Flood 2014), vectorised."""
    z = (z + _GAMMA).astype(np.uint64)
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _key(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = _mix(np.array([seed], dtype=np.uint64))[0]
    return np.uint64(int(k) ^ ((tensor_id & 0xFFFFFF) << 40))


def _raw(key: np.uint64, counters: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        return _mix(counters.astype(np.uint64) ^ key)


def round_to_bf16(x32: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result is
    float32 with the low 16 bits cleared."""
    bits = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def round_to_f16(x32: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest IEEE binary16 (ties to even); result is float32."""
    return np.ascontiguousarray(x32, dtype=np.float32).astype(np.float16).astype(np.float32)


def round_to(x32: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x32)
    if dtype == "f16":
        return round_to_f16(x32)
    if dtype == "f32":
        return np.ascontiguousarray(x32, dtype=np.float32)
    raise ValueError(f"dtype must be 'f32', 'bf16' or 'f16', got {dtype!r}")


def _finish(v64: np.ndarray, dtype: str) -> np.ndarray:
    return round_to(v64.astype(np.float32), dtype)


def uniform(shape, a: float, *, seed: int, tensor_id: int, dtype: str) -> np.ndarray:
    """U[-a, a) tensor; element i (row-major) uses counter i."""
    n = int(np.prod(shape, dtype=np.int64))
    out = np.empty(n, dtype=np.float32)
    key = _key(seed, tensor_id)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        c = np.arange(lo, hi, dtype=np.uint64)
        u0 = (_raw(key, c) >> np.uint64(11)).astype(np.float64) * 2.0 ** -53
        out[lo:hi] = _finish(-a + 2.0 * a * u0, dtype)
    return out.reshape(shape)


def normal(shape, *, seed: int, tensor_id: int, dtype: str) -> np.ndarray:
    """N(0,1) tensor; element i uses counters 2i and 2i+1."""
    n = int(np.prod(shape, dtype=np.int64))
    out = np.empty(n, dtype=np.float32)
    key = _key(seed, tensor_id)
    for lo in range(0, n, _CHUNK):
        hi = min(n, lo + _CHUNK)
        c = np.arange(lo, hi, dtype=np.uint64) * np.uint64(2)
        u1 = ((_raw(key, c) >> np.uint64(11)).astype(np.float64) + 1.0) * 2.0 ** -53
        u0 = (_raw(key, c + np.uint64(1)) >> np.uint64(11)).astype(np.float64) * 2.0 ** -53
        out[lo:hi] = _finish(np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u0), dtype)
    return out.reshape(shape)


# ----------------------------------------------------------------------------
# The five workloads (tensor ids are fixed so tensors of one config differ).
# Every function takes optional size overrides so the tests can draw small,
# ragged versions of the same recipe.
# ----------------------------------------------------------------------------

def config1(M=128, K=256, N=256, seed=0):
    """fp32 Linear + bias + GELU(erf) + LayerNorm."""
    return dict(
        x=normal((M, K), seed=seed, tensor_id=1, dtype="f32"),
        w=uniform((K, N), 1.0 / 16, seed=seed, tensor_id=2, dtype="f32"),
        b=uniform((N,), 1.0 / 16, seed=seed, tensor_id=3, dtype="f32"),
        gamma=np.ones((N,), np.float32),
        beta=np.zeros((N,), np.float32),
        eps=1e-5,
    )


def config2(M=4096, K=4096, N=4096, seed=0, dtype="bf16"):
    """16-bit (bf16 unless dtype="f16") Linear + bias + SiLU + scale(0.5) + residual."""
    return dict(
        x=normal((M, K), seed=seed, tensor_id=11, dtype=dtype),
        w=uniform((K, N), 1.0 / 64, seed=seed, tensor_id=12, dtype=dtype),
        b=uniform((N,), 1.0 / 64, seed=seed, tensor_id=13, dtype=dtype),
        r=normal((M, N), seed=seed, tensor_id=14, dtype=dtype),
        scale=0.5,
    )


def config3(M=8192, D=4096, F=16384, seed=0, affine=False, dtype="bf16"):
    """16-bit pre-LN transformer MLP block; weights U(+-1/sqrt(fan_in))."""
    if affine:
        gamma = 1.0 + uniform((D,), 0.5, seed=seed, tensor_id=26, dtype=dtype)
        beta = uniform((D,), 0.1, seed=seed, tensor_id=27, dtype=dtype)
        gamma = round_to(gamma.astype(np.float32), dtype)
    else:
        gamma = np.ones((D,), np.float32)
        beta = np.zeros((D,), np.float32)
    return dict(
        x=normal((M, D), seed=seed, tensor_id=21, dtype=dtype),
        w1=uniform((D, F), 1.0 / np.sqrt(D), seed=seed, tensor_id=22, dtype=dtype),
        b1=uniform((F,), 1.0 / np.sqrt(D), seed=seed, tensor_id=23, dtype=dtype),
        w2=uniform((F, D), 1.0 / np.sqrt(F), seed=seed, tensor_id=24, dtype=dtype),
        b2=uniform((D,), 1.0 / np.sqrt(F), seed=seed, tensor_id=25, dtype=dtype),
        gamma=gamma, beta=beta, eps=1e-5,
    )


def config4(M=2048, K=4096, N=32000, seed=0, dtype="bf16"):
    """16-bit logits GEMM + fp32 row softmax."""
    return dict(
        x=normal((M, K), seed=seed, tensor_id=31, dtype=dtype),
        w=uniform((K, N), 1.0 / 64, seed=seed, tensor_id=32, dtype=dtype),
    )


def config5(B=8, H=32, S=2048, D=128, seed=0, dtype="bf16"):
    """16-bit causal attention."""
    return dict(
        q=normal((B, H, S, D), seed=seed, tensor_id=41, dtype=dtype),
        k=normal((B, H, S, D), seed=seed, tensor_id=42, dtype=dtype),
        v=normal((B, H, S, D), seed=seed, tensor_id=43, dtype=dtype),
        scale=1.0 / np.sqrt(D),
    )


def attention_block(B=4, S=1024, E=2048, seed=0, affine=True, dtype="bf16"):
    """16-bit pre-LN attention block with fused projections (heads of 128); weights U(+-1/sqrt(E))."""
    a = 1.0 / np.sqrt(E)
    if affine:
        gamma = round_to((1.0 + uniform((E,), 0.5, seed=seed, tensor_id=56, dtype=dtype)).astype(np.float32), dtype)
        beta = uniform((E,), 0.1, seed=seed, tensor_id=57, dtype=dtype)
    else:
        gamma, beta = np.ones((E,), np.float32), np.zeros((E,), np.float32)
    return dict(
        x=normal((B, S, E), seed=seed, tensor_id=51, dtype=dtype),
        w_qkv=uniform((E, 3 * E), a, seed=seed, tensor_id=52, dtype=dtype),
        b_qkv=uniform((3 * E,), a, seed=seed, tensor_id=53, dtype=dtype),
        w_o=uniform((E, E), a, seed=seed, tensor_id=54, dtype=dtype),
        b_o=uniform((E,), a, seed=seed, tensor_id=55, dtype=dtype),
        gamma=gamma, beta=beta, eps=1e-5, scale=1.0 / np.sqrt(128.0), num_heads=E // 128,
    )


def grouped_linear(T=16384, K=2048, N=4096, G=32, seed=0, dtype="bf16"):
    """16-bit mixture-of-experts style grouped linear: T rows split over G groups of uneven size (one group is
    empty, sizes are not multiples of the tile), weights U(+-1/sqrt(K))."""
    a = 1.0 / np.sqrt(K)
    # group sizes: seeded uniform weights, one group forced empty, remainder to the last group
    wts = uniform((G,), 0.5, seed=seed, tensor_id=66, dtype="f32").astype(np.float64) + 0.6
    if G > 2:
        wts[G // 2] = 0.0
    sizes = np.floor(wts / wts.sum() * T).astype(np.int64)
    sizes[-1] += T - sizes.sum()
    offsets = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    return dict(
        x=normal((T, K), seed=seed, tensor_id=61, dtype=dtype),
        w=uniform((G, K, N), a, seed=seed, tensor_id=62, dtype=dtype),
        b=uniform((G, N), a, seed=seed, tensor_id=63, dtype=dtype),
        r=normal((T, N), seed=seed, tensor_id=64, dtype=dtype),
        offsets=offsets,
    )
