"""numpy front end of the fp64 CPU oracle (TEST INFRASTRUCTURE ONLY).

Compiles ``pike_oracle.c`` with gcc on first use and exposes its functions on
numpy arrays.  Nothing here is imported by the CUDA package; only the tests,
the smoke check and the bench's CPU-baseline leg may use it.

Every function takes any real dtype and upcasts to float64 (bf16 inputs are
passed as float32 arrays holding bf16-representable values, so the upcast is
exact) and returns float64.  ``rows=`` selects a subset of output rows; rows
are independent in every chain, so the subset is exact for those rows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pike_oracle.c")
_LIB = os.path.join(_HERE, "_pike_oracle.so")
_lock = threading.Lock()
_lib = None

ACT = {"none": 0, "gelu_erf": 1, "gelu_tanh": 2, "silu": 3}
REDUCE = {"none": 0, "layernorm": 1, "softmax": 2}


def build(force: bool = False) -> str:
    """Compile the C oracle into a shared object next to its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=gnu99", "-ffp-contract=off",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            d, dp, lp = ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p
            L, I = ctypes.c_long, ctypes.c_int
            for name in ("oracle_gelu_erf", "oracle_gelu_tanh", "oracle_silu"):
                getattr(lib, name).restype = d
                getattr(lib, name).argtypes = [d]
            lib.oracle_linear.restype = None
            lib.oracle_linear.argtypes = [dp, dp, dp, dp, L, L, L]
            lib.oracle_layernorm_rows.restype = None
            lib.oracle_layernorm_rows.argtypes = [dp, L, L, dp, dp, d]
            lib.oracle_softmax_rows.restype = None
            lib.oracle_softmax_rows.argtypes = [dp, L, L]
            lib.oracle_linear_epilogue.restype = None
            lib.oracle_linear_epilogue.argtypes = [dp, dp, dp, dp, dp, dp, I, d, I, d, dp, L, L, L]
            lib.oracle_mlp_block.restype = I
            lib.oracle_mlp_block.argtypes = [dp, dp, dp, d, dp, dp, dp, dp, I, dp, L, L, L]
            lib.oracle_attention_block.restype = I
            lib.oracle_attention_block.argtypes = [dp, dp, dp, d, dp, dp, dp, dp, d, I, dp, L, L, L]
            lib.oracle_attention_rows.restype = I
            lib.oracle_attention_rows.argtypes = [dp, lp, L, dp, dp, L, L, d, I, dp]
            _lib = lib
    return _lib


def _f64(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    """Threads the OpenMP runtime will use for the row loops."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else (os.cpu_count() or 1)


# -- scalar activations -------------------------------------------------------
def gelu_erf(y: float) -> float:
    return _load().oracle_gelu_erf(float(y))


def gelu_tanh(y: float) -> float:
    return _load().oracle_gelu_tanh(float(y))


def silu(y: float) -> float:
    return _load().oracle_silu(float(y))


# -- building blocks ----------------------------------------------------------
def linear(x, w, b=None):
    x, w, b = _f64(x), _f64(w), _f64(b)
    M, K = x.shape
    K2, N = w.shape
    assert K == K2 and (b is None or b.shape == (N,))
    y = np.empty((M, N), np.float64)
    _load().oracle_linear(_p(x), _p(w), _p(b), _p(y), M, K, N)
    return y


def layernorm(v, gamma=None, beta=None, eps=1e-5):
    v = np.array(v, dtype=np.float64, order="C", copy=True)
    M, N = v.shape
    gamma, beta = _f64(gamma), _f64(beta)
    _load().oracle_layernorm_rows(_p(v), M, N, _p(gamma), _p(beta), float(eps))
    return v


def softmax(v):
    v = np.array(v, dtype=np.float64, order="C", copy=True)
    M, N = v.shape
    _load().oracle_softmax_rows(_p(v), M, N)
    return v


# -- chains ---------------------------------------------------------------------
def linear_epilogue(x, w, bias=None, residual=None, gamma=None, beta=None, *, act="none",
                    scale=1.0, reduce="none", eps=1e-5, rows=None):
    """out = reduce( scale*act(x @ w + bias) + residual ),  w is [K,N]."""
    if rows is not None:
        rows = np.asarray(rows, dtype=np.int64)
        x = np.asarray(x)[rows]
        residual = None if residual is None else np.asarray(residual)[rows]
    x, w, bias, residual = _f64(x), _f64(w), _f64(bias), _f64(residual)
    gamma, beta = _f64(gamma), _f64(beta)
    M, K = x.shape
    N = w.shape[1]
    assert w.shape[0] == K
    out = np.empty((M, N), np.float64)
    _load().oracle_linear_epilogue(_p(x), _p(w), _p(bias), _p(residual), _p(gamma), _p(beta),
                                   ACT[act], float(scale), REDUCE[reduce], float(eps),
                                   _p(out), M, K, N)
    return out


def mlp_block(x, gamma, beta, w1, b1, w2, b2, *, act="gelu_tanh", eps=1e-5, rows=None):
    """out = x + act(LN(x) @ w1 + b1) @ w2 + b2  (pre-LN block, un-normalised residual)."""
    if rows is not None:
        x = np.asarray(x)[np.asarray(rows, dtype=np.int64)]
    x, gamma, beta = _f64(x), _f64(gamma), _f64(beta)
    w1, b1, w2, b2 = _f64(w1), _f64(b1), _f64(w2), _f64(b2)
    M, D = x.shape
    F = w1.shape[1]
    assert w1.shape == (D, F) and w2.shape == (F, D)
    out = np.empty((M, D), np.float64)
    rc = _load().oracle_mlp_block(_p(x), _p(gamma), _p(beta), float(eps), _p(w1), _p(b1),
                                  _p(w2), _p(b2), ACT[act], _p(out), M, D, F)
    if rc:
        raise MemoryError("oracle_mlp_block: allocation failed")
    return out


def attention_head(q, k, v, *, scale, causal, rows=None):
    """One head: q,k,v [S,D] -> O[rows,D] (all rows if rows is None)."""
    q, k, v = np.asarray(q), _f64(k), _f64(v)
    S, D = k.shape
    pos = np.arange(q.shape[0], dtype=np.int64) if rows is None else np.asarray(rows, dtype=np.int64)
    if causal:
        assert q.shape[0] == S, "causal attention needs S_q == S_k"
    qr = _f64(q[pos])
    pos = np.ascontiguousarray(pos, dtype=np.int64)
    out = np.empty((len(pos), D), np.float64)
    rc = _load().oracle_attention_rows(_p(qr), pos.ctypes.data_as(ctypes.c_void_p), len(pos),
                                       _p(k), _p(v), S, D, float(scale), int(bool(causal)), _p(out))
    if rc:
        raise MemoryError("oracle_attention_rows: allocation failed")
    return out


def attention(q, k, v, *, scale, causal):
    """q,k,v [B,H,S,D] -> O [B,H,S,D], every head through attention_head."""
    q, k, v = np.asarray(q), np.asarray(k), np.asarray(v)
    B, H, S, D = q.shape
    out = np.empty((B, H, S, D), np.float64)
    for b in range(B):
        for h in range(H):
            out[b, h] = attention_head(q[b, h], k[b, h], v[b, h], scale=scale, causal=causal)
    return out


def attention_block(x, gamma, beta, w_qkv, b_qkv, w_o, b_o, *, num_heads, scale, causal, eps=1e-5):
    """x [B,S,E] -> x + attention(LN(x) @ w_qkv + b_qkv) @ w_o + b_o; qkv columns are q | k | v, heads contiguous."""
    x = _f64(x)
    B, S, E = x.shape
    gamma, beta, w_qkv, b_qkv, w_o, b_o = (_f64(a) for a in (gamma, beta, w_qkv, b_qkv, w_o, b_o))
    assert w_qkv.shape == (E, 3 * E) and w_o.shape == (E, E) and E % num_heads == 0
    out = np.empty((B, S, E), np.float64)
    for b in range(B):
        xb, ob = np.ascontiguousarray(x[b]), np.empty((S, E), np.float64)
        rc = _load().oracle_attention_block(_p(xb), _p(gamma), _p(beta), float(eps), _p(w_qkv), _p(b_qkv), _p(w_o),
                                            _p(b_o), float(scale), int(bool(causal)), _p(ob), S, E, num_heads)
        if rc:
            raise MemoryError("oracle_attention_block: allocation failed")
        out[b] = ob
    return out


def grouped_linear_epilogue(x, w, bias, residual, offsets, *, act="none", scale=1.0):
    """Rows offsets[g]..offsets[g+1] of x go through weight matrix w[g] ([G,K,N]) and bias row bias[g]:
    out[r] = scale*act(x[r] @ w[g] + bias[g]) + residual[r].  Each group is one call of the linear chain."""
    x, w = np.asarray(x), np.asarray(w)
    offsets = [int(o) for o in offsets]
    G, K, N = w.shape
    assert len(offsets) == G + 1 and offsets[0] == 0 and offsets[-1] == x.shape[0]
    out = np.zeros((x.shape[0], N), np.float64)
    for g in range(G):
        lo, hi = offsets[g], offsets[g + 1]
        assert lo <= hi
        if hi > lo:
            out[lo:hi] = linear_epilogue(x[lo:hi], w[g], None if bias is None else np.asarray(bias)[g],
                                         None if residual is None else np.asarray(residual)[lo:hi],
                                         act=act, scale=scale)
    return out


def softmax_shard_stats(x, w_shard, bias_shard=None, *, act="none", scale=1.0, rows=None):
    """One GPU's half of a softmax whose columns are split over GPUs: the un-normalised values
    v = scale*act(x @ w_shard + bias_shard) of the slice and, per row, (max_n v, sum_n exp(v - max))."""
    v = linear_epilogue(x, w_shard, bias_shard, act=act, scale=scale, rows=rows)
    m = v.max(axis=1)
    l = np.exp(v - m[:, None]).sum(axis=1)
    return v, np.stack([m, l], axis=1)


def softmax_shard_finish(v, all_stats):
    """Second half: all_stats [R,M,2] holds every slice's (max, sum) per row;
    m = max_r m_r, l = sum_r l_r*exp(m_r - m), result exp(v - m)/l for this slice's columns."""
    all_stats = _f64(all_stats)
    m = all_stats[:, :, 0].max(axis=0)
    l = (all_stats[:, :, 1] * np.exp(all_stats[:, :, 0] - m[None, :])).sum(axis=0)
    return np.exp(_f64(v) - m[:, None]) / l[:, None]
