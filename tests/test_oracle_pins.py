"""Pins for the fp64 CPU oracle.

The paper prints no worked numeric example for any operator chain, so the
oracle is pinned to things outside itself: closed forms and tabulated constants,
invariants, exact integer brute force, 50-digit evaluations with mpmath, and
library routines (numpy / scipy / torch fp64 on the CPU) on small shapes.  The
cases are chosen so that a dropped term, a wrong sign or index, a swapped
epilogue step or a transposed operand fails at least one of them.
"""
import math

import mpmath
import numpy as np
import pytest
import scipy.special
import torch

from oracle import pike_oracle as O

mpmath.mp.dps = 50
RNG = np.random.default_rng(1234)


# ----------------------------------------------------------------------------
# activations
# ----------------------------------------------------------------------------
# Tabulated closed-form values: GELU_erf(y) = y * Phi(y) with Phi the standard
# normal CDF (Phi(1) = 0.841344746068542948..., Phi(2) = 0.977249868051820792...);
# SiLU(1) = 1/(1+1/e); the tanh-form values are 50-digit mpmath evaluations.
ACT_POINTS = [
    ("gelu_erf", 0.0, 0.0),
    ("gelu_erf", 1.0, 0.8413447460685429),
    ("gelu_erf", -1.0, -0.15865525393145707),
    ("gelu_erf", 2.0, 1.9544997361036416),
    ("gelu_tanh", 1.0, 0.8411919906082768),
    ("gelu_tanh", -1.0, -0.15880800939172324),
    ("gelu_tanh", 2.0, 1.954597694087775),
    ("gelu_tanh", 3.0, 2.996362607918227),
    ("silu", 0.0, 0.0),
    ("silu", 1.0, 0.7310585786300049),
    ("silu", -1.0, -0.2689414213699951),
    ("silu", 2.0, 1.7615941559557646),
]


@pytest.mark.parametrize("name,y,want", ACT_POINTS)
def test_activation_known_points(name, y, want):
    assert abs(getattr(O, name)(y) - want) <= 1e-15


def _mp_act(name, y):
    y = mpmath.mpf(y)
    if name == "gelu_erf":
        return y * mpmath.ncdf(y)
    if name == "gelu_tanh":
        return y / 2 * (1 + mpmath.tanh(mpmath.sqrt(2 / mpmath.pi) * (y + mpmath.mpf("0.044715") * y ** 3)))
    return y * (1 / (1 + mpmath.e ** (-y)))


@pytest.mark.parametrize("name", ["gelu_erf", "gelu_tanh", "silu"])
def test_activation_vs_50_digit_evaluation(name):
    for y in np.linspace(-9, 9, 73):
        got = getattr(O, name)(float(y))
        want = float(_mp_act(name, float(y)))
        assert abs(got - want) <= 4e-16 * max(1.0, abs(want)), (name, y)


@pytest.mark.parametrize("name", ["gelu_erf", "gelu_tanh", "silu"])
def test_activation_odd_part_identity_and_limits(name):
    f = getattr(O, name)
    for y in [0.1, 0.5, 1.0, 2.5, 7.0]:
        assert abs(f(y) - f(-y) - y) <= 1e-15 * max(1, y)      # f(y) - f(-y) = y
    assert abs(f(30.0) - 30.0) <= 1e-11 and abs(f(-30.0)) <= 1e-11
    assert not math.isnan(f(-745.0)) and not math.isnan(f(745.0))


def test_gelu_erf_matches_scipy_ndtr():
    y = np.linspace(-6, 6, 101)
    want = y * scipy.special.ndtr(y)
    got = np.array([O.gelu_erf(v) for v in y])
    np.testing.assert_allclose(got, want, rtol=0, atol=2e-15)


# ----------------------------------------------------------------------------
# linear
# ----------------------------------------------------------------------------
def test_linear_integer_brute_force_exact():
    M, K, N = 3, 5, 4                               # all different: catches transposes
    x = RNG.integers(-9, 10, size=(M, K))
    w = RNG.integers(-9, 10, size=(K, N))
    b = RNG.integers(-9, 10, size=(N,))
    want = [[sum(int(x[m, k]) * int(w[k, n]) for k in range(K)) + int(b[n]) for n in range(N)]
            for m in range(M)]
    got = O.linear(x, w, b)
    assert got.shape == (M, N)
    assert (got == np.array(want, dtype=np.float64)).all()


def test_linear_identity_outer_product_and_no_bias():
    x = RNG.standard_normal((4, 6))
    b = RNG.standard_normal(6)
    assert np.array_equal(O.linear(x, np.eye(6), b), x + b)
    assert np.array_equal(O.linear(x, np.eye(6)), x)
    col, row = RNG.standard_normal((5, 1)), RNG.standard_normal((1, 7))
    assert np.array_equal(O.linear(col, row), col * row)       # K = 1


def test_linear_matches_second_loop_order_and_library():
    M, K, N = 7, 33, 19
    x, w, b = RNG.standard_normal((M, K)), RNG.standard_normal((K, N)), RNG.standard_normal(N)
    got = O.linear(x, w, b)
    dot_order = np.array([[math.fsum(x[m, k] * w[k, n] for k in range(K)) + b[n] for n in range(N)]
                          for m in range(M)])
    np.testing.assert_allclose(got, dot_order, rtol=0, atol=1e-13)
    np.testing.assert_allclose(got, x @ w + b, rtol=0, atol=1e-13)


# ----------------------------------------------------------------------------
# LayerNorm
# ----------------------------------------------------------------------------
def test_layernorm_mean_and_variance_closed_form():
    v = RNG.standard_normal((6, 257)) * 3.0 + 1.5
    eps = 1e-5
    z = O.layernorm(v, eps=eps)
    assert np.abs(z.mean(axis=1)).max() <= 1e-12
    var = v.var(axis=1)                              # biased
    np.testing.assert_allclose(z.var(axis=1), var / (var + eps), rtol=1e-12)


def test_layernorm_affine_invariance_constant_row_and_gamma_beta():
    v = RNG.standard_normal((3, 64))
    z0 = O.layernorm(v, eps=0.0)
    np.testing.assert_allclose(O.layernorm(2.5 * v + 7.0, eps=0.0), z0, atol=1e-12)
    np.testing.assert_allclose(O.layernorm(-v, eps=0.0), -z0, atol=1e-12)
    g, b = RNG.standard_normal(64), RNG.standard_normal(64)
    np.testing.assert_allclose(O.layernorm(v, g, b, eps=0.0), z0 * g + b, atol=1e-12)
    const = np.full((2, 64), 3.25)
    np.testing.assert_allclose(O.layernorm(const, g, b, eps=1e-5), np.broadcast_to(b, (2, 64)), atol=1e-12)


def test_layernorm_eps_inside_sqrt_and_library():
    v = RNG.standard_normal((5, 48)) * 0.01           # small variance: eps placement matters
    g, b = RNG.standard_normal(48), RNG.standard_normal(48)
    want = torch.nn.functional.layer_norm(torch.from_numpy(v), (48,), torch.from_numpy(g),
                                          torch.from_numpy(b), eps=1e-3).numpy()
    np.testing.assert_allclose(O.layernorm(v, g, b, eps=1e-3), want, atol=1e-12)
    # a two-element row has a closed form: (+-d/2)/sqrt(d^2/4 + eps)
    d, eps = 0.2, 0.01
    z = O.layernorm(np.array([[1.0, 1.0 + d]]), eps=eps)
    want = (d / 2) / math.sqrt(d * d / 4 + eps)
    np.testing.assert_allclose(z, [[-want, want]], atol=1e-14)


# ----------------------------------------------------------------------------
# softmax
# ----------------------------------------------------------------------------
def test_softmax_invariants():
    v = RNG.standard_normal((5, 301)) * 4
    p = O.softmax(v)
    assert np.abs(p.sum(axis=1) - 1).max() <= 1e-12
    assert (p > 0).all() and (p <= 1).all()
    for c in (3.0, 1e4, -1e4):
        np.testing.assert_allclose(O.softmax(v + c), p, rtol=1e-9, atol=0)
    assert np.isfinite(O.softmax(v * 1e3)).all()
    np.testing.assert_allclose(O.softmax(np.full((2, 9), -4.0)), np.full((2, 9), 1 / 9), atol=1e-15)
    assert (np.argmax(p, axis=1) == np.argmax(v, axis=1)).all()


def test_softmax_two_element_logistic_and_library():
    a, b = 0.3, -1.1
    p = O.softmax(np.array([[a, b]]))
    np.testing.assert_allclose(p[0, 0], 1 / (1 + math.exp(b - a)), atol=1e-15)
    v = RNG.standard_normal((4, 37))
    np.testing.assert_allclose(O.softmax(v), scipy.special.softmax(v, axis=1), atol=1e-15)


# ----------------------------------------------------------------------------
# attention
# ----------------------------------------------------------------------------
def _qkv(S, D):
    return (RNG.standard_normal((S, D)), RNG.standard_normal((S, D)), RNG.standard_normal((S, D)))


def test_attention_special_cases():
    S, D = 9, 5
    q, k, v = _qkv(S, D)
    sc = 1 / math.sqrt(D)
    o = O.attention_head(q, k, v, scale=sc, causal=True)
    np.testing.assert_allclose(o[0], v[0], atol=1e-15)                  # row 0 sees only key 0
    ones = O.attention_head(q, k, np.ones((S, D)), scale=sc, causal=True)
    np.testing.assert_allclose(ones, 1.0, atol=1e-14)                   # V == 1 -> O == 1
    run_mean = np.cumsum(v, axis=0) / np.arange(1, S + 1)[:, None]
    np.testing.assert_allclose(O.attention_head(np.zeros((S, D)), k, v, scale=sc, causal=True),
                               run_mean, atol=1e-14)                    # Q == 0 -> running mean
    same_k = np.broadcast_to(k[:1], (S, D))
    np.testing.assert_allclose(O.attention_head(q, same_k, v, scale=sc, causal=True), run_mean, atol=1e-14)
    np.testing.assert_allclose(O.attention_head(q[:1], k[:1], v[:1], scale=sc, causal=False), v[:1], atol=1e-15)
    full = O.attention_head(q, k, v, scale=sc, causal=False)
    perm = RNG.permutation(S)
    np.testing.assert_allclose(O.attention_head(q, k[perm], v[perm], scale=sc, causal=False), full, atol=1e-14)
    # the last causal row sees every key, so it equals the non-causal last row
    np.testing.assert_allclose(o[-1], full[-1], atol=1e-14)


def test_attention_equals_explicit_masked_dense_form_and_row_subset():
    S, D = 13, 7
    q, k, v = _qkv(S, D)
    sc = 0.37
    for causal in (False, True):
        s = O.linear(q, k.T) * sc                      # scores through the matmul oracle
        if causal:
            s[np.triu_indices(S, 1)] = -np.inf
        want = O.linear(O.softmax(s), v)
        got = O.attention_head(q, k, v, scale=sc, causal=causal)
        np.testing.assert_allclose(got, want, atol=1e-14)
        rows = [12, 0, 5]
        np.testing.assert_array_equal(O.attention_head(q, k, v, scale=sc, causal=causal, rows=rows), got[rows])


def test_attention_matches_library_sdpa_fp64():
    B, H, S, D = 2, 3, 17, 8
    q, k, v = (RNG.standard_normal((B, H, S, D)) for _ in range(3))
    sc = 1 / math.sqrt(D)
    for causal in (False, True):
        want = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=causal, scale=sc).numpy()
        np.testing.assert_allclose(O.attention(q, k, v, scale=sc, causal=causal), want, atol=1e-13)


def test_attention_scale_is_applied_before_softmax():
    S, D = 6, 4
    q, k, v = _qkv(S, D)
    a = O.attention_head(q, k, v, scale=0.5, causal=True)
    b = O.attention_head(q * 0.5, k, v, scale=1.0, causal=True)
    np.testing.assert_allclose(a, b, atol=1e-14)
    assert np.abs(a - O.attention_head(q, k, v, scale=1.0, causal=True)).max() > 1e-3


# ----------------------------------------------------------------------------
# chains
# ----------------------------------------------------------------------------
def test_linear_epilogue_special_cases_fix_the_step_order():
    M, K, N = 4, 6, 6
    x, w = RNG.standard_normal((M, K)), RNG.standard_normal((K, N))
    b, r = RNG.standard_normal(N), RNG.standard_normal((M, N))
    np.testing.assert_array_equal(O.linear_epilogue(x, w, b, r, act="silu", scale=0.0), r)
    np.testing.assert_array_equal(O.linear_epilogue(x, np.eye(K)), x)
    # x = 0: out = scale*act(bias) + residual -> bias is inside the activation,
    # scale is outside it and the residual is outside the scale
    got = O.linear_epilogue(np.zeros((M, K)), w, b, r, act="gelu_erf", scale=0.5)
    want = 0.5 * (b * scipy.special.ndtr(b)) + r
    np.testing.assert_allclose(got, want, atol=1e-15)
    rows = [3, 1]
    full = O.linear_epilogue(x, w, b, r, act="gelu_tanh", scale=0.5, reduce="layernorm")
    np.testing.assert_array_equal(O.linear_epilogue(x, w, b, r, act="gelu_tanh", scale=0.5,
                                                    reduce="layernorm", rows=rows), full[rows])


@pytest.mark.parametrize("act,reduce", [("gelu_erf", "layernorm"), ("silu", "none"), ("none", "softmax"),
                                        ("gelu_tanh", "none")])
def test_linear_epilogue_matches_library_composition(act, reduce):
    M, K, N = 5, 24, 12
    t = lambda a: torch.from_numpy(a)
    x, w = RNG.standard_normal((M, K)), RNG.standard_normal((K, N)) / 4
    b, r = RNG.standard_normal(N), RNG.standard_normal((M, N))
    g, be = RNG.standard_normal(N), RNG.standard_normal(N)
    y = t(x) @ t(w) + t(b)
    F = torch.nn.functional
    y = {"gelu_erf": lambda v: F.gelu(v), "gelu_tanh": lambda v: F.gelu(v, approximate="tanh"),
         "silu": F.silu, "none": lambda v: v}[act](y)
    y = 0.75 * y + t(r)
    if reduce == "layernorm":
        y = F.layer_norm(y, (N,), t(g), t(be), eps=1e-5)
    elif reduce == "softmax":
        y = torch.softmax(y, dim=-1)
    got = O.linear_epilogue(x, w, b, r, g, be, act=act, scale=0.75, reduce=reduce, eps=1e-5)
    np.testing.assert_allclose(got, y.numpy(), atol=1e-13)


def test_mlp_block_special_cases_and_library_composition():
    M, D, Fh = 4, 10, 14
    t = lambda a: torch.from_numpy(a)
    x = RNG.standard_normal((M, D)) * 2 + 0.5
    g, be = RNG.standard_normal(D), RNG.standard_normal(D)
    w1, b1 = RNG.standard_normal((D, Fh)) / 3, RNG.standard_normal(Fh)
    w2, b2 = RNG.standard_normal((Fh, D)) / 3, RNG.standard_normal(D)
    # W2 = 0 -> out = x + b2 (the residual is the un-normalised input)
    np.testing.assert_allclose(O.mlp_block(x, g, be, w1, b1, np.zeros((Fh, D)), b2), x + b2, atol=1e-15)
    F = torch.nn.functional
    z = F.layer_norm(t(x), (D,), t(g), t(be), eps=1e-5)
    want = t(x) + F.gelu(z @ t(w1) + t(b1), approximate="tanh") @ t(w2) + t(b2)
    got = O.mlp_block(x, g, be, w1, b1, w2, b2, act="gelu_tanh", eps=1e-5)
    np.testing.assert_allclose(got, want.numpy(), atol=1e-13)
    np.testing.assert_array_equal(O.mlp_block(x, g, be, w1, b1, w2, b2, rows=[2, 0]), got[[2, 0]])


def test_attention_block_special_cases_and_library_composition():
    B, S, E, H = 2, 7, 12, 3
    Dh = E // H
    t = lambda a: torch.from_numpy(a)
    x = RNG.standard_normal((B, S, E)) * 1.5 + 0.3
    g, be = RNG.standard_normal(E), RNG.standard_normal(E)
    wq, bq = RNG.standard_normal((E, 3 * E)) / 3, RNG.standard_normal(3 * E)
    wo, bo = RNG.standard_normal((E, E)) / 3, RNG.standard_normal(E)
    kw = dict(num_heads=H, scale=0.4, eps=1e-5)
    # w_o = 0 -> out = x + b_o: the residual is the un-normalised input and the bias is outside the attention
    np.testing.assert_allclose(O.attention_block(x, g, be, wq, bq, np.zeros((E, E)), bo, causal=True, **kw), x + bo, atol=1e-15)
    F = torch.nn.functional
    for causal in (True, False):
        z = F.layer_norm(t(x), (E,), t(g), t(be), eps=1e-5)
        qkv = z @ t(wq) + t(bq)
        q, k, v = (qkv[..., i * E:(i + 1) * E].reshape(B, S, H, Dh).permute(0, 2, 1, 3) for i in range(3))
        a = F.scaled_dot_product_attention(q, k, v, is_causal=causal, scale=0.4).permute(0, 2, 1, 3).reshape(B, S, E)
        want = t(x) + a @ t(wo) + t(bo)
        got = O.attention_block(x, g, be, wq, bq, wo, bo, causal=causal, **kw)
        np.testing.assert_allclose(got, want.numpy(), atol=1e-12)
    # causal: the first position attends to itself only, so its output does not depend on later positions
    x2 = x.copy()
    x2[:, 1:] += 1.0
    a1 = O.attention_block(x, g, be, wq, bq, wo, bo, causal=True, **kw)
    a2 = O.attention_block(x2, g, be, wq, bq, wo, bo, causal=True, **kw)
    np.testing.assert_allclose(a1[:, 0], a2[:, 0], atol=1e-13)


def test_grouped_linear_matches_per_group_library_matmul_and_single_group_case():
    T, K, N, Gn = 11, 6, 5, 4
    x, w = RNG.standard_normal((T, K)), RNG.standard_normal((Gn, K, N))
    b, r = RNG.standard_normal((Gn, N)), RNG.standard_normal((T, N))
    offsets = [0, 3, 3, 9, 11]                                   # one empty group
    got = O.grouped_linear_epilogue(x, w, b, r, offsets, act="silu", scale=0.5)
    for g in range(Gn):
        lo, hi = offsets[g], offsets[g + 1]
        y = torch.from_numpy(x[lo:hi]) @ torch.from_numpy(w[g]) + torch.from_numpy(b[g])
        want = 0.5 * torch.nn.functional.silu(y) + torch.from_numpy(r[lo:hi])
        np.testing.assert_allclose(got[lo:hi], want.numpy(), atol=1e-13)
    # a row moved to another group changes (only) that row
    got2 = O.grouped_linear_epilogue(x, w, b, r, [0, 2, 3, 9, 11], act="silu", scale=0.5)
    assert np.abs(got2[2] - got[2]).max() > 1e-3 and np.array_equal(np.delete(got2, 2, 0), np.delete(got, 2, 0))
    one = O.grouped_linear_epilogue(x, w[:1], b[:1], r, [0, T], act="gelu_tanh")
    np.testing.assert_array_equal(one, O.linear_epilogue(x, w[0], b[0], r, act="gelu_tanh"))
