"""Supplementary gates beside the contractual bf16 bar (|gpu - oracle| <= 2e-2 + 2e-2*|oracle|).

That bar cannot see some mistakes on the benchmark recipes: a bias of at most 1/64 moves the output by
less than the tolerance, so a dropped or mis-indexed bias would pass.  Here every index-heavy path of
the 16-bit GEMM chain is run on small-integer operands INCLUDING bias and residual, with fp32 output and
no activation: every product and partial sum is exact in fp32 and in the oracle's fp64, so the two must
agree bit for bit and any wrong row, column, group or k index shows up as a mismatch.  A tight bound
(< 2e-3) per activation on fp32 outputs covers the activation code the exact cases leave out.  Every
case writes into tensors and workspaces that sit between sentinel bands (compute-sanitizer is not
available where these tests run): a store outside the tensor fails the test.
"""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import Guarded, check_bf16, dev, guarded_workspace, host64, ints

pytestmark = pytest.mark.gpu
BF16, F16, F32 = torch.bfloat16, torch.float16, torch.float32


def _status_ok():
    import paper_2511_16964_b200 as P
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)


def _int_case(M, K, N, seed):
    rng = np.random.default_rng(seed)
    return dict(x=ints(rng, (M, K)), w=ints(rng, (K, N)), b=ints(rng, (N,), -8, 8), r=ints(rng, (M, N), -16, 16))


# (M, K, N): one ragged tile; ragged M/N/K over several tiles; the half-tile round (10 x 8 tiles on 74 clusters,
# last column tile 136 wide); more tiles than clusters with a ragged last column tile; a tall skinny problem
SHAPES = [(128, 64, 256), (300, 192, 328), (2560, 64, 1928), (2560, 256, 2312), (5000, 72, 8)]


@pytest.mark.parametrize("dtype", [BF16, F16])
@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_integer_operands_with_bias_and_residual_are_exact(M, K, N, w_is_nk, dtype):
    import paper_2511_16964_b200 as P
    c = _int_case(M, K, N, seed=M + K + N)
    w = np.ascontiguousarray(c["w"].T) if w_is_nk else c["w"]
    out = Guarded((M, N), F32, pitch=N + 12)                   # padded rows: stores must also respect the pitch
    P.pike_linear_epilogue(dev(c["x"], dtype), dev(w, dtype), dev(c["b"], dtype), dev(c["r"], dtype), scale=0.5,
                           out_dtype=F32, w_is_nk=w_is_nk, out=out.t)
    _status_ok()
    out.check(f"{M}x{K}x{N}")
    want = O.linear_epilogue(c["x"], c["w"], c["b"], c["r"], scale=0.5)
    assert np.array_equal(host64(out.t), want), f"{M}x{K}x{N} nk={w_is_nk} {dtype}"


@pytest.mark.parametrize("bias_dtype,res_dtype", [(F32, BF16), (BF16, F32), (F32, F32)])
def test_integer_operands_with_fp32_side_tensors_are_exact(bias_dtype, res_dtype):
    import paper_2511_16964_b200 as P
    M, K, N = 300, 192, 328
    c = _int_case(M, K, N, seed=7)
    out = Guarded((M, N), F32)
    P.pike_linear_epilogue(dev(c["x"], BF16), dev(c["w"], BF16), dev(c["b"], bias_dtype), dev(c["r"], res_dtype),
                           out_dtype=F32, out=out.t)
    _status_ok()
    out.check("fp32 side tensors")
    assert np.array_equal(host64(out.t), O.linear_epilogue(c["x"], c["w"], c["b"], c["r"]))


def test_integer_operands_16bit_output_is_exact_when_representable():
    import paper_2511_16964_b200 as P
    M, K, N = 700, 8, 520                                       # |sum| <= 8*3*3 + 8 + 16 = 96: exact in bf16
    c = _int_case(M, K, N, seed=8)
    for dtype in (BF16, F16):
        out = Guarded((M, N), dtype, pitch=N + 8)
        P.pike_linear_epilogue(dev(c["x"], dtype), dev(c["w"], dtype), dev(c["b"], dtype), dev(c["r"], dtype), out=out.t)
        _status_ok()
        out.check("16-bit out")
        assert np.array_equal(host64(out.t), O.linear_epilogue(c["x"], c["w"], c["b"], c["r"]))


@pytest.mark.parametrize("dtype", [BF16, F16])
@pytest.mark.parametrize("w_is_nk", [False, True])
def test_grouped_integer_operands_with_group_bias_are_exact(w_is_nk, dtype):
    """Groups of 0, 1, 255, 256, 257 and 700 rows (empty groups first, in the middle and last), [G,N] bias."""
    import paper_2511_16964_b200 as P
    sizes = [0, 257, 0, 1, 256, 700, 255, 0]
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    T, K, N, Gn = int(off[-1]), 72, 328, len(sizes)
    rng = np.random.default_rng(9)
    x, w = ints(rng, (T, K)), ints(rng, (Gn, K, N))
    b, r = ints(rng, (Gn, N), -8, 8), ints(rng, (T, N), -16, 16)
    wd = np.ascontiguousarray(w.transpose(0, 2, 1)) if w_is_nk else w
    out = Guarded((T, N), F32, pitch=N + 4)
    P.pike_grouped_linear_epilogue(dev(x, dtype), dev(wd, dtype), dev(b, dtype), dev(r, dtype),
                                   torch.from_numpy(off).cuda(), out_dtype=F32, w_is_nk=w_is_nk, out=out.t)
    _status_ok()
    out.check("grouped")
    assert np.array_equal(host64(out.t), O.grouped_linear_epilogue(x, w, b, r, off))


def test_grouped_many_small_groups_are_exact():
    """300 groups of 0..40 rows: far more groups than row tiles, most row-tile indices are empty."""
    import paper_2511_16964_b200 as P
    rng = np.random.default_rng(10)
    sizes = rng.integers(0, 41, 300)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    T, K, N, Gn = int(off[-1]), 64, 264, len(sizes)
    x, w, b = ints(rng, (T, K)), ints(rng, (Gn, K, N), -2, 2), ints(rng, (Gn, N), -8, 8)
    out = Guarded((T, N), F32)
    P.pike_grouped_linear_epilogue(dev(x, BF16), dev(w, BF16), dev(b, BF16), None, torch.from_numpy(off).cuda(),
                                   out_dtype=F32, out=out.t)
    _status_ok()
    out.check("many groups")
    assert np.array_equal(host64(out.t), O.grouped_linear_epilogue(x, w, b, None, off))


def test_grouped_more_groups_than_the_shared_memory_table_holds():
    """5000 groups of 0..4 rows: past 4096 groups the kernel finds a row tile's group by bisection over the offsets
    themselves (most row-tile indices are then empty and skipped)."""
    import paper_2511_16964_b200 as P
    rng = np.random.default_rng(18)
    sizes = rng.integers(0, 5, 5000)
    off = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
    T, K, N, Gn = int(off[-1]), 64, 64, len(sizes)
    x, w, b = ints(rng, (T, K)), ints(rng, (Gn, K, N), -2, 2), ints(rng, (Gn, N), -8, 8)
    out = Guarded((T, N), F32)
    P.pike_grouped_linear_epilogue(dev(x, BF16), dev(w, BF16), dev(b, BF16), None, torch.from_numpy(off).cuda(),
                                   out_dtype=F32, out=out.t)
    _status_ok()
    out.check("5000 groups")
    assert np.array_equal(host64(out.t), O.grouped_linear_epilogue(x, w, b, None, off))


@pytest.mark.parametrize("bad", ["past_the_end", "decreasing", "negative"])
def test_grouped_offsets_that_break_the_contract_touch_nothing_outside(bad):
    """The kernel reads the offsets from device memory the host cannot check: whatever is there, stores stay inside
    `out` (rows of well-formed groups still get their values)."""
    import paper_2511_16964_b200 as P
    T, K, N = 600, 64, 264
    rng = np.random.default_rng(11)
    x, w, b = ints(rng, (T, K)), ints(rng, (3, K, N)), ints(rng, (3, N), -8, 8)
    off = {"past_the_end": [0, 200, 400, T + 300], "decreasing": [0, 400, 200, T], "negative": [-50, 200, 400, T]}[bad]
    out = Guarded((T, N), F32, pitch=N + 4, fill=-1.0)
    P.pike_grouped_linear_epilogue(dev(x, BF16), dev(w, BF16), dev(b, BF16), None,
                                   torch.tensor(off, dtype=torch.int32, device="cuda"), out_dtype=F32, out=out.t)
    _status_ok()
    out.check(bad)
    got = host64(out.t)
    if bad == "past_the_end":          # groups 0 and 1 are well formed; group 2 is cut at T
        want = O.grouped_linear_epilogue(x, w, b, None, [0, 200, 400, T])
        assert np.array_equal(got, want)
    elif bad == "negative":            # group 0 starts at the clamped 0
        assert np.array_equal(got, O.grouped_linear_epilogue(x, w, b, None, [0, 200, 400, T]))


@pytest.mark.parametrize("act", ["none", "gelu_erf", "gelu_tanh", "silu"])
@pytest.mark.parametrize("M,K,N,w_is_nk", [(300, 192, 328, False), (2560, 64, 1928, True)])
def test_tight_bound_on_fp32_outputs_per_activation(act, M, K, N, w_is_nk):
    """With fp32 output the only differences left are accumulation order and the activation's approximation:
    2e-3 absolute is an order of magnitude above them and well below the bias (up to 1/64) times the
    activation's slope, so a dropped bias, scale or residual fails here."""
    import paper_2511_16964_b200 as P
    c = G.config2(M=M, K=K, N=N, seed=12)
    w = np.ascontiguousarray(c["w"].T) if w_is_nk else c["w"]
    out = Guarded((M, N), F32)
    P.pike_linear_epilogue(dev(c["x"], BF16), dev(w, BF16), dev(c["b"], BF16), dev(c["r"], BF16), act=act, scale=0.75,
                           out_dtype=F32, w_is_nk=w_is_nk, out=out.t)
    _status_ok()
    out.check(act)
    want = O.linear_epilogue(c["x"], c["w"], c["b"], c["r"], act=act, scale=0.75)
    assert np.abs(host64(out.t) - want).max() < 2e-3
    # the same oracle with the bias dropped is far outside that bound: the gate can see the bias
    no_bias = O.linear_epilogue(c["x"], c["w"], None, c["r"], act=act, scale=0.75)
    assert np.abs(no_bias - want).max() > 4e-3


@pytest.mark.parametrize("reduce", ["softmax", "layernorm"])
def test_split_row_reductions_stay_inside_output_and_workspace(reduce):
    import paper_2511_16964_b200 as P
    M, K, N = 300, 64, 1000
    c = G.config2(M=M, K=K, N=N, seed=13)
    x, w, b = dev(c["x"], BF16), dev(c["w"], BF16), dev(c["b"], BF16)
    need = P.pike_linear_epilogue_workspace(x, w, reduce=reduce, out_dtype=F32)
    assert need == ((M * 4 * 8 + 255) // 256) * 256             # 4 column tiles, one 8-byte pair per (row, tile)
    gws, ws = guarded_workspace(need)
    out = Guarded((M, N), F32, pitch=N + 8)
    P.pike_linear_epilogue(x, w, b, None, reduce=reduce, out_dtype=F32, out=out.t, workspace=ws)
    _status_ok()
    out.check(reduce)
    gws.check(reduce + " workspace")
    want = O.linear_epilogue(c["x"], c["w"], c["b"], None, reduce=reduce)
    if reduce == "softmax":
        assert (np.abs(host64(out.t) - want) <= 1e-3 * want + 1e-9).all()
    else:
        assert np.abs(host64(out.t) - want).max() < 2e-3


def test_mlp_block_stays_inside_output_and_workspace():
    import paper_2511_16964_b200 as P
    c = G.config3(M=333, D=136, F=1032, seed=14, affine=True)
    t = {k: dev(c[k], BF16) for k in ("x", "gamma", "beta", "w1", "b1", "w2", "b2")}
    gws, ws = guarded_workspace(P.pike_mlp_block_workspace(t["x"], t["w1"]))
    out = Guarded((333, 136), BF16)
    P.pike_mlp_block(t["x"], t["gamma"], t["beta"], t["w1"], t["b1"], t["w2"], t["b2"], eps=c["eps"], out=out.t,
                     workspace=ws)
    _status_ok()
    out.check("mlp out")
    gws.check("mlp workspace")
    check_bf16(host64(out.t), O.mlp_block(c["x"], c["gamma"], c["beta"], c["w1"], c["b1"], c["w2"], c["b2"],
                                          eps=c["eps"]), what="guarded mlp block")


@pytest.mark.parametrize("S,D,causal", [(300, 128, True), (129, 64, False), (1, 128, True)])
def test_attention_stays_inside_its_output(S, D, causal):
    import paper_2511_16964_b200 as P
    c = G.config5(B=2, H=3, S=S, D=D, seed=15)
    out = Guarded((2, 3, S, D), BF16)
    P.pike_attention_chain(dev(c["q"], BF16), dev(c["k"], BF16), dev(c["v"], BF16), scale=float(c["scale"]),
                           causal=causal, out=out.t)
    _status_ok()
    out.check("attention out")
    check_bf16(host64(out.t), O.attention(c["q"], c["k"], c["v"], scale=c["scale"], causal=causal),
               what="guarded attention")


def test_attention_block_stays_inside_output_and_workspace():
    import paper_2511_16964_b200 as P
    c = G.attention_block(B=2, S=200, E=256, seed=16)
    t = {k: dev(c[k], BF16) for k in ("x", "gamma", "beta", "w_qkv", "b_qkv", "w_o", "b_o")}
    gws, ws = guarded_workspace(P.pike_attention_block_workspace(t["x"], scale=float(c["scale"])))
    out = Guarded((2, 200, 256), BF16)
    P.pike_attention_block(t["x"], t["gamma"], t["beta"], t["w_qkv"], t["b_qkv"], t["w_o"], t["b_o"],
                           scale=float(c["scale"]), causal=True, eps=c["eps"], out=out.t, workspace=ws)
    _status_ok()
    out.check("block out")
    gws.check("block workspace")
    want = O.attention_block(c["x"], c["gamma"], c["beta"], c["w_qkv"], c["b_qkv"], c["w_o"], c["b_o"], num_heads=2,
                             scale=c["scale"], causal=True, eps=c["eps"])
    check_bf16(host64(out.t), want, what="guarded attention block")


def test_fp32_chain_stays_inside_its_output():
    import paper_2511_16964_b200 as P
    c = G.config1(M=37, K=100, N=200, seed=17)
    out = Guarded((37, 200), F32, pitch=203)                    # the fp32 path takes any row pitch
    P.pike_linear_epilogue(dev(c["x"], F32), dev(c["w"], F32), dev(c["b"], F32), None, dev(c["gamma"], F32),
                           dev(c["beta"], F32), act="gelu_erf", reduce="layernorm", eps=c["eps"], out=out.t)
    _status_ok()
    out.check("fp32 chain")
    want = O.linear_epilogue(c["x"], c["w"], c["b"], None, c["gamma"], c["beta"], act="gelu_erf", reduce="layernorm",
                             eps=c["eps"])
    assert np.abs(host64(out.t) - want).max() <= 1e-4


def test_a_workspace_that_overlaps_a_tensor_is_refused():
    import paper_2511_16964_b200 as P
    x = torch.zeros((64, 64), dtype=BF16, device="cuda")
    w = torch.zeros((64, 512), dtype=BF16, device="cuda")
    out = torch.empty((64, 512), dtype=F32, device="cuda")
    with pytest.raises(P.PikeError) as e:
        P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32, out=out, workspace=out.view(torch.uint8).view(-1))
    assert e.value.code == 7
