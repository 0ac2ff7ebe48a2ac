"""GPU parity: the logits + softmax chain as ONE kernel (PIKE_FLAG_ONE_PASS) - a stripe's logits stay in tensor
memory across all CTA pairs, per-tile pairs go through the workspace, the CTAs wait for one another (bounded), every
probability is written once.  Same gates as the two-kernel form, plus guard bands and the failure-detection path."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import Guarded, check_bf16, dev, guarded_workspace, host64

pytestmark = pytest.mark.gpu
BF16, F16, F32 = torch.bfloat16, torch.float16, torch.float32


def _gates(got, want, what):
    check_bf16(got, want, what=what)                              # contractual (vacuous for tiny p)
    big = want >= 1e-7
    rel = np.abs(got - want)[big] / want[big]
    assert rel.max() <= 1e-3, f"{what}: max relative error {rel.max():.2e}"
    assert np.abs(got.sum(axis=1) - 1).max() <= 1e-5, f"{what}: row sums"
    assert (got.argmax(axis=1) == want.argmax(axis=1)).all(), f"{what}: argmax"


def _run(c, *, act="none", scale=1.0, bias=None, residual=None, w_is_nk=False, dtype=BF16, pitch_pad=0):
    import paper_2511_16964_b200 as P
    M, N = c["x"].shape[0], c["w"].shape[1]
    w = np.ascontiguousarray(c["w"].T) if w_is_nk else c["w"]
    x, wd = dev(c["x"], dtype), dev(w, dtype)
    need = P.pike_linear_epilogue_workspace(x, wd, reduce="softmax", out_dtype=F32, w_is_nk=w_is_nk, one_pass=True)
    gws, ws = guarded_workspace(need)
    out = Guarded((M, N), F32, pitch=N + pitch_pad)
    P.pike_linear_epilogue(x, wd, dev(bias, dtype), dev(residual, dtype), act=act, scale=scale, reduce="softmax",
                           out_dtype=F32, w_is_nk=w_is_nk, one_pass=True, out=out.t, workspace=ws)
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    out.check("one-pass out")
    gws.check("one-pass workspace")
    return host64(out.t)


@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("M,K,N", [(130, 64, 1000), (64, 128, 256), (5, 256, 8), (700, 192, 2312), (300, 72, 37888)])
def test_small_ragged_and_widest_shapes(M, K, N, w_is_nk):
    # 1 to 148 column tiles (37888 = 148 x 256 is the widest row the chip's tensor memory holds), 1 to 3 stripes
    c = G.config4(M=M, K=K, N=N, seed=71)
    got = _run(c, w_is_nk=w_is_nk, pitch_pad=8)
    _gates(got, O.linear_epilogue(c["x"], c["w"], reduce="softmax"), f"one-pass {M}x{K}x{N} nk={w_is_nk}")


@pytest.mark.parametrize("dtype", [BF16, F16])
def test_with_bias_activation_scale_and_residual(dtype):
    c = G.config2(M=300, K=192, N=1000, seed=72, dtype="f16" if dtype == F16 else "bf16")
    got = _run(c, act="silu", scale=0.5, bias=c["b"], residual=c["r"], dtype=dtype)
    want = O.linear_epilogue(c["x"], c["w"], c["b"], c["r"], act="silu", scale=0.5, reduce="softmax")
    _gates(got, want, "one-pass with epilogue")


def test_extreme_logits():
    c = G.config4(M=64, K=128, N=1000, seed=73)
    got = _run(c, scale=400.0)
    want = O.linear_epilogue(c["x"], c["w"], scale=400.0, reduce="softmax")
    assert np.isfinite(got).all() and np.abs(got - want).max() <= 2e-3
    assert np.abs(got.sum(axis=1) - 1).max() <= 1e-5 and (got.argmax(axis=1) == want.argmax(axis=1)).all()


def test_agrees_with_the_two_kernel_form_and_is_reproducible():
    import paper_2511_16964_b200 as P
    c = G.config4(M=520, K=256, N=3000, seed=74)
    x, w = dev(c["x"], BF16), dev(c["w"], BF16)
    a = P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32, one_pass=True)
    b = P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32, one_pass=True)
    two = P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32)
    torch.cuda.synchronize()
    assert torch.equal(a, b)                                              # bit-reproducible
    assert (a - two).abs().max().item() <= 1e-3 * two.max().item()       # same values up to the exponential's rounding


def test_config4_full_size_one_row_per_cta_block():
    c = G.config4()
    rows = np.unique(np.concatenate([[b * 128 + (37 * b + 5) % 128 for b in range(16)], [0, 127, 128, 2047]]))
    got = _run(c)[rows]
    _gates(got, O.linear_epilogue(c["x"], c["w"], reduce="softmax", rows=rows), "one-pass config 4")


def test_rows_wider_than_the_chip_are_refused():
    import paper_2511_16964_b200 as P
    x = torch.zeros((8, 64), dtype=BF16, device="cuda")
    w = torch.zeros((64, 37888 + 256), dtype=BF16, device="cuda")
    with pytest.raises(P.PikeError) as e:
        P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32, one_pass=True)
    assert e.value.code == 6                 # PIKE_ERR_UNSUPPORTED: 149 column tiles do not fit 148 accumulators
    with pytest.raises(P.PikeError) as e:    # the flag belongs to the softmax reduction only
        P.pike_linear_epilogue(x, torch.zeros((64, 64), dtype=BF16, device="cuda"), one_pass=True)
    assert e.value.code == 6


def test_a_cta_that_never_counts_itself_in_is_reported_not_waited_for_forever():
    """Failure detection without a GPU fault: block 0 withholds its arrival on the stripe counters, its peers' bounded
    waits run out after 2 ms, the kernel still ends, the status word says where, and the next call is correct."""
    import paper_2511_16964_b200 as P
    c = G.config4(M=600, K=128, N=1000, seed=75)
    x, w = dev(c["x"], BF16), dev(c["w"], BF16)
    assert P.pike_get_last_device_status() == (0, 0)
    P.pike_set_wait_limit_ns(2_000_000)
    try:
        P.pike_test_withhold_partials()
        P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32, one_pass=True)
        torch.cuda.synchronize()                         # ... and the kernel still terminates
        status, where = P.pike_get_last_device_status()
        assert status == 10                              # PIKE_ERR_TIMEOUT
        assert where >> 16 == 1 and where & 0xFFFF == 5  # GEMM family, the stripe wait
        assert P.pike_get_last_device_status() == (0, 0)
    finally:
        P.pike_set_wait_limit_ns(0)
    got = host64(P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32, one_pass=True))
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    _gates(got, O.linear_epilogue(c["x"], c["w"], reduce="softmax"), "one-pass after a reported timeout")
