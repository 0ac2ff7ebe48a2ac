"""The workspace-free softmax chain, for hosts of the library that cannot allocate.

Some callers (a server whose pool owns the whole device heap, a plugin inside another
framework's step, a thread that must not enter cudaMalloc) cannot give
pike_linear_epilogue the workspace it asks for.  pike_linear_softmax_noalloc keeps its
scratch in an array inside the library.  This test calls it through the C ABI twice in
a row (the array is shared and keeps the first call's contents, so the second call
proves nothing stale leaks through) and compares each result with the CPU oracle under
the softmax gates of the other parity tests; the regular entry point on the same
inputs is compared as an extra.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import dev, host64

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def _compare(got, want, what):
    got = host64(got)
    want = want if isinstance(want, np.ndarray) else host64(want)
    assert np.isfinite(got).all()
    assert (np.abs(got - want) <= 2e-2 + 2e-2 * np.abs(want)).all(), what      # the bf16 bar of the other tests
    big = want >= 1e-7
    assert (np.abs(got - want)[big] / want[big]).max() <= 1e-3, what            # and the softmax gates
    assert np.abs(got.sum(axis=1) - 1).max() <= 1e-5, what
    assert (got.argmax(axis=1) == want.argmax(axis=1)).all(), what


def test_two_calls_in_a_row_match_the_workspace_entry_point():
    import paper_2511_16964_b200 as P
    # first call: several column tiles, ragged edges, bias and an activation
    a = G.config2(M=300, K=192, N=1000, seed=21)
    xa, wa, ba = dev(a["x"], BF16), dev(a["w"], BF16), dev(a["b"], BF16)
    out_a = torch.empty((300, 1000), dtype=F32, device="cuda")
    P.pike_linear_softmax_noalloc(xa, wa, ba, out=out_a, act="silu", scale=0.5)
    # second call straight after it: other shape, [N,K] weights, no bias; the scratch still
    # holds the first call's partials
    b = G.config4(M=130, K=256, N=2048, seed=22)
    xb, wb = dev(b["x"], BF16), dev(np.ascontiguousarray(b["w"].T), BF16)
    out_b = torch.empty((130, 2048), dtype=F32, device="cuda")
    P.pike_linear_softmax_noalloc(xb, wb, out=out_b, w_is_nk=True)
    torch.cuda.synchronize()
    st, where = P.pike_get_last_device_status()
    assert st == 0, f"device status {st} at {where:#x}"

    # the expected values come from the CPU oracle ...
    _compare(out_a, O.linear_epilogue(a["x"], a["w"], a["b"], act="silu", scale=0.5, reduce="softmax"), "first call")
    _compare(out_b, O.linear_epilogue(b["x"], b["w"], reduce="softmax"), "second call")
    # ... and, as an extra, the entry point that takes a workspace gives the same values
    same_a = P.pike_linear_epilogue(xa, wa, ba, act="silu", scale=0.5, reduce="softmax", out_dtype=F32)
    same_b = P.pike_linear_epilogue(xb, wb, reduce="softmax", out_dtype=F32, w_is_nk=True)
    torch.cuda.synchronize()
    _compare(out_a, same_a, "first call vs workspace entry point")
    _compare(out_b, same_b, "second call vs workspace entry point")
    # and the first problem again, now after the second one overwrote the scratch
    out_a2 = torch.empty_like(out_a)
    P.pike_linear_softmax_noalloc(xa, wa, ba, out=out_a2, act="silu", scale=0.5)
    torch.cuda.synchronize()
    assert torch.equal(out_a2, out_a)


def test_a_non_finite_scale_is_refused_like_everywhere_else():
    import paper_2511_16964_b200 as P
    x = torch.zeros((16, 64), dtype=BF16, device="cuda")
    w = torch.zeros((64, 64), dtype=BF16, device="cuda")
    out = torch.empty((16, 64), dtype=F32, device="cuda")
    for bad in (float("inf"), float("-inf"), float("nan")):
        with pytest.raises(P.PikeError) as e:
            P.pike_linear_softmax_noalloc(x, w, out=out, scale=bad)
        assert e.value.code == 6            # PIKE_ERR_UNSUPPORTED, as pike_linear_epilogue answers


def test_problems_larger_than_the_built_in_scratch_are_refused():
    import paper_2511_16964_b200 as P
    M, N = 2048, 33024                      # 2048 * 129 tiles = 264192 pairs > 262144
    x = torch.zeros((M, 8), dtype=BF16, device="cuda")
    w = torch.zeros((8, N), dtype=BF16, device="cuda")
    out = torch.empty((M, N), dtype=F32, device="cuda")
    with pytest.raises(P.PikeError) as e:
        P.pike_linear_softmax_noalloc(x, w, out=out)
    assert e.value.code == 7                # PIKE_ERR_WORKSPACE: the built-in scratch is too small
    # exactly at the limit is accepted (2048 * 128 tiles)
    w2 = torch.zeros((8, 32768), dtype=BF16, device="cuda")
    out2 = torch.empty((M, 32768), dtype=F32, device="cuda")
    P.pike_linear_softmax_noalloc(x, w2, out=out2)
    torch.cuda.synchronize()
    assert abs(float(out2[0].sum()) - 1.0) < 1e-5
