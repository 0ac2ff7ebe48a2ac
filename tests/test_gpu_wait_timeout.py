"""Failure detection without a GPU fault: a bounded in-kernel wait that runs out is reported as a
status, the kernel still runs to its end, and the library keeps working afterwards."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, dev, host64

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def test_a_wait_that_nothing_satisfies_times_out_and_is_reported():
    import paper_2511_16964_b200 as P
    c = G.config2(M=256, K=128, N=256, seed=31)
    x, w = dev(c["x"], BF16), dev(c["w"], BF16)
    assert P.pike_get_last_device_status() == (0, 0)
    P.pike_set_wait_limit_ns(2_000_000)              # 2 ms instead of 2 s
    try:
        P.pike_test_withhold_loads()                 # the next GEMM's producers issue no loads
        P.pike_linear_epilogue(x, w)                 # its MMA thread waits for data that never comes
        torch.cuda.synchronize()                     # ... and the kernel still terminates
        status, where = P.pike_get_last_device_status()
        assert status == 10                          # PIKE_ERR_TIMEOUT
        # GEMM kernel; whichever starved wait hits the limit first records itself: the MMA warp's
        # "operands landed" barrier (2) or the epilogue warps' "accumulator ready" barrier (4)
        assert where >> 16 == 1 and where & 0xFFFF in (2, 4)
        assert P.pike_get_last_device_status() == (0, 0)  # reading clears it
    finally:
        P.pike_set_wait_limit_ns(0)
    # the hook applied to one launch only, and the context is intact: the same call is now correct
    got = host64(P.pike_linear_epilogue(x, w))
    torch.cuda.synchronize()
    check_bf16(got, O.linear_epilogue(c["x"], c["w"]), what="GEMM after a reported timeout")
    assert P.pike_get_last_device_status() == (0, 0)


def test_the_fp32_chain_reports_bulk_copies_that_never_land():
    """The small-problem fp32 kernel stages aligned operands with bulk copies on one mbarrier; with the copies
    withheld its bounded wait runs out, the cluster still meets at its barriers and exits, and the next call is right."""
    import paper_2511_16964_b200 as P
    F32 = torch.float32
    c = G.config1()
    args = [dev(c[k], F32) for k in ("x", "w", "b")] + [None, dev(c["gamma"], F32), dev(c["beta"], F32)]
    kw = dict(act="gelu_erf", reduce="layernorm", eps=c["eps"])
    assert P.pike_get_last_device_status() == (0, 0)
    P.pike_set_wait_limit_ns(2_000_000)
    try:
        P.pike_test_withhold_loads()
        P.pike_linear_epilogue(*args, **kw)
        torch.cuda.synchronize()
        status, where = P.pike_get_last_device_status()
        assert status == 10                          # PIKE_ERR_TIMEOUT
        assert where >> 16 == 4 and where & 0xFFFF == 1          # fp32 chain, its one barrier
        assert P.pike_get_last_device_status() == (0, 0)
    finally:
        P.pike_set_wait_limit_ns(0)
    got = host64(P.pike_linear_epilogue(*args, **kw))
    torch.cuda.synchronize()
    want = O.linear_epilogue(c["x"], c["w"], c["b"], None, c["gamma"], c["beta"], **kw)
    assert np.abs(got - want).max() <= 1e-4
    assert P.pike_get_last_device_status() == (0, 0)
