"""GPU parity: logits + softmax with the columns split into slices, as several GPUs would hold them.
One GPU runs the slices one after the other (the slices never wait on one another: the exchange between
the two library calls is a host-ordered gather), then every slice is finished with all slices' row pairs.
Bars: the softmax gates of the unsharded chain (relative error <= 1e-3 on p >= 1e-7, row sums, arg-max)."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import dev, host64

pytestmark = pytest.mark.gpu
BF16, F16, F32 = torch.bfloat16, torch.float16, torch.float32


def _gates(got, want, what):
    assert np.isfinite(got).all(), what
    assert (np.abs(got - want) <= 2e-2 + 2e-2 * np.abs(want)).all(), what      # contractual (vacuous for tiny p)
    big = want >= 1e-7
    rel = np.abs(got - want)[big] / want[big]
    assert rel.max() <= 1e-3, f"{what}: max relative error {rel.max():.2e}"
    assert np.abs(got.sum(axis=1) - 1).max() <= 1e-5, f"{what}: row sums"
    assert (got.argmax(axis=1) == want.argmax(axis=1)).all(), f"{what}: argmax"


def _sharded(c, cuts, *, bias=None, act="none", scale=1.0, w_is_nk=False, dt=BF16, check_stats=True):
    import paper_2511_16964_b200 as P
    x = dev(c["x"], dt)
    outs, stats = [], []
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        w = c["w"][:, lo:hi]
        w = np.ascontiguousarray(w.T) if w_is_nk else np.ascontiguousarray(w)
        b = None if bias is None else dev(bias[lo:hi], dt)
        o, s = P.pike_linear_softmax_shard_local(x, dev(w, dt), b, act=act, scale=scale, w_is_nk=w_is_nk)
        if check_stats:
            _, want_s = O.softmax_shard_stats(c["x"], c["w"][:, lo:hi], None if bias is None else bias[lo:hi],
                                              act=act, scale=scale)
            got_s = host64(s)
            assert np.abs(got_s[:, 0] - want_s[:, 0]).max() <= 2e-3 * max(1.0, np.abs(want_s[:, 0]).max())
            # the sum is relative to the slice's own maximum: compare l*exp(m) through logs
            assert np.abs((np.log(got_s[:, 1]) + got_s[:, 0]) - (np.log(want_s[:, 1]) + want_s[:, 0])).max() <= 2e-3
        outs.append(o)
        stats.append(s)
    all_stats = torch.stack(stats).contiguous()
    for o in outs:
        P.pike_linear_softmax_shard_finish(o, all_stats)
    torch.cuda.synchronize()
    st, where = P.pike_get_last_device_status()
    assert st == 0, f"device status {st} at {where:#x}"
    return np.concatenate([host64(o) for o in outs], axis=1)


@pytest.mark.parametrize("w_is_nk", [False, True])
@pytest.mark.parametrize("M,K,N,cuts", [(130, 64, 1000, [0, 504, 1000]), (130, 64, 1000, [0, 8, 264, 1000]),
                                        (5, 256, 16, [0, 8, 16]), (300, 128, 2048, [0, 512, 1024, 1536, 2048]),
                                        (64, 128, 256, [0, 256])])
def test_slices_combine_to_the_full_softmax(M, K, N, cuts, w_is_nk):
    c = G.config4(M=M, K=K, N=N, seed=8)
    got = _sharded(c, cuts, w_is_nk=w_is_nk)
    _gates(got, O.linear_epilogue(c["x"], c["w"], reduce="softmax"), f"sharded softmax {M}x{K}x{N} {cuts}")


def test_bias_activation_and_scale_before_the_softmax():
    c = G.config4(M=77, K=128, N=520, seed=9)
    b = G.uniform((520,), 0.5, seed=9, tensor_id=78, dtype="bf16")
    got = _sharded(c, [0, 264, 520], bias=b, act="gelu_tanh", scale=4.0)
    _gates(got, O.linear_epilogue(c["x"], c["w"], b, act="gelu_tanh", scale=4.0, reduce="softmax"), "bias+act+scale")


def test_maximum_in_another_slice():
    """One column dominates every row; the slices that do not hold it must scale by exp(m_r - m)."""
    c = G.config4(M=40, K=64, N=512, seed=10)
    w = c["w"].copy()
    w[:, 300] = 0.25 * np.sign(c["x"][7])            # a large logit in column 300 for row 7
    c = dict(x=c["x"], w=w)
    got = _sharded(c, [0, 256, 512])
    want = O.linear_epilogue(c["x"], c["w"], reduce="softmax")
    assert want[7, 300] > 0.99
    _gates(got, want, "dominant column")


def test_ieee_half_slices():
    c = G.config4(M=130, K=64, N=1000, seed=11, dtype="f16")
    got = _sharded(c, [0, 504, 1000], dt=F16)
    _gates(got, O.linear_epilogue(c["x"], c["w"], reduce="softmax"), "f16 sharded softmax")


def test_helper_without_a_process_group_is_the_single_gpu_chain():
    import paper_2511_16964_b200 as P
    c = G.config4(M=130, K=64, N=1000, seed=12)
    got = host64(P.linear_softmax_vocab_sharded(dev(c["x"], BF16), dev(c["w"], BF16)))
    _gates(got, O.linear_epilogue(c["x"], c["w"], reduce="softmax"), "one shard")


def test_config4_full_size_two_slices_sampled_rows():
    c = G.config4()
    rows = np.array([0, 1, 127, 128, 777, 1024, 2046, 2047])
    got = _sharded(c, [0, 16000, 32000], check_stats=False)[rows]
    _gates(got, O.linear_epilogue(c["x"], c["w"], reduce="softmax", rows=rows), "config 4 over two slices")


def test_rejections():
    import paper_2511_16964_b200 as P
    from paper_2511_16964_b200 import binding as B
    c = G.config4(M=16, K=64, N=64, seed=1)
    x, w = dev(c["x"], BF16), dev(c["w"], BF16)
    out, stats = P.pike_linear_softmax_shard_local(x, w)
    with pytest.raises(TypeError):
        P.pike_linear_softmax_shard_finish(out, torch.zeros((1, 15, 2), device="cuda"))       # wrong row count
    with pytest.raises(P.PikeError) as e:                                                       # fp32 inputs
        P.pike_linear_softmax_shard_local(x.float(), w.float())
    assert e.value.code == 3
    with pytest.raises(P.PikeError) as e:                                                       # 16-bit output slice
        P.pike_linear_softmax_shard_finish(out.to(BF16), torch.stack([stats]))
    assert e.value.code == 3
    with pytest.raises(P.PikeError) as e:                                                       # workspace too small
        P.pike_linear_softmax_shard_local(x, w, workspace=torch.empty(0, dtype=torch.uint8, device="cuda"))
    assert e.value.code == 7
    torch.cuda.synchronize()
