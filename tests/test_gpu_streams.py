"""Every chain enqueues on the caller's stream: inputs produced on a side stream (after a deliberately long
kernel) are consumed correctly without any device-wide synchronisation in between, and two chains issued to two
streams do not disturb each other."""
import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, check_f32, dev, host64

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def _busy(stream, n=1 << 26):
    """Something long-running on `stream`, so that work queued after it really waits for stream order."""
    with torch.cuda.stream(stream):
        a = torch.ones(n, device="cuda")
        for _ in range(8):
            a = a * 1.0001
    return a


def test_chains_follow_the_order_of_a_side_stream():
    import paper_2511_16964_b200 as P
    side = torch.cuda.Stream()
    c2 = G.config2(M=300, K=192, N=328, seed=31)
    c5 = G.config5(B=1, H=2, S=300, seed=32)
    c1 = G.config1(M=40, K=64, N=72, seed=33)
    # host tensors first; the device copies are made ON the side stream, behind the busy kernel
    hx, hw, hb, hr = (torch.from_numpy(np.ascontiguousarray(c2[k], np.float32)).to(BF16).pin_memory() for k in "xwbr")
    hq, hk, hv = (torch.from_numpy(np.ascontiguousarray(c5[k], np.float32)).to(BF16).pin_memory() for k in "qkv")
    h1 = {k: torch.from_numpy(np.ascontiguousarray(c1[k], np.float32)).pin_memory() for k in ("x", "w", "b", "gamma", "beta")}
    keep = _busy(side)
    with torch.cuda.stream(side):
        x, w, b, r = (t.to("cuda", non_blocking=True) for t in (hx, hw, hb, hr))
        q, k, v = (t.to("cuda", non_blocking=True) for t in (hq, hk, hv))
        d1 = {n: t.to("cuda", non_blocking=True) for n, t in h1.items()}
        got2 = P.pike_linear_epilogue(x, w, b, r, act="silu", scale=0.5, stream=side)
        got4 = P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=F32, stream=side)
        got5 = P.pike_attention_chain(q, k, v, scale=float(c5["scale"]), causal=True, stream=side)
        got1 = P.pike_linear_epilogue(d1["x"], d1["w"], d1["b"], None, d1["gamma"], d1["beta"], act="gelu_erf",
                                      reduce="layernorm", eps=c1["eps"], stream=side)
    side.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    check_bf16(host64(got2), O.linear_epilogue(c2["x"], c2["w"], c2["b"], c2["r"], act="silu", scale=0.5), what="side stream GEMM")
    want4 = O.linear_epilogue(c2["x"], c2["w"], reduce="softmax")
    assert np.abs(host64(got4) - want4).max() <= 1e-3 * want4.max() and np.abs(host64(got4).sum(1) - 1).max() <= 1e-5
    check_bf16(host64(got5), O.attention(c5["q"], c5["k"], c5["v"], scale=c5["scale"], causal=True), what="side stream attention")
    check_f32(host64(got1), O.linear_epilogue(c1["x"], c1["w"], c1["b"], None, c1["gamma"], c1["beta"], act="gelu_erf",
                                              reduce="layernorm", eps=c1["eps"]), what="side stream fp32 chain")
    del keep


def test_two_streams_at_once():
    import paper_2511_16964_b200 as P
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    c3 = G.config3(M=333, D=136, F=1032, seed=34, affine=True)
    c5 = G.config5(B=2, H=3, S=257, seed=35)
    t3 = {k: dev(c3[k], BF16) for k in ("x", "gamma", "beta", "w1", "b1", "w2", "b2")}
    q, k, v = (dev(c5[n], BF16) for n in "qkv")
    torch.cuda.synchronize()
    outs3, outs5 = [], []
    for _ in range(3):      # interleaved submissions; each stream has its own workspace and outputs
        with torch.cuda.stream(s1):
            outs3.append(P.pike_mlp_block(t3["x"], t3["gamma"], t3["beta"], t3["w1"], t3["b1"], t3["w2"], t3["b2"],
                                          act="gelu_tanh", eps=c3["eps"], stream=s1))
        with torch.cuda.stream(s2):
            outs5.append(P.pike_attention_chain(q, k, v, scale=float(c5["scale"]), causal=False, stream=s2))
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    want3 = O.mlp_block(c3["x"], c3["gamma"], c3["beta"], c3["w1"], c3["b1"], c3["w2"], c3["b2"], eps=c3["eps"])
    want5 = O.attention(c5["q"], c5["k"], c5["v"], scale=c5["scale"], causal=False)
    for o in outs3:
        check_bf16(host64(o), want3, what="mlp block on stream 1")
    for o in outs5:
        check_bf16(host64(o), want5, what="attention on stream 2")


def test_temporaries_belong_to_the_stream_the_kernels_run_on():
    """The wrappers allocate missing outputs and workspaces for the stream given as `stream=`, even when another
    stream is current: a block freed when the wrapper returns must not be handed to the current stream's next
    allocation while the side stream's kernels still use it.  Here the default stream is current, the kernels are
    queued on a busy side stream with workspace=None, and the default stream at once allocates and overwrites
    tensors of the very sizes the temporaries had."""
    import paper_2511_16964_b200 as P
    side = torch.cuda.Stream()
    c4 = G.config4(M=300, K=192, N=1000, seed=36)
    c3 = G.config3(M=333, D=136, F=1032, seed=37, affine=True)
    x4, w4 = dev(c4["x"], BF16), dev(c4["w"], BF16)
    t3 = {k: dev(c3[k], BF16) for k in ("x", "gamma", "beta", "w1", "b1", "w2", "b2")}
    need4 = P.pike_linear_epilogue_workspace(x4, w4, reduce="softmax", out_dtype=F32)
    need3 = P.pike_mlp_block_workspace(t3["x"], t3["w1"])
    torch.cuda.synchronize()
    keep = _busy(side)                                       # the side stream's kernels will start late
    got4 = P.pike_linear_epilogue(x4, w4, reduce="softmax", out_dtype=F32, stream=side)
    got3 = P.pike_mlp_block(t3["x"], t3["gamma"], t3["beta"], t3["w1"], t3["b1"], t3["w2"], t3["b2"], eps=c3["eps"],
                            stream=side)
    junk = []
    for _ in range(4):                                       # current (default) stream: same sizes, overwritten at once
        junk.append(torch.full((max(need4, 256),), 0x7F, dtype=torch.uint8, device="cuda"))
        junk.append(torch.full((max(need3, 256),), 0x7F, dtype=torch.uint8, device="cuda"))
    side.synchronize()
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    want4 = O.linear_epilogue(c4["x"], c4["w"], reduce="softmax")
    g4 = host64(got4)
    assert (np.abs(g4 - want4) <= 1e-3 * want4 + 1e-9).all() and np.abs(g4.sum(1) - 1).max() <= 1e-5
    check_bf16(host64(got3), O.mlp_block(c3["x"], c3["gamma"], c3["beta"], c3["w1"], c3["b1"], c3["w2"], c3["b2"],
                                         eps=c3["eps"]), what="mlp block with a temporary workspace on a side stream")
    del keep, junk


def test_chains_replay_from_a_cuda_graph():
    """With caller-owned outputs and workspaces a chain call allocates nothing and synchronises nothing, so a
    sequence of calls can be captured into a CUDA graph once and replayed: every replay on new input CONTENTS (same
    buffers) gives bit for bit what the same calls give when issued directly."""
    import paper_2511_16964_b200 as P
    c3 = G.config3(M=300, D=136, F=520, seed=41, affine=True)
    c5 = G.config5(B=1, H=2, S=300, seed=42)
    c1 = G.config1(M=40, K=64, N=72, seed=43)
    x3, g3, be3, w1, b1, w2, b2 = (dev(c3[k], BF16) for k in ("x", "gamma", "beta", "w1", "b1", "w2", "b2"))
    q, k, v = (dev(c5[n], BF16) for n in "qkv")
    d1 = {n: dev(c1[n], F32) for n in ("x", "w", "b", "gamma", "beta")}
    wl = dev(c3["w1"], BF16)                                            # logits weights for the softmax chain
    out3, out5 = torch.empty_like(x3), torch.empty_like(q)
    out1 = torch.empty((40, 72), device="cuda", dtype=F32)
    out4 = torch.empty((300, 520), device="cuda", dtype=F32)
    ws3 = torch.empty(P.pike_mlp_block_workspace(x3, w1), dtype=torch.uint8, device="cuda")
    ws4 = torch.empty(P.pike_linear_epilogue_workspace(x3, wl, reduce="softmax", out_dtype=F32), dtype=torch.uint8,
                      device="cuda")

    def calls(stream=None):
        P.pike_linear_epilogue(d1["x"], d1["w"], d1["b"], None, d1["gamma"], d1["beta"], act="gelu_erf",
                               reduce="layernorm", eps=c1["eps"], out=out1, stream=stream)
        P.pike_mlp_block(x3, g3, be3, w1, b1, w2, b2, act="gelu_tanh", eps=c3["eps"], out=out3, workspace=ws3,
                         stream=stream)
        P.pike_linear_epilogue(out3, wl, reduce="softmax", out_dtype=F32, out=out4, workspace=ws4, stream=stream)
        P.pike_attention_chain(q, k, v, scale=float(c5["scale"]), causal=True, out=out5, stream=stream)

    calls()                                  # warm: tensor maps encoded, the library's lazy state settled
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        calls()
    for rep in range(3):
        x3.copy_(dev(G.config3(M=300, D=136, F=520, seed=50 + rep, affine=True)["x"], BF16))
        q.copy_(dev(G.config5(B=1, H=2, S=300, seed=60 + rep)["q"], BF16))
        d1["x"].copy_(dev(G.config1(M=40, K=64, N=72, seed=70 + rep)["x"], F32))
        for o in (out1, out3, out4, out5):
            o.zero_()
        graph.replay()
        torch.cuda.synchronize()
        got = [o.clone() for o in (out1, out3, out4, out5)]
        for o in (out1, out3, out4, out5):
            o.zero_()
        calls()
        torch.cuda.synchronize()
        for a, b in zip(got, (out1, out3, out4, out5)):
            assert torch.equal(a.view(torch.int32) if a.dtype == F32 else a.view(torch.int16),
                               b.view(torch.int32) if b.dtype == F32 else b.view(torch.int16))
    assert P.pike_get_last_device_status() == (0, 0)
    # and the replayed MLP block is the right answer, not merely a reproducible one
    c3r = G.config3(M=300, D=136, F=520, seed=52, affine=True)
    want = O.mlp_block(c3r["x"], c3["gamma"], c3["beta"], c3["w1"], c3["b1"], c3["w2"], c3["b2"], act="gelu_tanh", eps=c3["eps"])
    check_bf16(host64(out3), want, what="graph replay MLP block")
