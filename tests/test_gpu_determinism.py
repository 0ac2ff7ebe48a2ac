"""Repeated calls on the same inputs give bit-identical outputs (no race between the warp roles, no
dependence on what ran before), over a shuffled mix of shapes and chains."""
import random

import pytest
import torch

import pike_inputs as G
from util import dev

pytestmark = pytest.mark.gpu
BF16 = torch.bfloat16


def test_outputs_are_bitwise_reproducible():
    import paper_2511_16964_b200 as P
    rng = random.Random(0)
    cases = []
    for n, (M, K, N) in enumerate([(1, 8, 8), (77, 64, 72), (300, 192, 328), (1000, 1024, 1000), (2560, 64, 2048)]):
        c = G.config2(M=M, K=K, N=N, seed=40 + n)
        x, w, b, r = (dev(c[k], BF16) for k in "xwbr")
        cases.append(lambda x=x, w=w, b=b, r=r: P.pike_linear_epilogue(x, w, b, r, act="silu", scale=0.5))
        cases.append(lambda x=x, w=w: P.pike_linear_epilogue(x, w, reduce="softmax", out_dtype=torch.float32))
        cases.append(lambda x=x, w=w: P.pike_linear_epilogue(x, w, reduce="layernorm"))
    for n, (B, H, S, D) in enumerate([(1, 1, 1, 128), (2, 3, 129, 64), (1, 3, 640, 128), (2, 1, 1500, 128)]):
        c = G.config5(B=B, H=H, S=S, D=D, seed=50 + n)
        q, k, v = (dev(c[name], BF16) for name in "qkv")
        cases.append(lambda q=q, k=k, v=v, D=D: P.pike_attention_chain(q, k, v, scale=D ** -0.5, causal=True))
    c3 = G.config3(M=333, D=136, F=1032, seed=60)
    x3, w1, w2 = (dev(c3[name], BF16) for name in ("x", "w1", "w2"))
    cases.append(lambda: P.pike_mlp_block(x3, None, None, w1, None, w2, None))

    ref = [c().clone() for c in cases]
    torch.cuda.synchronize()
    for it in range(20):
        order = list(range(len(cases)))
        rng.shuffle(order)
        outs = [(i, cases[i]()) for i in order]
        torch.cuda.synchronize()
        assert P.pike_get_last_device_status() == (0, 0)
        for i, o in outs:
            assert torch.equal(o, ref[i]), f"case {i} differs from its first run in repetition {it}"
