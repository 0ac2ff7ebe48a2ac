"""Two handles used from two host threads at once, through the raw C ABI (the header promises: one handle
per host thread, no state shared between handles)."""
import ctypes
import threading

import numpy as np
import pytest
import torch

import pike_inputs as G
from oracle import pike_oracle as O
from util import check_bf16, check_f32, dev, host64

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def test_two_handles_on_two_threads():
    from paper_2511_16964_b200 import binding as B
    lib = B.load_library()
    c2 = G.config2(M=600, K=256, N=520, seed=61)
    c1 = G.config1(M=40, K=64, N=72, seed=62)
    c5 = G.config5(B=1, H=2, S=300, seed=63)
    x2, w2, b2, r2 = (dev(c2[k], BF16) for k in "xwbr")
    x1, w1, b1 = (dev(c1[k], F32) for k in ("x", "w", "b"))
    q, k, v = (dev(c5[n], BF16) for n in "qkv")
    torch.cuda.synchronize()
    results, errors = {}, []

    def worker(tid):
        try:
            h = ctypes.c_void_p()
            assert lib.pike_create(ctypes.byref(h), 0) == 0
            stream = torch.cuda.Stream()
            sp = ctypes.c_void_p(stream.cuda_stream)
            outs = []
            for rep in range(10):                      # both threads hammer the same kernels on their own handles
                o2 = torch.empty((600, 520), dtype=BF16, device="cuda")
                o1 = torch.empty((40, 72), dtype=F32, device="cuda")
                o5 = torch.empty_like(q)
                e2 = B._epilogue("silu", 0.5, "none", 0.0, BF16, 0)
                e1 = B._epilogue("gelu_erf", 1.0, "layernorm", 1e-5, F32, 0)
                e5 = B._epilogue("none", float(c5["scale"]), "none", 0.0, BF16, B.FLAG_CAUSAL)
                rc = lib.pike_linear_epilogue(h, B._tensor(x2), B._tensor(w2), B._tensor(b2), B._tensor(r2), None, None,
                                              e2, B._tensor(o2), None, 0, sp)
                rc |= lib.pike_linear_epilogue(h, B._tensor(x1), B._tensor(w1), B._tensor(b1), None, None, None,
                                               e1, B._tensor(o1), None, 0, sp)
                rc |= lib.pike_attention_chain(h, B._tensor(q), B._tensor(k), B._tensor(v), e5,
                                               B._tensor(o5), None, 0, sp)
                assert rc == 0
                outs.append((o2, o1, o5))
            stream.synchronize()
            st, where = ctypes.c_int(0), ctypes.c_uint32(0)
            assert lib.pike_get_last_device_status(h, ctypes.byref(st), ctypes.byref(where)) == 0 and st.value == 0
            assert lib.pike_destroy(h) == 0
            results[tid] = outs
        except BaseException as exc:                   # surfaced in the main thread
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    want2 = O.linear_epilogue(c2["x"], c2["w"], c2["b"], c2["r"], act="silu", scale=0.5)
    want1 = O.linear_epilogue(c1["x"], c1["w"], c1["b"], act="gelu_erf", reduce="layernorm")
    want5 = O.attention(c5["q"], c5["k"], c5["v"], scale=c5["scale"], causal=True)
    for tid in (0, 1):
        for o2, o1, o5 in results[tid]:
            check_bf16(host64(o2), want2, what=f"thread {tid} GEMM")
            check_f32(host64(o1), want1, what=f"thread {tid} fp32 chain")
            check_bf16(host64(o5), want5, what=f"thread {tid} attention")


def test_more_distinct_buffers_than_the_tensor_map_cache_holds():
    """The handle keeps the 48 most recently used tensor maps; calls on 70 different activation buffers (and then on
    the first ones again, whose maps have been evicted meanwhile) must all come out right."""
    import paper_2511_16964_b200 as P
    c = G.config2(M=130, K=64, N=264, seed=64)
    w, b = dev(c["w"], BF16), dev(c["b"], BF16)
    want = O.linear_epilogue(c["x"], c["w"], c["b"], act="gelu_tanh")
    xs = [dev(c["x"], BF16).clone() for _ in range(70)]
    outs = [P.pike_linear_epilogue(x, w, b, act="gelu_tanh") for x in xs]
    outs += [P.pike_linear_epilogue(x, w, b, act="gelu_tanh") for x in xs[:5]]
    torch.cuda.synchronize()
    assert P.pike_get_last_device_status() == (0, 0)
    for o in outs:
        check_bf16(host64(o), want, what="tensor-map cache")


def test_kernel_selection_log_goes_to_stderr_when_asked_for():
    """PIKE_LOG=1 at handle creation: one stderr line per kernel selection; nothing without it."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import torch, paper_2511_16964_b200 as P\n"
            "x = torch.zeros((64, 64), device='cuda', dtype=torch.bfloat16); w = torch.zeros((64, 256), device='cuda', dtype=torch.bfloat16)\n"
            "P.pike_linear_epilogue(x, w, reduce='softmax', out_dtype=torch.float32); torch.cuda.synchronize()\n")
    for flag, expect in (("1", True), ("0", False)):
        res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, cwd=root,
                             env=dict(os.environ, PIKE_LOG=flag), timeout=300)
        assert res.returncode == 0, res.stderr[-1000:]
        lines = [l for l in res.stderr.splitlines() if l.startswith("[pike] ")]
        assert (len(lines) == 2) == expect, res.stderr[-1000:]
        if expect:
            assert "gemm_bf16_kernel M=64 K=64 N=256" in lines[0] and "softmax_finish_kernel" in lines[1]


def test_results_do_not_depend_on_programmatic_dependent_launch():
    """PIKE_PDL=0 at handle creation takes the launch attribute off: the chains' results are bit-identical with it
    on (the default) and off, over back-to-back calls that reuse one output and one workspace."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import torch, hashlib, paper_2511_16964_b200 as P\n"
            "g = torch.Generator(device='cuda').manual_seed(5)\n"
            "r = lambda *s: (torch.randn(*s, device='cuda', generator=g) * 0.5).to(torch.bfloat16)\n"
            "x, gm, bt, w1, b1, w2, b2 = r(640, 512), r(512), r(512), r(512, 1024) * 0.1, r(1024), r(1024, 512) * 0.1, r(512)\n"
            "ws = torch.empty(P.pike_mlp_block_workspace(x, w1), dtype=torch.uint8, device='cuda'); out = torch.empty_like(x)\n"
            "wl = r(512, 3000) * 0.1\n"
            "h = hashlib.sha256()\n"
            "for i in range(20):\n"
            "    P.pike_mlp_block(x, gm, bt, w1, b1, w2, b2, out=out, workspace=ws)\n"
            "    p = P.pike_linear_epilogue(out, wl, reduce='softmax', out_dtype=torch.float32)\n"
            "    x = out.clone()\n"
            "    h.update(p.cpu().numpy().tobytes()); h.update(out.view(torch.int16).cpu().numpy().tobytes())\n"
            "print('DIGEST', h.hexdigest())\n")
    digests = []
    for flag in ("1", "0"):
        res = subprocess.run([sys.executable, "-c", code], capture_output=True, text=True, cwd=root,
                             env=dict(os.environ, PIKE_PDL=flag), timeout=300)
        assert res.returncode == 0, res.stderr[-1000:]
        digests.append([l for l in res.stdout.splitlines() if l.startswith("DIGEST")][0])
    assert digests[0] == digests[1]
