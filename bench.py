#!/usr/bin/env python
"""Benchmark of the fused operator chains on B200.

One *step* is one pass of the whole hot path: the five chain workloads C1..C5
(fp32 linear+GELU+LayerNorm, bf16 linear+SiLU+scale+residual, bf16 MLP block, bf16
logits+softmax, bf16 causal attention) run back to back through the library's public
API.  `value` is GEMM TFLOP/s of the whole step (2 flops per multiply-add of the
GEMMs only; attention counts the causal half), aggregated over all ranks.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 launch under torchrun; every rank runs the same suite on its own GPU
(rows / heads are independent, so the path shards without any collective: weak
scaling) and rank 0 prints one JSON line.  `--impl reference` times the fp64 CPU
oracle on a bounded row sample of the same workloads on the host cores.

The K timed steps run twice: once with nothing but the library calls between the two outer events
(`value`, `ms_per_step`: what a caller gets) and once more with every chain and every kernel launch
between its own pair of CUDA events (`instrumented_ms_per_step`, a few per cent longer: 26 event records
per step, and a kernel behind an event cannot start its prologue in its predecessor's tail);
`per_config`, `kernels` and `roofline` come from the instrumented pass.

Beside the contract's keys the line carries:
  sustained   the same step looped for at least two seconds with the clocks sampled: the
              power-capped regime, with its own roofline against the sustained library figure
  per_config  per chain: ms, TFLOP/s, fraction of the nominal 2250 TFLOP/s, eager time and
              speed-up; X1..X4 (the further workloads, outside `value`) when N == 1
  context     other ways to run the same chains on this GPU (fused library attention,
              torch.compile): context rows, never a denominator
  kernels     live device time per kernel of the library, with its own bound
  host_call_us  what one call costs on the host (C ABI through prebuilt ctypes arguments)
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused_chain_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
# x, W, residual and output once each: C2 134.2 MB, C3 GEMM1 469.8 MB, C3 GEMM2 469.8 MB, C4 541.1 MB
GEMM_ALGORITHMIC_BYTES_PER_STEP = 1.615e9
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the four gemm_bf16_kernel launches of one step,
# from the ncu captures summarised in profiles/gemm_bf16_kernel_dram_per_step.md: the value used, the spread
# over repeated captures, and the SHA-256 (first 16 hex digits) of the kernel's sources at capture time.  The
# line reports the traffic only while the sources still hash to that value.
GEMM_DRAM_CAPTURE = {"bytes": 2.5207e9, "min": 2.5181e9, "max": 2.5239e9, "captures": 3, "sources_sha16": "0c8a6814caf58ca6"}
GEMM_SOURCES = ("paper_2511_16964_b200/csrc/kernels/gemm_bf16.cu", "paper_2511_16964_b200/csrc/kernels/gemm_tile.cuh",
                "paper_2511_16964_b200/csrc/device/ptx.cuh", "paper_2511_16964_b200/csrc/device/act.cuh",
                "paper_2511_16964_b200/csrc/kernels/kernels.h")


def sources_sha16(paths=GEMM_SOURCES) -> str:
    h = hashlib.sha256()
    for p in paths:
        with open(os.path.join(ROOT, p), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


# ----------------------------------------------------------------------------
# workload definition (shapes from the five configs; flops = GEMM flops only)
# ----------------------------------------------------------------------------
def flops_per_config():
    return {
        "C1": 2.0 * 128 * 256 * 256,
        "C2": 2.0 * 4096 * 4096 * 4096,
        "C3": 2.0 * 2 * 8192 * 4096 * 16384,
        "C4": 2.0 * 2048 * 4096 * 32000,
        "C5": 4.0 * 8 * 32 * 128 * (2048 * 2049 / 2),
        # X1 (not part of the default step): attention block with fused projections, B8 S2048 E4096 (32 heads)
        "X1": 2.0 * 16384 * 4096 * (3 * 4096) + 4.0 * 8 * 32 * 128 * (2048 * 2049 / 2) + 2.0 * 16384 * 4096 * 4096,
        # X2 (not part of the default step): grouped linear + SiLU, 16384 rows over 32 weight matrices 2048 x 4096
        "X2": 2.0 * 16384 * 2048 * 4096,
        # X3 (not part of the default step): C4's logits + softmax with the 32000 columns split over the ranks
        # (whole-job flops; every rank does 1/world of them)
        "X3": 2.0 * 2048 * 4096 * 32000,
        # X4 (not part of the default step): C4's logits + softmax as ONE kernel (PIKE_FLAG_ONE_PASS)
        "X4": 2.0 * 2048 * 4096 * 32000,
    }


# flops of the launches of gemm_bf16_kernel inside each workload
def gemm_kernel_flops():
    f = flops_per_config()
    return {"C2": f["C2"], "C3": f["C3"], "C4": f["C4"], "X1": 2.0 * 16384 * 4096 * (4 * 4096), "X2": f["X2"],
            "X3": f["X3"], "X4": f["X4"]}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------
# clocks sampling during the timed region
# ----------------------------------------------------------------------------
class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, period_ms: int = 20):
        self.index, self.rows, self.proc, self.period_ms = index, [], None, period_ms
        self.t_first = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms",
                 str(self.period_ms), "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            if self.t_first is None:
                self.t_first = time.perf_counter()
            self.rows.append([c.strip() for c in line.split(",")])

    def wait_first_sample(self, timeout=3.0):
        """nvidia-smi needs a moment to start: a short region would otherwise end before the first sample."""
        t0 = time.perf_counter()
        while self.proc is not None and not self.rows and time.perf_counter() - t0 < timeout:
            time.sleep(0.005)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_min_mhz": min(sm) if sm else None,
                "sm_max_mhz": max(mx) if mx else None, "power_w_max": max(power) if power else None,
                "samples": len(sm), "period_ms": self.period_ms, "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# the CPU oracle on a bounded sample (cpu_baseline leg and --impl reference)
# ----------------------------------------------------------------------------
ORACLE_SAMPLE = {"C1": 128, "C2": 4096, "C3": 288, "C4": 576, "C5_heads": 72}


def oracle_sample_step(inputs):
    """One pass of the oracle over the bounded sample; returns (flops, seconds, seconds per config)."""
    from oracle import pike_oracle as O
    f = flops_per_config()
    c1, c2, c3, c4, c5 = (inputs[k] for k in ("C1", "C2", "C3", "C4", "C5"))
    n = ORACLE_SAMPLE
    flops, per = 0.0, {}
    t0 = t = time.perf_counter()

    def lap(name):
        nonlocal t
        now = time.perf_counter()
        per[name] = now - t
        t = now

    O.linear_epilogue(c1["x"], c1["w"], c1["b"], None, c1["gamma"], c1["beta"], act="gelu_erf",
                      reduce="layernorm", eps=c1["eps"])
    flops += f["C1"]
    lap("C1")
    O.linear_epilogue(c2["x"], c2["w"], c2["b"], c2["r"], act="silu", scale=0.5, rows=np.arange(n["C2"]))
    flops += f["C2"] * n["C2"] / 4096
    lap("C2")
    O.mlp_block(c3["x"], c3["gamma"], c3["beta"], c3["w1"], c3["b1"], c3["w2"], c3["b2"], act="gelu_tanh",
                eps=c3["eps"], rows=np.arange(n["C3"]))
    flops += f["C3"] * n["C3"] / 8192
    lap("C3")
    O.linear_epilogue(c4["x"], c4["w"], reduce="softmax", rows=np.arange(n["C4"]))
    flops += f["C4"] * n["C4"] / 2048
    lap("C4")
    for i in range(n["C5_heads"]):
        b, h = divmod(i, 32)
        O.attention_head(c5["q"][b, h], c5["k"][b, h], c5["v"][b, h], scale=c5["scale"], causal=True)
    flops += f["C5"] * n["C5_heads"] / 256
    lap("C5")
    return flops, time.perf_counter() - t0, per


def oracle_full_size_seconds(per):
    """Seconds the oracle would need for the whole step: every config's sample time scaled by rows (or heads)
    total / sampled - rows and heads are independent, so the cost is linear in them."""
    n = ORACLE_SAMPLE
    scale = {"C1": 1.0, "C2": 4096 / n["C2"], "C3": 8192 / n["C3"], "C4": 2048 / n["C4"], "C5": 256 / n["C5_heads"]}
    return {k: per[k] * scale[k] for k in per}


def oracle_sample_text():
    n = ORACLE_SAMPLE
    return (f"C1 all 128 rows; C2 first {n['C2']} of 4096 rows; C3 first {n['C3']} of 8192 rows; "
            f"C4 first {n['C4']} of 2048 rows; C5 first {n['C5_heads']} of 256 heads (rows and heads are independent)")


ALL = ("C1", "C2", "C3", "C4", "C5")          # the step
EXTRA = ("X1", "X2", "X3", "X4")             # further workloads: with --only, or after the step when N == 1


def max_over_ranks(ms: float, world: int, device=None) -> float:
    """The slowest rank's time: the whole job is only done when the last rank is."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_tflops(step_flops: float, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank processes one full suite per step (weak scaling)."""
    return world * step_flops / (ms_per_step * 1e-3) / 1e12


def rank_env():
    """(rank, world, local_rank) as torchrun exports them; a plain `python bench.py` is rank 0 of 1."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def per_rank_flops(only, world: int) -> dict:
    """GEMM flops ONE rank processes per step, per workload.  C1..C5, X1, X2 are replicated (every rank runs the
    whole workload on its own rows or heads: weak scaling, job_tflops multiplies by world); X3 splits the columns of
    one problem over the ranks (strong scaling), so a rank does 1/world of it."""
    f = {k: v for k, v in flops_per_config().items() if k in only}
    if "X3" in f:
        f["X3"] /= world
    return f


def make_inputs(only=ALL):
    import pike_inputs as G
    gen = {"C1": G.config1, "C2": G.config2, "C3": G.config3, "C4": G.config4, "C5": G.config5,
           "X1": lambda: G.attention_block(B=8, S=2048, E=4096), "X2": G.grouped_linear,
           "X3": G.config4, "X4": G.config4}
    return {k: gen[k]() for k in only}


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on the host cores."""
    rank, _, _ = rank_env()
    if rank != 0:
        return 0
    from oracle import pike_oracle as O
    O.build()
    inputs = make_inputs()
    for _ in range(max(0, args.ref_warmup)):
        oracle_sample_step(inputs)
    total_f, total_t, per = 0.0, 0.0, {}
    for _ in range(args.ref_steps):
        fl, dt, per = oracle_sample_step(inputs)
        total_f += fl
        total_t += dt
    value = total_f / total_t / 1e12
    full = oracle_full_size_seconds(per)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.ref_steps, "warmup": args.ref_warmup, "ms_per_step": 1e3 * total_t / args.ref_steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "C1-C5 chain suite", "note": "fp64 CPU oracle on a bounded row sample per step; "
                   "the requested --steps/--warmup are mapped to %d/%d oracle passes" % (args.ref_steps, args.ref_warmup)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
                         "sample": oracle_sample_text(), "full_size_seconds_extrapolated": sum(full.values()),
                         "full_size_seconds_per_config": full},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)
    return 0


# ----------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------
class Suite:
    """Device tensors, outputs, workspaces and the chain calls of a set of workloads."""

    def __init__(self, P, torch, device, only, rank=0, world=1):
        BF16, F32 = torch.bfloat16, torch.float32
        self.only = tuple(only)
        self.inputs = inputs = make_inputs(self.only)

        def pin(a, dtype):
            return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dtype).pin_memory()

        c1, c2, c3, c4, c5 = (inputs.get(k) for k in ALL)
        x1, x2, x3, x4 = (inputs.get(k) for k in EXTRA)
        host_act, wts = {}, {}   # activations are copied host -> device every e2e step; weights stay resident in HBM
        if c1:
            host_act.update(c1x=pin(c1["x"], F32))
            wts.update(c1w=pin(c1["w"], F32), c1b=pin(c1["b"], F32), c1g=pin(c1["gamma"], F32), c1be=pin(c1["beta"], F32))
        if c2:
            host_act.update(c2x=pin(c2["x"], BF16), c2r=pin(c2["r"], BF16))
            wts.update(c2w=pin(c2["w"], BF16), c2b=pin(c2["b"], BF16))
        if c3:
            host_act.update(c3x=pin(c3["x"], BF16))
            wts.update(c3w1=pin(c3["w1"], BF16), c3b1=pin(c3["b1"], BF16), c3w2=pin(c3["w2"], BF16),
                       c3b2=pin(c3["b2"], BF16), c3g=pin(c3["gamma"], BF16), c3be=pin(c3["beta"], BF16))
        if c4:
            host_act.update(c4x=pin(c4["x"], BF16))
            wts.update(c4w=pin(c4["w"], BF16))
        if c5:
            host_act.update(c5q=pin(c5["q"], BF16), c5k=pin(c5["k"], BF16), c5v=pin(c5["v"], BF16))
        if x1:
            host_act.update(x1x=pin(x1["x"], BF16))
            wts.update(x1wq=pin(x1["w_qkv"], BF16), x1bq=pin(x1["b_qkv"], BF16), x1wo=pin(x1["w_o"], BF16),
                       x1bo=pin(x1["b_o"], BF16), x1g=pin(x1["gamma"], BF16), x1be=pin(x1["beta"], BF16))
        if x2:
            host_act.update(x2x=pin(x2["x"], BF16))
            wts.update(x2w=pin(x2["w"], BF16), x2b=pin(x2["b"], BF16))
        x3_cols = (0, 0)
        if x3:
            x3_cols = P.vocab_shard_range(32000, rank, world)
            host_act.update(x3x=pin(x3["x"], BF16))
            wts.update(x3w=pin(x3["w"][:, x3_cols[0]:x3_cols[1]], BF16))
        if x4:
            host_act.update(x4x=pin(x4["x"], BF16))
            wts.update(x4w=pin(x4["w"], BF16))
        self.host_act = host_act
        self.d = d = {k: v.to(device) for k, v in host_act.items()}
        d.update({k: v.to(device) for k, v in wts.items()})
        shapes = {"C1": ((128, 256), F32), "C2": ((4096, 4096), BF16), "C3": ((8192, 4096), BF16),
                  "C4": ((2048, 32000), F32), "C5": ((8, 32, 2048, 128), BF16), "X1": ((8, 2048, 4096), BF16),
                  "X2": ((16384, 4096), BF16), "X3": ((2048, x3_cols[1] - x3_cols[0]), F32), "X4": ((2048, 32000), F32)}
        self.out = out = {k: torch.empty(shapes[k][0], dtype=shapes[k][1], device=device) for k in self.only}
        self.host_out = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in out.items()}
        ws0 = torch.empty(256, dtype=torch.uint8, device=device)
        ws3 = ws4 = wsx = wsx3 = wsx4 = ws0
        if x4:
            wsx4 = torch.empty(P.pike_linear_epilogue_workspace(d["x4x"], d["x4w"], reduce="softmax", out_dtype=F32,
                                                                one_pass=True), dtype=torch.uint8, device=device)
        if x3:
            wsx3 = torch.empty(P.pike_linear_softmax_shard_workspace(d["x3x"], d["x3w"]), dtype=torch.uint8, device=device)
        if x1:
            wsx = torch.empty(P.pike_attention_block_workspace(d["x1x"], scale=float(x1["scale"])), dtype=torch.uint8,
                              device=device)
        if c3:
            ws3 = torch.empty(P.pike_mlp_block_workspace(d["c3x"], d["c3w1"]), dtype=torch.uint8, device=device)
        if c4:
            ws4 = torch.empty(P.pike_linear_epilogue_workspace(d["c4x"], d["c4w"], reduce="softmax", out_dtype=F32),
                              dtype=torch.uint8, device=device)
        x2off = torch.from_numpy(x2["offsets"]).to(device) if x2 else None
        if x2:
            d["x2off_host"] = [int(o) for o in x2["offsets"]]
        chains = {
            "C1": lambda: P.pike_linear_epilogue(d["c1x"], d["c1w"], d["c1b"], None, d["c1g"], d["c1be"], act="gelu_erf",
                                                 reduce="layernorm", eps=c1["eps"], out=out["C1"], workspace=ws0),
            "C2": lambda: P.pike_linear_epilogue(d["c2x"], d["c2w"], d["c2b"], d["c2r"], act="silu", scale=0.5,
                                                 out=out["C2"], workspace=ws0),
            "C3": lambda: P.pike_mlp_block(d["c3x"], d["c3g"], d["c3be"], d["c3w1"], d["c3b1"], d["c3w2"], d["c3b2"],
                                           act="gelu_tanh", eps=c3["eps"], out=out["C3"], workspace=ws3),
            "C4": lambda: P.pike_linear_epilogue(d["c4x"], d["c4w"], reduce="softmax", out_dtype=F32, out=out["C4"],
                                                 workspace=ws4),
            "C5": lambda: P.pike_attention_chain(d["c5q"], d["c5k"], d["c5v"], scale=float(c5["scale"]), causal=True,
                                                 out=out["C5"]),
            "X1": lambda: P.pike_attention_block(d["x1x"], d["x1g"], d["x1be"], d["x1wq"], d["x1bq"], d["x1wo"], d["x1bo"],
                                                 scale=float(x1["scale"]), causal=True, eps=x1["eps"], out=out["X1"],
                                                 workspace=wsx),
            "X2": lambda: P.pike_grouped_linear_epilogue(d["x2x"], d["x2w"], d["x2b"], None, x2off, act="silu",
                                                         out=out["X2"]),
            # the exchange between the two library calls is an all-gather of 16 KiB per rank over the default group
            "X3": lambda: P.linear_softmax_vocab_sharded(d["x3x"], d["x3w"], out=out["X3"], workspace=wsx3),
            "X4": lambda: P.pike_linear_epilogue(d["x4x"], d["x4w"], reduce="softmax", out_dtype=F32, one_pass=True,
                                                 out=out["X4"], workspace=wsx4),
        }
        self.chains = {n: chains[n] for n in chains if n in self.only}
        self.names = list(self.chains)
        self.attn_scale = float((c5 or x1 or {"scale": 1.0})["scale"])

    def step(self, torch, events=None):
        for n in self.names:
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            self.chains[n]()
            if events is not None:
                e1.record()
                events[n].append((e0, e1))


def timed_steps(P, torch, suite, steps, barrier, sampler=None, instrument=True):
    """`steps` steps bracketed by a barrier + synchronise on both sides, timed with CUDA events on the launching
    stream; returns (total ms, mean ms per chain, per-kernel profile, clocks).  With `instrument` every chain and
    every kernel launch is bracketed by its own pair of events (26 event records per step, which also keep a
    kernel's prologue from overlapping its predecessor's tail); without it nothing but the calls is enqueued
    between the two outer events, and the per-chain and per-kernel results are None."""
    if not instrument:
        if sampler is not None:
            sampler.start()
            sampler.wait_first_sample()
        barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        for _ in range(steps):
            suite.step(torch)
        t1.record()
        barrier()
        return t0.elapsed_time(t1), None, None, (sampler.stop() if sampler is not None else None)
    events = {n: [] for n in suite.names}
    if sampler is not None:
        sampler.start()
        sampler.wait_first_sample()
    P.pike_profile_begin()
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(steps):
        suite.step(torch, events)
    t1.record()
    barrier()
    total_ms = t0.elapsed_time(t1)
    prof = P.pike_profile_end()
    clocks = sampler.stop() if sampler is not None else None
    per_cfg = {n: float(np.mean([a.elapsed_time(b) for a, b in events[n]])) for n in suite.names}
    return total_ms, per_cfg, prof, clocks


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2511_16964_b200 as P

    rank, world, local_rank = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)
    P.load_library()

    only = args.only
    suite = Suite(P, torch, device, only, rank, world)
    names = suite.names
    f = per_rank_flops(only, world)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up, then the timed region ------------------------------------------------
    for _ in range(args.warmup):
        suite.step(torch)
    barrier()
    st, where = P.pike_get_last_device_status()
    if st != 0:
        raise SystemExit(f"device status {st} at {where:#x} during warm-up")

    # the timed region proper: exactly K steps with nothing but the library calls between the two events ...
    total_ms, _, _, clocks = timed_steps(P, torch, suite, args.steps, barrier,
                                         ClockSampler(local_rank) if rank == 0 else None, instrument=False)
    total_ms = max_over_ranks(total_ms, world, device)
    ms_per_step = total_ms / args.steps
    # ... and the same K steps once more with every chain and every kernel launch between its own events: the
    # per-config and per-kernel times and the roofline come from this pass, which the events make a few per cent longer
    instr_ms, per_cfg_ms, prof, _ = timed_steps(P, torch, suite, args.steps, barrier)
    instr_ms = max_over_ranks(instr_ms, world, device)
    step_flops = sum(f.values())
    value = job_tflops(step_flops, world, ms_per_step)

    # ---- end to end: host buffers in, host buffers out, copies inside the timed region ---
    e2e_steps = max(1, min(args.steps, 5))
    host_act, host_out, d, out, chains = suite.host_act, suite.host_out, suite.d, suite.out, suite.chains
    h2d = sum(v.numel() * v.element_size() for v in host_act.values())
    d2h = sum(v.numel() * v.element_size() for v in host_out.values())

    # Copies run on their own streams so that a workload's input upload, its kernels and the download of the
    # previous result overlap (PCIe is full duplex); events order them per workload: kernels after their inputs,
    # the download after the kernels, the next upload after the kernels that read the old inputs, the next kernels
    # after the download that reads the old output.  Every byte still moves inside the timed region.
    cur, s_in, s_out = torch.cuda.current_stream(), torch.cuda.Stream(device=device), torch.cuda.Stream(device=device)
    ins_of = {n: [k for k in host_act if k[:2].upper() == n] for n in names}
    ev_in, ev_done, ev_out = ({n: torch.cuda.Event() for n in names} for _ in range(3))
    ran = {"once": False}

    def e2e_step():
        with torch.cuda.stream(s_in):
            for n in names:
                if ran["once"]:
                    s_in.wait_event(ev_done[n])
                for k in ins_of[n]:
                    d[k].copy_(host_act[k], non_blocking=True)
                ev_in[n].record(s_in)
        for n in names:
            cur.wait_event(ev_in[n])
            if ran["once"]:
                cur.wait_event(ev_out[n])
            chains[n]()
            ev_done[n].record(cur)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[n])
                host_out[n].copy_(out[n], non_blocking=True)
                ev_out[n].record(s_out)
        ran["once"] = True

    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    cur.wait_stream(s_in)
    cur.wait_stream(s_out)
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    # the host copies of the results are the device buffers, bit for bit
    e2e_match = all(bool(torch.equal(host_out[n], out[n].cpu())) for n in names)
    e2e_ms = max_over_ranks(e2e_ms, world, device)
    e2e_value = job_tflops(step_flops, world, e2e_ms)

    # ---- warm series: each chain 20 times back to back (nothing else evicts its operands from L2 in between;
    # only the chains whose tensors fit the 126 MB L2 differ from the cold per-step times) ------------------
    warm_ms = {}
    for n in names:
        for _ in range(3):
            chains[n]()
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record()
        for _ in range(20):
            chains[n]()
        w1.record()
        torch.cuda.synchronize()
        warm_ms[n] = w0.elapsed_time(w1) / 20
    # The whole step captured once into a CUDA graph and replayed: what the launch path costs beyond the kernels
    # (a chain call only launches kernels into caller-owned buffers, so it can be captured).  Context, not `value`.
    graph_ms = None
    if tuple(only) == ALL:
        try:
            gstream = torch.cuda.Stream(device=device)
            gstream.wait_stream(torch.cuda.current_stream())
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.stream(gstream):
                for n in names:
                    chains[n]()
                gstream.synchronize()
                with torch.cuda.graph(graph, stream=gstream):
                    for n in names:
                        chains[n]()
                for _ in range(3):
                    graph.replay()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record()
                for _ in range(20):
                    graph.replay()
                g1.record()
            torch.cuda.synchronize()
            graph_ms = g0.elapsed_time(g1) / 20
            del graph
        except Exception as exc:           # noqa: BLE001 - a context figure must never break the benchmark
            graph_ms = "failed: " + repr(exc)[:160]

    # ---- sustained: the same step looped for seconds, clocks sampled: the power-capped regime ------------
    sustained = None
    peaks = load_peaks()
    if args.sustained_seconds > 0 and tuple(only) == ALL:
        n_steps = max(args.steps, int(args.sustained_seconds * 1e3 / ms_per_step) + 1)
        s_ms, _, _, s_clocks = timed_steps(P, torch, suite, n_steps, barrier,
                                           ClockSampler(local_rank, 50) if rank == 0 else None, instrument=False)
        s_ms = max_over_ranks(s_ms, world, device)
        s_instr_ms, s_cfg, s_prof, _ = timed_steps(P, torch, suite, n_steps, barrier)
        s_instr_ms = max_over_ranks(s_instr_ms, world, device)
        gl, gms = s_prof["gemm_bf16"]
        gtf = sum(gemm_kernel_flops()[k] for k in ("C2", "C3", "C4")) * n_steps / (gms * 1e-3) / 1e12
        sustained = {
            "steps": n_steps, "seconds": s_ms * 1e-3, "ms_per_step": s_ms / n_steps,
            "instrumented_ms_per_step": s_instr_ms / n_steps,
            "value": job_tflops(step_flops, world, s_ms / n_steps), "unit": UNIT, "clocks": s_clocks,
            "per_config": {n: {"ms": s_cfg[n], "tflops": f[n] / (s_cfg[n] * 1e-3) / 1e12,
                               "frac_of_nominal_2250": f[n] / (s_cfg[n] * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS,
                               "meets_60pct_of_nominal": bool(f[n] / (s_cfg[n] * 1e-3) / 1e12 >= 0.6 * NOMINAL_BF16_TFLOPS)}
                           for n in names},
            "roofline": {"kernel": "gemm_bf16_kernel", "bound": "tensor", "achieved": gtf,
                         "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "frac": gtf / peaks["bf16_tflops_sustained"],
                         "peak_source": f"{peaks['source']} cuBLAS bf16, sustained figure",
                         "frac_of_nominal_2250": gtf / NOMINAL_BF16_TFLOPS, "launches": gl},
            "kernels": {k: {"launches": v[0], "ms_per_step": v[1] / n_steps} for k, v in s_prof.items()},
        }

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return 0

    # ---- rank 0 only: eager comparison, context rows, further workloads, parity, CPU baseline, JSON -------
    gemm_launches, gemm_ms = prof["gemm_bf16"]
    gkf = gemm_kernel_flops()
    gemm_flops = sum(gkf[k] / (world if k == "X3" else 1) for k in gkf if k in f)
    gemm_tflops = gemm_flops * args.steps / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else None
    # a long timed region runs under the power cap: compare with the sustained library figure
    capped = total_ms > 500.0 or "sw_power_cap" in (clocks or {}).get("reasons", [])
    peak = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
    cap = GEMM_DRAM_CAPTURE
    traffic_valid = tuple(only) == ALL and cap["bytes"] is not None and cap["sources_sha16"] == sources_sha16()
    roofline = {
        "kernel": "gemm_bf16_kernel", "bound": "tensor", "achieved": gemm_tflops, "peak": peak, "unit": "TFLOP/s",
        "frac": (gemm_tflops / peak) if gemm_tflops else None,
        "peak_source": f"{peaks['source']} cuBLAS bf16, {'sustained' if capped else 'burst'} figure",
        "frac_of_nominal_2250": (gemm_tflops / NOMINAL_BF16_TFLOPS) if gemm_tflops else None,
        "launches": gemm_launches,
        # DRAM bytes of the kernel's four launches of one step from the ncu captures summarised under profiles/;
        # null for partial suites and whenever the kernel's sources no longer hash to the captured build
        "traffic": cap["bytes"] if traffic_valid else None,
        "traffic_min_max": [cap["min"], cap["max"]] if traffic_valid else None,
        "traffic_captures": cap["captures"] if traffic_valid else None,
        "traffic_sources_sha16": cap["sources_sha16"], "sources_sha16_now": sources_sha16(),
        "traffic_unit": "bytes per step (4 launches)", "algorithmic_bytes": GEMM_ALGORITHMIC_BYTES_PER_STEP,
    }

    if "X3" in only and not args.no_eager:   # the eager comparison is the unsharded chain on one GPU
        d["x3w_full"] = torch.from_numpy(np.ascontiguousarray(suite.inputs["X3"]["w"], np.float32)).to(torch.bfloat16).to(device)
    eager_ms = {} if args.no_eager else eager_baseline(torch, d, suite.attn_scale, names)
    context = None if (args.no_eager or args.no_context) else context_rows(torch, d, suite.attn_scale, names)
    library_gemm = None if args.no_eager else library_gemm_context(torch, device, ClockSampler(local_rank, 50))
    if tuple(only) != ALL:
        args.no_parity = args.no_cpu_baseline = args.no_extras = True      # partial suites are profiling runs

    def config_row(n, ms, fl, warm=None, eager=None):
        row = {"ms": ms, "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_nominal_2250": fl / (ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS}
        row["meets_60pct_of_nominal"] = bool(row["frac_of_nominal_2250"] >= 0.6)
        if warm is not None:
            row["warm_ms"] = warm
        if eager is not None:
            row["eager_ms"] = eager
            row["speedup_vs_eager"] = eager / ms
        return row

    per_config = {n: config_row(n, per_cfg_ms[n], f[n], warm_ms[n], eager_ms.get(n)) for n in names}
    kernels = {k: {"launches": v[0], "ms_per_step": v[1] / args.steps} for k, v in prof.items()}
    # the other kernels of the default step against their own bounds (algorithmic bytes / flops per launch)
    if tuple(only) == ALL:
        def _bw(name, nbytes, into=kernels):
            ms = into[name]["ms_per_step"]
            gbs = nbytes / (ms * 1e-3) / 1e9 if ms > 0 else None
            into[name].update(bound="hbm", achieved=gbs, unit="GB/s", peak=peaks["hbm_gbs"],
                              frac=(gbs / peaks["hbm_gbs"]) if gbs else None)
        for block, pk in ((kernels, peak), (sustained["kernels"] if sustained else None, peaks["bf16_tflops_sustained"])):
            if block is None:
                continue
            _bw("layernorm_bf16", 2.0 * 8192 * 4096 * 2, block)                      # C3 prologue: x in, z out
            _bw("softmax_finish", 2.0 * 2048 * 32000 * 4 + 2048 * 125 * 8, block)    # C4: logits in, probabilities out, pairs
            ms = block["attention_bf16"]["ms_per_step"]
            tf = f["C5"] / (ms * 1e-3) / 1e12 if ms > 0 else None
            block["attention_bf16"].update(bound="tensor + sfu", achieved=tf, unit="TFLOP/s", peak=pk,
                                           frac=(tf / pk) if tf else None,
                                           frac_of_nominal_2250=(tf / NOMINAL_BF16_TFLOPS) if tf else None)

    parity = None if args.no_parity else parity_spot_check(suite.inputs, out)
    host_call_us = None if tuple(only) != ALL else host_call_overhead(P, torch, suite)

    cpu_baseline = None
    if not args.no_cpu_baseline:
        from oracle import pike_oracle as O
        fl, dt, per = oracle_sample_step(suite.inputs)
        full = oracle_full_size_seconds(per)
        cpu_baseline = {"value": fl / dt / 1e12, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle",
                        "sample": oracle_sample_text(), "seconds": dt,
                        "full_size_seconds_extrapolated": sum(full.values()), "full_size_seconds_per_config": full}

    # ---- the further workloads (outside `value`): one at a time, each with its own tensors ---------------
    variants = None
    if world == 1 and not args.no_extras:
        del suite, d, out, chains, host_act, host_out
        torch.cuda.empty_cache()
        for x in EXTRA:
            per_config[x] = extra_workload(P, torch, device, x, not args.no_eager)
        variants = variant_rows(P, torch, device)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "instrumented_ms_per_step": instr_ms / args.steps, "higher_is_better": True,
        "scaling": "strong" if tuple(only) == ("X3",) else "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": ("" if tuple(only) == ALL else "SUBSET " + ",".join(only) + " of the ") +
                               "C1-C5 chain suite (fp32 linear+GELU+LN 128x256x256; bf16 linear+SiLU+scale+residual "
                               "4096^3; bf16 MLP block 8192x4096x16384; bf16 logits+softmax 2048x4096x32000; bf16 "
                               "causal attention B8 H32 S2048 D128)",
                   "l2": "no explicit flush: one step streams about 3.4 GB of distinct tensors, 27x the 126 MB L2, "
                         "so every chain starts with its inputs evicted",
                   "warm_ms": "per_config.warm_ms = the same chain 20 times back to back without per-kernel events "
                              "(short bursts run at higher clocks; for C1 it is the host's call rate)",
                   "extras": "per_config X1..X4 are further workloads timed after the step (10 runs each, tensors "
                             "larger than L2), not part of value; X4 = C4 as one kernel (PIKE_FLAG_ONE_PASS)",
                   "graph": "graph_replay_ms_per_step = the five chains captured once into a CUDA graph, replayed 20 times "
                            "back to back (no per-kernel events): context, not part of value",
                   "weights": "resident in HBM", "flops": "GEMM multiply-adds x2; attention counts the causal half"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "host_results_match_device": e2e_match,
                "copies": "overlapped with the kernels on separate streams"},
        "gpu_launches": int(sum(v[0] for v in prof.values())),
        "roofline": roofline, "cpu_baseline": cpu_baseline,
        "frac_of_nominal_2250": value / world / NOMINAL_BF16_TFLOPS,
        "sustained": sustained, "per_config": per_config, "context": context, "kernels": kernels, "parity": parity,
        "host_call_us": host_call_us, "library_gemm_same_box": library_gemm,
        "graph_replay_ms_per_step": graph_ms, "variants": variants,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def extra_workload(P, torch, device, name, with_eager, iters=10):
    """One of X1..X4 on its own: 3 warm-up runs, then `iters` runs timed one by one with CUDA events."""
    s = Suite(P, torch, device, (name,))
    fl = flops_per_config()[name]
    for _ in range(3):
        s.chains[name]()
    torch.cuda.synchronize()
    ts = []
    P.pike_profile_begin()
    for _ in range(iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        s.chains[name]()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    prof = P.pike_profile_end()
    ms = float(np.mean(ts))
    row = {"ms": ms, "tflops": fl / (ms * 1e-3) / 1e12, "frac_of_nominal_2250": fl / (ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS,
           "min_ms": float(min(ts)), "runs": iters, "in_value": False,
           "kernels": {k: {"launches": v[0] // iters, "ms": v[1] / iters} for k, v in prof.items() if v[0]}}
    gms = prof["gemm_bf16"][1] / iters
    if gms > 0:
        row["gemm_kernel_tflops"] = gemm_kernel_flops()[name] / (gms * 1e-3) / 1e12
    if with_eager:
        if name == "X3":
            s.d["x3w_full"] = s.d["x3w"]
        e = eager_baseline(torch, s.d, s.attn_scale, [name])
        row["eager_ms"] = e[name]
        row["speedup_vs_eager"] = e[name] / ms
    st, where = P.pike_get_last_device_status()
    row["device_status"] = st
    del s
    torch.cuda.empty_cache()
    return row


def variant_rows(P, torch, device, runs=5):
    """Further shapes and types the entry points accept (parity of each in tests/): timed here cold, one by one, on
    seeded random tensors; never part of `value`.  TFLOP/s counts GEMM flops (attention: the live half under the mask)."""
    BF16, F16, F32 = torch.bfloat16, torch.float16, torch.float32
    g = torch.Generator(device=device).manual_seed(2511)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)

    def rn(*shape, dt=BF16, sc=1.0):
        return (torch.randn(*shape, device=device, generator=g) * sc).to(dt)

    def attn(B, H, S, Sk, D, dt, causal):
        q, k, v = rn(B, H, S, D, dt=dt), rn(B, H, Sk, D, dt=dt), rn(B, H, Sk, D, dt=dt)
        o = torch.empty_like(q)
        fl = 4.0 * B * H * D * (S * (S + 1) / 2 if causal else S * Sk)
        return (lambda: P.pike_attention_chain(q, k, v, scale=D ** -0.5, causal=causal, out=o)), fl

    def linear(M, K, N, dt, **kw):
        x, w, b = rn(M, K, dt=dt), rn(K, N, dt=dt, sc=K ** -0.5), rn(N, dt=dt)
        r = rn(M, N, dt=dt) if kw.pop("residual", False) else None
        gm, be = (rn(N, dt=dt), rn(N, dt=dt)) if kw.get("reduce") == "layernorm" else (None, None)
        o = torch.empty((M, N), dtype=kw.get("out_dtype", dt), device=device)
        nbytes = P.pike_linear_epilogue_workspace(x, w, **{k: v for k, v in kw.items() if k in ("act", "scale", "reduce", "eps", "out_dtype")})
        ws = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=device)
        return (lambda: P.pike_linear_epilogue(x, w, b, r, gm, be, out=o, workspace=ws, **kw)), 2.0 * M * K * N

    cases = {
        "attention non-causal bf16 B8 H32 S2048 D128": lambda: attn(8, 32, 2048, 2048, 128, BF16, False),
        "attention causal bf16 B8 H64 S2048 D64": lambda: attn(8, 64, 2048, 2048, 64, BF16, True),
        "attention causal f16 B8 H32 S2048 D128": lambda: attn(8, 32, 2048, 2048, 128, F16, True),
        "cross attention bf16 B8 H32 S1024 Sk4096 D128": lambda: attn(8, 32, 1024, 4096, 128, BF16, False),
        "linear+GELU+LayerNorm (split-row epilogue) bf16 8192x4096x4096": lambda: linear(8192, 4096, 4096, BF16, act="gelu_tanh", reduce="layernorm"),
        "linear+SiLU+scale+residual f16 4096^3": lambda: linear(4096, 4096, 4096, F16, act="silu", scale=0.5, residual=True),
        # the fp32 CUDA-core chain on a problem that fills the chip (the path is built for small, latency-bound chains)
        "linear+GELU(erf)+LayerNorm fp32 8192x1024x1024": lambda: linear(8192, 1024, 1024, F32, act="gelu_erf", reduce="layernorm"),
    }
    rows = {}
    for name, make in cases.items():
        try:
            fn, fl = make()
            ms = _timed_cold(torch, fn, flush, iters=runs)
            rows[name] = {"ms": ms, "tflops": fl / (ms * 1e-3) / 1e12,
                          "frac_of_nominal_2250": fl / (ms * 1e-3) / 1e12 / NOMINAL_BF16_TFLOPS}
            if " fp32 " in name:     # nominal bf16 tensor peak says nothing about fp32 FMAs: give the unfused eager time instead
                del rows[name]["frac_of_nominal_2250"]
                x, w, b = rn(8192, 1024, dt=F32), rn(1024, 1024, dt=F32, sc=1 / 32), rn(1024, dt=F32)
                gm, be = rn(1024, dt=F32), rn(1024, dt=F32)
                tf32 = torch.backends.cuda.matmul.allow_tf32
                torch.backends.cuda.matmul.allow_tf32 = False
                rows[name]["eager_fp32_ms"] = _timed_cold(
                    torch, lambda: torch.nn.functional.layer_norm(torch.nn.functional.gelu(x @ w + b), (1024,), gm, be),
                    flush, iters=runs)
                torch.backends.cuda.matmul.allow_tf32 = tf32
                del x, w, b, gm, be
            del fn
        except Exception as exc:           # noqa: BLE001 - a context row must never break the benchmark
            rows[name] = {"ms": None, "error": repr(exc)[:200]}
        torch.cuda.empty_cache()
    st, _ = P.pike_get_last_device_status()
    rows["device_status"] = st
    return rows


def host_call_overhead(P, torch, suite, calls=400):
    """Microseconds of host time one library call costs, without the Python wrappers: the C entry point is
    called through ctypes with argument structs built once, and only the enqueue loop is timed (the queue is
    drained before and after, and `calls` stays below the depth at which launches start to block)."""
    import ctypes
    from paper_2511_16964_b200 import binding as B
    lib, d, out = B.load_library(), suite.d, suite.out
    h = B._handle(out["C1"].device)
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    res = {}
    e1 = B._epilogue("gelu_erf", 1.0, "layernorm", 1e-5, torch.float32, 0)
    a1 = [B._tensor(d[k]) for k in ("c1x", "c1w", "c1b")] + [None] + [B._tensor(d[k]) for k in ("c1g", "c1be")]
    o1 = B._tensor(out["C1"])
    e2 = B._epilogue("silu", 0.5, "none", 0.0, torch.bfloat16, 0)
    a2 = [B._tensor(d[k]) for k in ("c2x", "c2w", "c2b", "c2r")] + [None, None]
    o2 = B._tensor(out["C2"])
    for name, args_, e, o, n in (("pike_linear_epilogue_fp32_128x256x256", a1, e1, o1, calls),
                                 ("pike_linear_epilogue_bf16_4096^3", a2, e2, o2, 60)):
        for _ in range(3):
            lib.pike_linear_epilogue(h, *args_, e, o, None, 0, stream)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(n):
            lib.pike_linear_epilogue(h, *args_, e, o, None, 0, stream)
        t1 = time.perf_counter()
        torch.cuda.synchronize()
        res[name] = (t1 - t0) / n * 1e6
    # the same fp32 call through the Python wrapper, for comparison
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(calls):
        suite.chains["C1"]()
    t1 = time.perf_counter()
    torch.cuda.synchronize()
    res["python_wrapper_fp32_128x256x256"] = (t1 - t0) / calls * 1e6
    return res


def _timed_cold(torch, fn, flush, iters=3):
    fn()
    fn()
    torch.cuda.synchronize()
    ts = []
    for _ in range(iters):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        ts.append(e0.elapsed_time(e1))
    return float(np.mean(ts))


def eager_ops(torch, d, scale):
    F = torch.nn.functional

    def attn():
        q, k, v = d["c5q"], d["c5k"], d["c5v"]
        S = q.shape[2]
        s = (q @ k.transpose(-1, -2)) * scale
        mask = torch.ones((S, S), dtype=torch.bool, device=q.device).tril()
        s = s.masked_fill(~mask, float("-inf"))
        return torch.softmax(s, dim=-1) @ v

    def x2_eager():     # the per-expert loop the grouped kernel replaces
        off = d["x2off_host"]
        outs = [F.silu(d["x2x"][off[g]:off[g + 1]] @ d["x2w"][g] + d["x2b"][g]) for g in range(len(off) - 1)
                if off[g + 1] > off[g]]
        return torch.cat(outs)

    def x1_eager():
        x = d["x1x"]
        B, S, E = x.shape
        H = E // 128
        z = F.layer_norm(x, (E,), d["x1g"], d["x1be"], 1e-5)
        qkv = (z @ d["x1wq"] + d["x1bq"]).view(B, S, 3, H, 128)
        q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))
        sc = (q @ k.transpose(-1, -2)) * scale
        mask = torch.ones((S, S), dtype=torch.bool, device=x.device).tril()
        a = (torch.softmax(sc.masked_fill(~mask, float("-inf")), dim=-1) @ v).permute(0, 2, 1, 3).reshape(B, S, E)
        return x + a @ d["x1wo"] + d["x1bo"]

    return {
        "C1": lambda: F.layer_norm(F.gelu(d["c1x"] @ d["c1w"] + d["c1b"]), (256,), d["c1g"], d["c1be"], 1e-5),
        "C2": lambda: 0.5 * F.silu(d["c2x"] @ d["c2w"] + d["c2b"]) + d["c2r"],
        "C3": lambda: d["c3x"] + F.gelu(F.layer_norm(d["c3x"], (4096,), d["c3g"], d["c3be"], 1e-5) @ d["c3w1"]
                                        + d["c3b1"], approximate="tanh") @ d["c3w2"] + d["c3b2"],
        "C4": lambda: torch.softmax(d["c4x"] @ d["c4w"], dim=-1, dtype=torch.float32),
        "C5": attn,
        "X1": x1_eager,
        "X2": x2_eager,
        "X3": lambda: torch.softmax(d["x3x"] @ d["x3w_full"], dim=-1, dtype=torch.float32),
        "X4": lambda: torch.softmax(d["x4x"] @ d["x4w"], dim=-1, dtype=torch.float32),
    }


def eager_baseline(torch, d, scale, names, iters=3):
    """The same ops as separate PyTorch calls (TF32 off); ms per config, L2 flushed before every timed run."""
    torch.backends.cuda.matmul.allow_tf32 = False
    torch.backends.cudnn.allow_tf32 = False
    ops = eager_ops(torch, d, scale)
    device = next(v for v in d.values() if hasattr(v, "device")).device
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    return {n: _timed_cold(torch, ops[n], flush, iters) for n in names}


def context_rows(torch, d, scale, names, budget_s=150.0):
    """Context only, never a denominator: the same chains through the library's fused attention
    (scaled_dot_product_attention) and through torch.compile (default mode), timed like the eager baseline.
    A row that fails or would exceed the time budget is reported as null with the reason."""
    F = torch.nn.functional
    device = next(v for v in d.values() if hasattr(v, "device")).device
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    rows, t_start = {}, time.perf_counter()
    if "C5" in names:
        try:
            rows["C5_sdpa_ms"] = _timed_cold(
                torch, lambda: F.scaled_dot_product_attention(d["c5q"], d["c5k"], d["c5v"], is_causal=True, scale=scale),
                flush)
        except Exception as exc:       # noqa: BLE001 - a context row must never break the benchmark
            rows["C5_sdpa_ms"], rows["C5_sdpa_error"] = None, repr(exc)[:200]
    # What plain streaming kernels of the row kernels' sizes reach on this GPU, cold like them: a copy of C3's
    # activations (as many bytes as its LayerNorm reads and writes), torch's own LayerNorm on them, and an in-place
    # elementwise pass over an fp32 buffer of C4's logits' size (the bytes of the softmax finishing pass).
    try:
        if "C3" in names:
            x = d["c3x"]
            y = torch.empty_like(x)
            rows["C3_layernorm_copy_same_bytes_ms"] = _timed_cold(torch, lambda: y.copy_(x), flush, iters=5)
            rows["C3_layernorm_torch_ms"] = _timed_cold(
                torch, lambda: F.layer_norm(x, (x.shape[1],), d["c3g"], d["c3be"], 1e-5), flush, iters=5)
        if "C4" in names:
            z = torch.empty((d["c4x"].shape[0], d["c4w"].shape[1]), dtype=torch.float32, device=device)
            rows["C4_finish_inplace_same_bytes_ms"] = _timed_cold(torch, lambda: z.mul_(1.0009765625), flush, iters=5)
            del z
    except Exception as exc:           # noqa: BLE001
        rows["streaming_rows_error"] = repr(exc)[:200]
    ops = eager_ops(torch, d, scale)
    for n in ("C2", "C3", "C5"):
        if n not in names:
            continue
        if time.perf_counter() - t_start > budget_s:
            rows[f"{n}_compile_ms"], rows[f"{n}_compile_error"] = None, "time budget for context rows used up"
            continue
        try:
            fn = torch.compile(ops[n])
            rows[f"{n}_compile_ms"] = _timed_cold(torch, fn, flush)
        except Exception as exc:       # noqa: BLE001
            rows[f"{n}_compile_ms"], rows[f"{n}_compile_error"] = None, repr(exc)[:200]
    rows["seconds_spent"] = time.perf_counter() - t_start
    rows["note"] = ("C5_sdpa = torch scaled_dot_product_attention (is_causal); *_compile = torch.compile(default) of the eager "
                    "composition; *_same_bytes = a plain copy / in-place pass moving the bytes of that row kernel, cold")
    return rows


def library_gemm_context(torch, device, sampler, seconds=0.6):
    """Context only: the vendor library's plain bf16 GEMM (torch.matmul, 8192^3) run back to back for
    about `seconds` on this very GPU, with the clock it sustained - the box-specific counterpart of
    the measured peak.  Not a denominator of any reported fraction."""
    a = torch.randn(8192, 8192, device=device, dtype=torch.bfloat16)
    b = torch.randn(8192, 8192, device=device, dtype=torch.bfloat16)
    for _ in range(3):
        a @ b
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    a @ b
    e1.record()
    torch.cuda.synchronize()
    iters = max(10, int(seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))
    sampler.start()
    e0.record()
    for _ in range(iters):
        a @ b
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / iters
    return {"op": "torch.matmul bf16 8192^3", "tflops": 2 * 8192.0 ** 3 / (ms * 1e-3) / 1e12, "iters": iters,
            "sm_mhz": clocks.get("sm_mhz"), "power_w_max": clocks.get("power_w_max")}


def parity_spot_check(inputs, out):
    """A few rows of every timed output buffer against the oracle (same tolerances as the tests)."""
    from oracle import pike_oracle as O
    c1, c2, c3, c4, c5 = (inputs[k] for k in ALL)
    h = {k: v.detach().to("cpu").double().numpy() for k, v in out.items() if k != "C5"}
    res = {}
    w1 = O.linear_epilogue(c1["x"], c1["w"], c1["b"], None, c1["gamma"], c1["beta"], act="gelu_erf",
                           reduce="layernorm", eps=c1["eps"])
    e = np.abs(h["C1"] - w1).max()
    res["C1"] = {"max_abs_err": float(e), "ok": bool(e <= 1e-4)}

    def bf(got, want):
        err = np.abs(got - want)
        return {"max_abs_err": float(err.max()), "ok": bool((err <= 2e-2 + 2e-2 * np.abs(want)).all())}

    rows = np.array([0, 1000, 2047, 4095])
    res["C2"] = bf(h["C2"][rows], O.linear_epilogue(c2["x"], c2["w"], c2["b"], c2["r"], act="silu", scale=0.5, rows=rows))
    rows = np.array([0, 8191])
    res["C3"] = bf(h["C3"][rows], O.mlp_block(c3["x"], c3["gamma"], c3["beta"], c3["w1"], c3["b1"], c3["w2"], c3["b2"],
                                              act="gelu_tanh", eps=c3["eps"], rows=rows))
    rows = np.array([0, 2047])
    want = O.linear_epilogue(c4["x"], c4["w"], reduce="softmax", rows=rows)
    got = h["C4"][rows]
    r4 = bf(got, want)
    r4["max_rel_err"] = float((np.abs(got - want)[want >= 1e-7] / want[want >= 1e-7]).max())
    r4["ok"] = bool(r4["ok"] and r4["max_rel_err"] <= 1e-3 and np.abs(got.sum(1) - 1).max() <= 1e-5)
    res["C4"] = r4
    rows = np.array([0, 127, 128, 1500, 2047])
    got5 = out["C5"][7, 31].detach().to("cpu").double().numpy()[rows]
    res["C5"] = bf(got5, O.attention_head(c5["q"][7, 31], c5["k"][7, 31], c5["v"][7, 31], scale=c5["scale"],
                                          causal=True, rows=rows))
    res["all_ok"] = all(v["ok"] for v in res.values())
    return res


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--only", type=lambda v: tuple(x for x in ALL + EXTRA if x in v.split(",")), default=ALL,
                    help="comma-separated subset of C1..C5 and X1..X4 (profiling runs; the default is the whole suite C1..C5)")
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--sustained-seconds", type=float, default=2.0,
                    help="length of the sustained loop reported beside the K timed steps (0 = skip)")
    ap.add_argument("--no-eager", action="store_true")
    ap.add_argument("--no-context", action="store_true", help="skip the scaled_dot_product_attention / torch.compile rows")
    ap.add_argument("--no-extras", action="store_true", help="skip the further workloads X1..X4")
    ap.add_argument("--no-parity", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args(argv)
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    # the oracle pass is ~10-30 s of CPU work: bound the number of passes
    args.ref_steps = max(1, min(args.steps, 3))
    args.ref_warmup = 1 if args.warmup > 0 else 0
    return args


def main(argv=None):
    args = parse_args(argv)
    return run_reference(args) if args.impl == "reference" else run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
