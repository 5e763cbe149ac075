#!/usr/bin/env python
"""Benchmark of the FP8 hot path on B200.

One "step" is one pass of the whole hot path over one synthetic batch of a
transformer linear layer (hidden 4096 -> 16384, 8192 tokens): for each of the
activations X, weights W (E4M3) and output gradients dY (E5M2) the two-pass
current scaling  amax -> scale -> quantize, one dequantize (the FP8 -> bf16
round trip), then the three FP8 GEMMs with fp32 accumulation and bf16 output
with epilogue amax: forward Y = X.W, dgrad dX = dY.W^T, wgrad dW = X^T.dY.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is whole-job TFLOP/s: GEMM flops of all ranks
divided by the max-over-ranks device time of the K steps, casts included.
`--impl reference` times the CPU oracle (the slow checker under oracle/) on a
bounded sample of the same step instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fp8_linear_step_gemm_tflops"
UNIT = "TFLOP/s"
WORKLOAD = ("transformer linear layer fwd+bwd, hidden 4096->16384, 8192 tokens: amax+scale+quantize of X,W (E4M3) and dY (E5M2), "
            "one dequantize, fprop/dgrad/wgrad FP8 GEMMs, bf16 out + epilogue amax")
TOKENS, D_IN, D_OUT, W_SIGMA = 8192, 4096, 16384, 0.02
# DRAM bytes (read + write) per launch from the ncu captures summarised under profiles/ (same workload):
# forward GEMM 168.5 MB + 225.5 MB; one-launch conversion, mean of the X, W and dY launches.
NCU_TRAFFIC_GEMM_BYTES = 3.94e8
NCU_TRAFFIC_QUANTIZE_CURRENT_BYTES = 2.68e8
NOMINAL_FP8_TFLOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0


def peaks():
    """measured roofline denominators (generated file), else the documented fallback"""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    except Exception:
        return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------
# clocks sampling
# ----------------------------------------------------------------------------

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); smax.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        busy = [c for c, p in zip(sm, power) if p >= 0.5 * max(power)] or sm
        return {"sm_mhz": statistics.median(busy), "sm_max_mhz": max(smax), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# the step on the GPU
# ----------------------------------------------------------------------------

class LinearStep:
    """Buffers and call sequence of one step.  Everything the step computes runs in the library's kernels."""

    def __init__(self, torch, api, synth, device, seed, tokens=TOKENS, d_in=D_IN, d_out=D_OUT, fused_cast=True):
        self.torch, self.api = torch, api
        self.fused_cast = fused_cast
        self.T, self.I, self.O = tokens, d_in, d_out
        dev = device
        bf, u8, f32 = torch.bfloat16, torch.uint8, torch.float32
        self.X = synth.activations(tokens * d_in, seed, dtype=bf, device=dev).view(tokens, d_in)
        self.W = synth.weights(d_in * d_out, seed, W_SIGMA, dtype=bf, device=dev).view(d_in, d_out)
        self.dY = synth.gradients(tokens * d_out, seed + 1, dtype=bf, device=dev).view(tokens, d_out)
        self.Xq = torch.empty(tokens, d_in, dtype=u8, device=dev)
        self.Wq = torch.empty(d_in, d_out, dtype=u8, device=dev)
        self.dYq = torch.empty(tokens, d_out, dtype=u8, device=dev)
        self.Xhat = torch.empty(tokens, d_in, dtype=bf, device=dev)
        self.Y = torch.empty(tokens, d_out, dtype=bf, device=dev)
        self.dX = torch.empty(tokens, d_in, dtype=bf, device=dev)
        self.dW = torch.empty(d_in, d_out, dtype=bf, device=dev)
        self.scal = torch.zeros(16, dtype=f32, device=dev)      # amax / scale / scale_inv per tensor, GEMM amaxes
        s = [self.scal[i:i + 1] for i in range(16)]
        self.ax, self.sx, self.six, self.aw, self.sw, self.siw, self.ag, self.sg, self.sig = s[:9]
        self.ay, self.adx, self.adw = s[9:12]
        self.gemm_flops = 3 * 2.0 * tokens * d_in * d_out
        # algorithmic HBM bytes of the cast part: two-pass (read, read, write) = 5 B per bf16 element; dequantize 3 B
        n_cast = tokens * d_in + d_in * d_out + tokens * d_out
        self.cast_bytes = 5.0 * n_cast + 3.0 * tokens * d_in

    def calls(self):
        """(label, thunk) for every library call of one step, in order"""
        a = self.api
        E4, E5, KM, MN = a.E4M3, a.E5M2, a.MAJOR_K, a.MAJOR_MN
        if self.fused_cast:
            casts = [
                # amax -> scale -> quantize of one tensor in one cooperative launch
                ("quantize_current", lambda: a.fp8_quantize_current(self.X, E4, self.Xq, self.ax, self.sx, self.six)),
                ("quantize_current", lambda: a.fp8_quantize_current(self.W, E4, self.Wq, self.aw, self.sw, self.siw)),
                ("quantize_current", lambda: a.fp8_quantize_current(self.dY, E5, self.dYq, self.ag, self.sg, self.sig)),
            ]
        else:
            casts = [
                ("amax", lambda: a.fp8_amax(self.X, self.ax)),
                ("scale", lambda: a.fp8_scale_from_amax(self.ax, E4, self.sx, self.six)),
                ("quantize", lambda: a.fp8_quantize(self.X, E4, self.sx, self.Xq)),
                ("amax", lambda: a.fp8_amax(self.W, self.aw)),
                ("scale", lambda: a.fp8_scale_from_amax(self.aw, E4, self.sw, self.siw)),
                ("quantize", lambda: a.fp8_quantize(self.W, E4, self.sw, self.Wq)),
                ("amax", lambda: a.fp8_amax(self.dY, self.ag)),
                ("scale", lambda: a.fp8_scale_from_amax(self.ag, E5, self.sg, self.sig)),
                ("quantize", lambda: a.fp8_quantize(self.dY, E5, self.sg, self.dYq)),
            ]
        return casts + [
            ("dequantize", lambda: a.fp8_dequantize(self.Xq, E4, self.six, self.Xhat)),
            # forward: Y[T,O] = X[T,I] . W[I,O]   (W stored with the output index contiguous)
            ("gemm_fprop", lambda: a.fp8_gemm(self.Xq, E4, KM, self.Wq, E4, MN, self.Y, self.six, self.siw, self.ay)),
            # dgrad: dX[T,I] = dY[T,O] . W^T      (W stored [I,O] is the [N,K] layout here)
            ("gemm_dgrad", lambda: a.fp8_gemm(self.dYq, E5, KM, self.Wq, E4, KM, self.dX, self.sig, self.siw, self.adx)),
            # wgrad: dW[I,O] = X^T . dY           (both operands stored with the contraction index outermost)
            ("gemm_wgrad", lambda: a.fp8_gemm(self.Xq, E4, MN, self.dYq, E5, MN, self.dW, self.six, self.sig, self.adw)),
        ]

    def run(self, only=None):
        for label, f in self.calls():
            if only is None or label == only:
                f()

    def run_timed(self, events):
        """one step with a CUDA event before each call and one after the last"""
        torch = self.torch
        row = []
        for label, f in self.calls():
            e = torch.cuda.Event(enable_timing=True)
            e.record()
            row.append((label, e))
            f()
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        row.append(("end", e))
        events.append(row)


def bench_cast_sweep(torch, api, synth, device, log2n, iters=20):
    """config-2 style bandwidth point: bf16 tensors of 2^log2n elements; single-pass quantize+amax, amax, dequantize.
    Calls alternate between two distinct tensors, so that no call finds in L2 what the previous one left there
    (the two-pass kernel ends its second pass where its first pass starts)."""
    n = 1 << log2n
    xs = [synth.normal_laplace_mixture(n, 1 + k, synth.T_ID, device=device) for k in range(2)]
    codes = [torch.empty(n, dtype=torch.uint8, device=device) for _ in range(2)]
    backs = [torch.empty(n, dtype=torch.bfloat16, device=device) for _ in range(2)]
    sc = torch.tensor([3.0, 1.0 / 3.0, 0.0], dtype=torch.float32, device=device)
    s, si, a = sc[0:1], sc[1:2], sc[2:3]
    sc2 = torch.zeros(2, dtype=torch.float32, device=device)
    s2, si2 = sc2[0:1], sc2[1:2]
    out = {}
    cases = {
        "quantize_e4m3_with_amax": (lambda i: api.fp8_quantize(xs[i], api.E4M3, s, codes[i], api.SATURATE, a), 3.0 * n),
        "quantize_e5m2_with_amax": (lambda i: api.fp8_quantize(xs[i], api.E5M2, s, codes[i], api.SATURATE, a), 3.0 * n),
        "amax": (lambda i: api.fp8_amax(xs[i], a), 2.0 * n),
        "quantize_current_e4m3": (lambda i: api.fp8_quantize_current(xs[i], api.E4M3, codes[i], a, s2, si2), 5.0 * n),
        "dequantize_e4m3": (lambda i: api.fp8_dequantize(codes[i], api.E4M3, si, backs[i]), 3.0 * n),
        "fake_quantize_e4m3": (lambda i: api.fp8_fake_quantize(xs[i], api.E4M3, s, si, backs[i]), 4.0 * n),
    }
    for name, (fn, nbytes) in cases.items():
        for k in range(4):
            fn(k & 1)
        torch.cuda.synchronize()
        # `iters` calls back to back between two events: the tensors (0.5 GB each at 2^28) are far larger than L2,
        # and launch gaps overlap with the previous call's tail as they do inside a real step
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for k in range(iters):
            fn(k & 1)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        out[name] = {"ms": round(ms, 4), "gbs": round(nbytes / ms / 1e6, 1)}
    del xs, codes, backs
    torch.cuda.empty_cache()
    return out


def bench_cast_sizes(torch, api, synth, device, pk, sizes=(20, 24, 28, 30)):
    """The bandwidth sweep over tensor sizes (bf16, 2^20 .. 2^30 elements).  Each kernel is timed twice:
     - "same_buffer": 20 back-to-back calls on one tensor; below ~126 MB of traffic the tensor stays in L2, so the
       figure is flagged l2_resident and is a latency / L2 number, not an HBM one;
     - "ring": a CUDA graph of calls that walk a ring of distinct tensors totalling more than 512 MB, so that every
       call misses L2: the HBM-honest figure for the small sizes (and the launch cost without host gaps)."""
    out = {}
    sc = torch.tensor([3.0, 1.0 / 3.0, 0.0, 0.0, 0.0], dtype=torch.float32, device=device)
    s, si, a, s2, si2 = sc[0:1], sc[1:2], sc[2:3], sc[3:4], sc[4:5]
    for log2n in sizes:
        n = 1 << log2n
        ring = max(1, -(-(640 << 20) // (2 * n)))            # tensors of 2n bytes totalling >= 640 MB
        if log2n >= 30:
            ring = 1                                         # 2 GB already
        total = ring * n
        x = synth.normal_laplace_mixture(total, 1, synth.T_ID, device=device)
        codes = torch.empty(total, dtype=torch.uint8, device=device)
        back = torch.empty(total, dtype=torch.bfloat16, device=device)
        xs = [x[i * n:(i + 1) * n] for i in range(ring)]
        cs = [codes[i * n:(i + 1) * n] for i in range(ring)]
        bs = [back[i * n:(i + 1) * n] for i in range(ring)]
        cases = {
            "amax": (lambda i: api.fp8_amax(xs[i], a), 2.0 * n),
            "quantize_e4m3_with_amax": (lambda i: api.fp8_quantize(xs[i], api.E4M3, s, cs[i], api.SATURATE, a), 3.0 * n),
            "quantize_current_e4m3": (lambda i: api.fp8_quantize_current(xs[i], api.E4M3, cs[i], a, s2, si2), 5.0 * n),
            "dequantize_e4m3": (lambda i: api.fp8_dequantize(cs[i], api.E4M3, si, bs[i]), 3.0 * n),
        }
        row = {"ring_tensors": ring}
        for name, (fn, nbytes) in cases.items():
            for _ in range(3):
                fn(0)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(20):
                fn(0)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / 20
            entry = {"same_buffer": {"us": round(ms * 1e3, 2), "gbs": round(nbytes / ms / 1e6, 1), "l2_resident": bool(nbytes < (126 << 20))}}
            calls = max(ring, 8)
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                for i in range(min(ring, 3)):
                    fn(i)
                side.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=side):
                    for i in range(calls):
                        fn(i % ring)
            torch.cuda.current_stream().wait_stream(side)
            graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
            gms = e0.elapsed_time(e1) / calls
            entry["ring"] = {"us": round(gms * 1e3, 2), "gbs": round(nbytes / gms / 1e6, 1),
                             "frac_of_measured_hbm": round(nbytes / gms / 1e6 / pk["hbm_gbs"], 4), "calls_in_graph": calls}
            del graph
            row[name] = entry
        out["2pow%d" % log2n] = row
        del x, codes, back, xs, cs, bs
        torch.cuda.empty_cache()
    return out


def bench_config(torch, api, synth, device, pk, which):
    """One of the five named workloads, every call timed alone (20 back-to-back launches after a short idle):
    1 = 256 x 256 fp32 tensors, casts and a 256^3 GEMM (latency-bound); 2 = the cast size sweep; 3 = hidden-4096
    forward (casts of X and W, forward GEMM); 4 = hidden-4096 backward (cast of dY, dgrad, wgrad); 5 = the
    175B-class FFN, hidden 12288 (casts of X, W, dY; forward and dgrad GEMMs)."""
    if which == 2:
        return bench_cast_sizes(torch, api, synth, device, pk)

    def timed(fn, n=20):
        torch.cuda.synchronize()
        time.sleep(0.25)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    bf, f32, u8 = torch.bfloat16, torch.float32, torch.uint8
    E4, E5, KM, MN = api.E4M3, api.E5M2, api.MAJOR_K, api.MAJOR_MN
    out = {}

    def cast(name, x, fmt):
        q = torch.empty(x.shape, dtype=u8, device=device)
        s = torch.zeros(3, dtype=f32, device=device)
        esz = x.element_size()
        ms = timed(lambda: api.fp8_quantize_current(x, fmt, q, s[0:1], s[1:2], s[2:3]))
        nbytes = (2 * esz + 1.0) * x.numel()
        out["quantize_current_" + name] = {"ms": round(ms, 4), "gbs": round(nbytes / ms / 1e6, 1),
                                           "frac_of_measured_hbm": round(nbytes / ms / 1e6 / pk["hbm_gbs"], 4)}
        return q, s[2:3]

    def gemm(name, A, fa, ma, B, fb, mb, M, N, K, si_a, si_b, dtype=bf, n=20):
        D = torch.empty(M, N, dtype=dtype, device=device)
        am = torch.zeros(1, dtype=f32, device=device)
        ms = timed(lambda: api.fp8_gemm(A, fa, ma, B, fb, mb, D, si_a, si_b, am), n)
        tf = 2.0 * M * N * K / ms / 1e9
        out["gemm_" + name] = {"ms": round(ms, 4), "tflops": round(tf, 1), "frac_of_2x_measured_bf16_burst": round(tf / (2 * pk["bf16_burst"]), 4),
                               "frac_of_nominal_4500": round(tf / 4500.0, 4)}

    if which == 1:
        A = synth.normal_with_scaled_outliers(256 * 256, 0, synth.A_ID, 0.005, 64.0, dtype=f32, device=device).view(256, 256)
        B = synth.normal_with_scaled_outliers(256 * 256, 0, synth.B_ID, 0.005, 64.0, dtype=f32, device=device).view(256, 256)
        Aq, sia = cast("A_256x256_fp32", A, E4)
        Bq, sib = cast("B_256x256_fp32", B, E4)
        gemm("256x256x256_fp32_out", Aq, E4, KM, Bq, E4, KM, 256, 256, 256, sia, sib, dtype=f32)
    elif which in (3, 4):
        T, I, O = TOKENS, D_IN, D_OUT
        X = synth.activations(T * I, 3, device=device).view(T, I)
        W = synth.weights(I * O, 3, W_SIGMA, device=device).view(I, O)
        Xq, six = cast("X_8192x4096", X, E4)
        Wq, siw = cast("W_4096x16384", W, E4)
        del X, W
        if which == 3:
            gemm("fprop_8192x16384x4096", Xq, E4, KM, Wq, E4, MN, T, O, I, six, siw)
        else:
            dY = synth.gradients(T * O, 4, device=device).view(T, O)
            Gq, sig = cast("dY_8192x16384", dY, E5)
            del dY
            gemm("dgrad_8192x4096x16384", Gq, E5, KM, Wq, E4, KM, T, I, O, sig, siw)
            gemm("wgrad_4096x16384x8192", Xq, E4, MN, Gq, E5, MN, I, O, T, six, sig)
    elif which == 5:
        T, I, O = 8192, 12288, 49152
        X = synth.activations(T * I, 5, device=device).view(T, I)
        Xq, six = cast("X_8192x12288", X, E4)
        del X
        W = synth.weights(I * O, 5, 0.006, device=device).view(I, O)
        Wq, siw = cast("W_12288x49152", W, E4)
        del W
        dY = synth.gradients(T * O, 5, device=device).view(T, O)
        Gq, sig = cast("dY_8192x49152", dY, E5)
        del dY
        torch.cuda.empty_cache()
        gemm("fprop_8192x49152x12288", Xq, E4, KM, Wq, E4, MN, T, O, I, six, siw, n=5)
        gemm("dgrad_8192x12288x49152", Gq, E5, KM, Wq, E4, KM, T, I, O, sig, siw, n=5)
    else:
        raise SystemExit("--config takes 1..5")
    return out


def bench_gemm_alone(torch, step, seconds=2.0):
    """The forward GEMM of the step by itself: best single launch (burst) and a back-to-back loop of at
    least `seconds` (sustained, under the power cap)."""
    call = dict(step.calls())["gemm_fprop"]
    flops = 2.0 * step.T * step.I * step.O
    for _ in range(3):
        call()
    torch.cuda.synchronize()
    best = 1e9
    for _ in range(10):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(); call(); e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    n = max(10, int(seconds * 1e3 / best))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(n):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    return {"shape": "M=%d N=%d K=%d, E4M3 x E4M3 -> bf16" % (step.T, step.O, step.I),
            "burst_tflops": round(flops / best / 1e9, 1), "sustained_tflops": round(flops / ms / 1e9, 1),
            "sustained_launches": n, "sustained_seconds": round(ms * n / 1e3, 2)}


def bench_next_rows(torch, api, synth, device, pk, iters=5):
    """The rows beyond the core path, each timed alone on workload-shaped tensors: simulated-FP8 round trip,
    per-channel weight scales, FP8-output GEMM, attention-style batched GEMM."""
    def timed(fn):
        """mean of `iters` groups of 4 back-to-back calls (launch gaps overlap the previous call, as inside a step);
        a short idle first, so that each kernel is timed alone and not in the power state its predecessor left"""
        torch.cuda.synchronize()
        time.sleep(0.25)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(4 * iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / (4 * iters)

    out = {}
    f32 = torch.float32
    sc = torch.tensor([3.0, 1.0 / 3.0, 0.0, 0.0], dtype=f32, device=device)
    s, si, a = sc[0:1], sc[1:2], sc[2:3]
    # simulated FP8 (quantize + dequantize in one pass), 2^28 bf16 elements: 4 B per element
    n = 1 << 28
    x = synth.normal_laplace_mixture(n, 1, synth.T_ID, device=device)
    y = torch.empty_like(x)
    ms = timed(lambda: api.fp8_fake_quantize(x, api.E4M3, s, si, y))
    out["fake_quantize_e4m3_2pow28"] = {"ms": round(ms, 4), "gbs": round(4.0 * n / ms / 1e6, 1), "frac_of_measured_hbm": round(4.0 * n / ms / 1e6 / pk["hbm_gbs"], 4)}
    del x, y
    # per-channel weight scales on W [4096 x 16384] bf16, one channel per output column
    W = synth.weights(D_IN * D_OUT, 3, W_SIGMA, device=device).view(D_IN, D_OUT)
    am = torch.empty(D_OUT, dtype=f32, device=device)
    sv, siv = torch.empty(D_OUT, dtype=f32, device=device), torch.empty(D_OUT, dtype=f32, device=device)
    Wq = torch.empty(D_IN, D_OUT, dtype=torch.uint8, device=device)
    nW = D_IN * D_OUT
    ms = timed(lambda: api.fp8_amax_channels(W, 0, am))
    out["amax_channels_cols_W"] = {"ms": round(ms, 4), "gbs": round(2.0 * nW / ms / 1e6, 1), "frac_of_measured_hbm": round(2.0 * nW / ms / 1e6 / pk["hbm_gbs"], 4)}
    api.fp8_scales_from_amax(am, api.E4M3, sv, siv)
    ms = timed(lambda: api.fp8_quantize_channels(W, 0, api.E4M3, sv, Wq))
    out["quantize_channels_cols_W"] = {"ms": round(ms, 4), "gbs": round(3.0 * nW / ms / 1e6, 1), "frac_of_measured_hbm": round(3.0 * nW / ms / 1e6 / pk["hbm_gbs"], 4)}
    # codes in both orientations from one pass (4 B per bf16 element): dY-shaped [8192 x 16384] and X-shaped [8192 x 4096]
    for name, (r_, c_) in (("quantize_transpose_dY_8192x16384", (TOKENS, D_OUT)), ("quantize_transpose_X_8192x4096", (TOKENS, D_IN))):
        xt = synth.gradients(r_ * c_, 4, device=device).view(r_, c_)
        o1 = torch.empty(r_, c_, dtype=torch.uint8, device=device)
        o2 = torch.empty(c_, r_, dtype=torch.uint8, device=device)
        ms = timed(lambda: api.fp8_quantize_transpose(xt, api.E5M2, s, o1, o2, a))
        out[name] = {"ms": round(ms, 4), "gbs": round(4.0 * r_ * c_ / ms / 1e6, 1), "frac_of_measured_hbm": round(4.0 * r_ * c_ / ms / 1e6 / pk["hbm_gbs"], 4)}
        del xt, o1, o2
    # forward GEMM with per-channel weight scales, and with FP8 (E4M3) output
    X = synth.activations(TOKENS * D_IN, 3, device=device).view(TOKENS, D_IN)
    Xq = torch.empty(TOKENS, D_IN, dtype=torch.uint8, device=device)
    sx = torch.zeros(3, dtype=f32, device=device)
    api.fp8_quantize_current(X, api.E4M3, Xq, sx[0:1], sx[1:2], sx[2:3])
    Y = torch.empty(TOKENS, D_OUT, dtype=torch.bfloat16, device=device)
    Yq = torch.empty(TOKENS, D_OUT, dtype=torch.uint8, device=device)
    flops = 2.0 * TOKENS * D_IN * D_OUT
    ms = timed(lambda: api.fp8_gemm_channel_scales(Xq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_MN, Y, sx[2:3], siv, a))
    out["gemm_fprop_channel_scales"] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1)}
    ms = timed(lambda: api.fp8_gemm_fp8out(Xq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_MN, Yq, api.E4M3, sx[2:3], si, s, a))
    out["gemm_fprop_fp8_output"] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1)}
    # split accumulation (partial sums every 2048 of K added in registers): forward K = 4096 and, on the same codes
    # read as dY-shaped operands, the dgrad shape K = 16384
    ms = timed(lambda: api.fp8_gemm(Xq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_MN, Y, sx[2:3], si, a, acc=api.ACC_SPLIT))
    out["gemm_fprop_split_accumulation"] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1)}
    dX = torch.empty(TOKENS, D_IN, dtype=torch.bfloat16, device=device)
    ms = timed(lambda: api.fp8_gemm(Yq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_K, dX, si, si, a, acc=api.ACC_SPLIT))
    out["gemm_dgrad_split_accumulation"] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1)}
    ms = timed(lambda: api.fp8_gemm(Yq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_K, dX, si, si, a))
    out["gemm_dgrad_same_codes_one_accumulator"] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1)}
    del dX
    del W, X, Y, Yq
    # a weight-bandwidth-bound product with few output tiles: 16 rows against W^T stored [4096 x 16384] (K = 16384),
    # plain and with the contraction cut into slices
    Xs = torch.randint(0, 0x78, (16, D_OUT), dtype=torch.uint8, device=device)
    Wt = torch.randint(0, 0x78, (D_IN, D_OUT), dtype=torch.uint8, device=device)          # [N = 4096, K = 16384], K-major
    Ys = torch.empty(16, D_IN, dtype=torch.bfloat16, device=device)
    sp, nb = api.fp8_gemm_splitk_workspace(16, D_IN, D_OUT)
    ws = torch.empty(max(nb // 4, 4), dtype=f32, device=device)
    ms = timed(lambda: api.fp8_gemm(Xs, api.E4M3, api.MAJOR_K, Wt, api.E4M3, api.MAJOR_K, Ys, si, si, a))
    out["gemm_16x4096x16384_one_launch"] = {"ms": round(ms, 4), "weight_gbs": round(D_IN * D_OUT / ms / 1e6, 1)}
    ms = timed(lambda: api.fp8_gemm_splitk(Xs, api.E4M3, api.MAJOR_K, Wt, api.E4M3, api.MAJOR_K, Ys, si, si, ws if nb else None, a))
    out["gemm_16x4096x16384_splitk"] = {"ms": round(ms, 4), "weight_gbs": round(D_IN * D_OUT / ms / 1e6, 1), "splits": sp}
    del Xs, Wt, Ys, ws
    # attention-style batched products: 32 heads, 4096 tokens, head dim 128: scores = Q.K^T, context = P.V
    H, S, Dh = 32, 4096, 128
    Q = torch.randint(0, 0x78, (H, S, Dh), dtype=torch.uint8, device=device)
    Kt = torch.randint(0, 0x78, (H, S, Dh), dtype=torch.uint8, device=device)
    P = torch.empty(H, S, S, dtype=torch.bfloat16, device=device)
    ms = timed(lambda: api.fp8_gemm_batched(Q, api.E4M3, api.MAJOR_K, Kt, api.E4M3, api.MAJOR_K, P, si, si, a))
    fl = 2.0 * H * S * S * Dh
    out["batched_scores_32x4096x4096x128"] = {"ms": round(ms, 4), "tflops": round(fl / ms / 1e9, 1),
                                              "output_gbs": round(2.0 * H * S * S / ms / 1e6, 1), "bound": "hbm (bf16 output, K = 128)"}
    Pq = torch.randint(0, 0x78, (H, S, S), dtype=torch.uint8, device=device)
    C = torch.empty(H, S, Dh, dtype=torch.bfloat16, device=device)
    ms = timed(lambda: api.fp8_gemm_batched(Pq, api.E4M3, api.MAJOR_K, Kt, api.E4M3, api.MAJOR_MN, C, si, si, a))
    out["batched_context_32x4096x128x4096"] = {"ms": round(ms, 4), "tflops": round(fl / ms / 1e9, 1)}
    del Q, Kt, P, Pq, C
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------
# the oracle arm (CPU)
# ----------------------------------------------------------------------------

_oracle_inputs = {}


def oracle_step(sample_tokens: int, threads: int, sample_out: int = D_OUT):
    """The same step on a bounded sample of the layer: `sample_tokens` tokens and `sample_out` output features
    (W is [d_in, sample_out], same recipe), run by the CPU oracle as it stands.
    Returns (seconds, gemm flops of the sample)."""
    import numpy as np
    import torch

    import oracle
    from paper_2209_05433_b200 import synth

    T, I, O = sample_tokens, D_IN, sample_out

    def bits(t):
        return t.view(torch.int16).numpy().view(np.uint16)

    key = (T, O)
    if key not in _oracle_inputs:                                  # synthetic inputs are made once, outside the timed part
        _oracle_inputs.clear()
        _oracle_inputs[key] = (bits(synth.activations(T * I, 3, dtype=torch.bfloat16)),
                               bits(synth.weights(I * O, 3, W_SIGMA, dtype=torch.bfloat16)),
                               bits(synth.gradients(T * O, 4, dtype=torch.bfloat16)))
    X, W, dY = _oracle_inputs[key]
    t0 = time.perf_counter()
    q, sinv = {}, {}
    for name, t, fmt in (("x", X, oracle.E4M3), ("w", W, oracle.E4M3), ("g", dY, oracle.E5M2)):
        s, si = oracle.scale_from_amax(oracle.amax(t, threads), fmt)
        q[name], sinv[name] = oracle.quantize(t, s, fmt, threads=threads), si
    oracle.dequantize(q["x"], sinv["x"], oracle.E4M3, "bf16", threads=threads)
    y, _ = oracle.gemm_rows(q["x"], oracle.E4M3, (I, 1), q["w"], oracle.E4M3, (O, 1), O, I, 0, T, sinv["x"], sinv["w"], threads)
    dx, _ = oracle.gemm_rows(q["g"], oracle.E5M2, (O, 1), q["w"], oracle.E4M3, (1, O), I, O, 0, T, sinv["g"], sinv["w"], threads)
    dw, _ = oracle.gemm_rows(q["x"], oracle.E4M3, (1, I), q["g"], oracle.E5M2, (O, 1), O, T, 0, I, sinv["x"], sinv["g"], threads)
    for r in (y, dx, dw):
        oracle.round_bf16_from_f64(r)
    dt = time.perf_counter() - t0
    return dt, 3 * 2.0 * T * I * O


def reference_sample(steps: int, warmup: int, threads: int):
    """(tokens, output features) of the per-step sample: 8 tokens and as many output features (multiples of
    256) as fit about 150 s for the whole run, at most the full layer (about 6 s per step on 8 cores).
    Every cost of the step (weight cast, three GEMMs, wgrad outputs) is linear in the feature count."""
    t_small, _ = oracle_step(8, threads, 256)                      # calibration on the smallest sample
    total = float(os.environ.get("FP8_BENCH_REFERENCE_SECONDS", "150"))      # wall-clock aim for the whole run
    budget = min(8.0, total / max(1, steps + warmup))
    grow = max(1.0, budget / max(t_small, 1e-3))
    sample_out = int(min(D_OUT, 256 * int(grow)))
    return 8, max(256, sample_out // 256 * 256)


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = os.cpu_count() or 1
    sample_tokens, sample_out = reference_sample(args.steps, args.warmup, threads)
    for _ in range(args.warmup):
        oracle_step(sample_tokens, threads, sample_out)
    times, flops = [], 0.0
    for _ in range(args.steps):
        dt, flops = oracle_step(sample_tokens, threads, sample_out)
        times.append(dt)
    total = sum(times)
    value = flops * len(times) / total / 1e12
    sample = "the same step on %d of the %d tokens and %d of the %d output features, CPU oracle as it stands" % (
        sample_tokens, TOKENS, sample_out, D_OUT)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 accumulation over decoded fp8 codes", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2209_05433_b200 import api, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    device = "cuda:%d" % local
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(device))
    api.load()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    if args.cast_sizes_only:
        print(json.dumps({"cast_sizes": bench_cast_sizes(torch, api, synth, device, peaks())}))
        return
    if args.config:
        print(json.dumps({"config": args.config, "results": bench_config(torch, api, synth, device, peaks(), args.config)}))
        return
    if args.next_rows_only:
        # profiling aid: only the kernels beyond the core path, each on workload-shaped tensors
        print(json.dumps({"next_rows": bench_next_rows(torch, api, synth, device, peaks(), iters=max(1, min(args.steps, 5)))}))
        return
    # independent batches per rank: no data-path collective (per-tensor amax is local to a rank's own tensors)
    step = LinearStep(torch, api, synth, device, seed=3 + 16 * rank, fused_cast=not args.unfused_cast)
    if args.only:
        # profiling aid: one full step to set the scales and codes, then only the named call, timed alone
        step.run()
        for _ in range(max(args.warmup, 1)):
            step.run(args.only)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            step.run(args.only)
        e1.record()
        torch.cuda.synchronize()
        print(json.dumps({"only": args.only, "steps": args.steps, "ms_per_step": e0.elapsed_time(e1) / args.steps}))
        return
    for _ in range(max(args.warmup, 3)):
        step.run()
    barrier()
    st, detail = api.fp8_async_status()
    if st != 0:
        raise SystemExit("device-side wait expired during warm-up (code %d)" % detail)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = api.fp8_launch_count()
    events = []
    barrier()
    for _ in range(args.steps):
        step.run_timed(events)
    barrier()
    launches = api.fp8_launch_count() - launches0
    total_ms = events[0][0][1].elapsed_time(events[-1][-1][1])
    per_label = {}
    for row in events:
        for (label, e0), (_, e1) in zip(row[:-1], row[1:]):
            per_label.setdefault(label, []).append(e0.elapsed_time(e1))
    if world > 1:
        t = torch.tensor([total_ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms = float(t.item())
    clocks = sampler.stop() if rank == 0 else None
    st, detail = api.fp8_async_status()
    if st != 0:
        raise SystemExit("device-side wait expired during the timed region (code %d)" % detail)

    # ---- end to end: pinned host inputs -> device, the step, results -> pinned host, EVERY step.
    # Three streams (copy in, compute, copy out) and two device buffer sets, so that the upload of step i+1 and
    # the download of step i-1 overlap the kernels of step i; each step still moves all of its own bytes.
    steps2 = [step, LinearStep(torch, api, synth, device, seed=3 + 16 * rank, fused_cast=not args.unfused_cast)]
    host_in = [torch.empty(t.shape, dtype=t.dtype).pin_memory().copy_(t) for t in (step.X, step.W, step.dY)]
    host_out = [[torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (st.Y, st.dX, st.dW)] for st in steps2]
    host_scal = [torch.empty(16, dtype=torch.float32).pin_memory() for _ in steps2]
    h2d = sum(t.numel() * t.element_size() for t in host_in)
    d2h = sum(t.numel() * t.element_size() for t in host_out[0]) + host_scal[0].numel() * 4
    s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    for s_ in (s_in, s_comp, s_out):
        s_.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s_comp):
        api.current_scaling_workspace(torch.device(device))          # workspace of the compute stream
    ev_in = [torch.cuda.Event() for _ in steps2]        # inputs of buffer set b are on the device
    ev_comp = [torch.cuda.Event() for _ in steps2]      # kernels of buffer set b are done
    ev_out = [torch.cuda.Event() for _ in steps2]       # outputs of buffer set b are on the host

    def e2e_step(i):
        b = i & 1
        st = steps2[b]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_comp[b])                  # the previous step on this set has consumed its inputs
            for h, d in zip(host_in, (st.X, st.W, st.dY)):
                d.copy_(h, non_blocking=True)
            ev_in[b].record(s_in)
        with torch.cuda.stream(s_comp):
            s_comp.wait_event(ev_in[b])
            s_comp.wait_event(ev_out[b])                 # its previous outputs have left the device buffers
            st.run()
            ev_comp[b].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[b])
            for h, d in zip(host_out[b], (st.Y, st.dX, st.dW)):
                h.copy_(d, non_blocking=True)
            host_scal[b].copy_(st.scal, non_blocking=True)
            ev_out[b].record(s_out)

    e2e_steps = max(2, min(args.steps, 10))
    for i in range(2):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(s_in)
    for i in range(e2e_steps):
        e2e_step(i)
    s_out.wait_stream(s_comp)
    s_out.wait_stream(s_in)
    e1.record(s_out)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([e2e_ms], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())

    if rank == 0:
        pk = peaks()
        ms_per_step = total_ms / args.steps
        value = step.gemm_flops * world / (ms_per_step * 1e-3) / 1e12
        avg = {k: sum(v) / len(v) for k, v in per_label.items()}
        calls_per_step = {k: len(v) // args.steps for k, v in per_label.items()}
        step_sum = sum(avg[k] * calls_per_step[k] for k in avg)
        kernels = {k: {"avg_ms": round(avg[k], 4), "calls_per_step": calls_per_step[k],
                       "share": round(avg[k] * calls_per_step[k] / step_sum, 4)} for k in avg}
        # dominant kernel: the FP8 GEMM (three launches per step of 2*T*I*O flops each)
        gemm_ms = (avg["gemm_fprop"] + avg["gemm_dgrad"] + avg["gemm_wgrad"]) / 3.0
        gemm_flops = 2.0 * TOKENS * D_IN * D_OUT
        achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12
        fp8_peak = 2.0 * pk["bf16_sustained"]            # fp8 : bf16 nominal ratio is 2
        roofline = {"bound": "tensor", "kernel": "k_gemm_fp8", "achieved": round(achieved, 1), "peak": round(fp8_peak, 1),
                    "unit": "TFLOP/s", "frac": round(achieved / fp8_peak, 4), "traffic": NCU_TRAFFIC_GEMM_BYTES,
                    "traffic_note": "DRAM bytes per launch, ncu capture of the forward GEMM (profiles/gemm_fp8_forward_hidden4096.md); algorithmic 3.69e8",
                    "peak_source": "2 x %s bf16 sustained cuBLAS TFLOP/s (fp8:bf16 nominal ratio)" % pk["source"],
                    "frac_of_nominal_4500": round(achieved / NOMINAL_FP8_TFLOPS, 4),
                    "per_gemm_tflops": {k: round(gemm_flops / (avg[k] * 1e-3) / 1e12, 1) for k in ("gemm_fprop", "gemm_dgrad", "gemm_wgrad")}}
        # the memory-bound half: amax + quantize (+ dequantize) of the step against HBM
        cast_labels = [k for k in ("quantize_current", "amax", "scale", "quantize", "dequantize") if k in avg]
        cast_ms = sum(avg[k] * calls_per_step[k] for k in cast_labels)
        cast_gbs = step.cast_bytes / (cast_ms * 1e-3) / 1e9
        n_x = TOKENS * D_IN + D_IN * D_OUT + TOKENS * D_OUT
        roofline_cast = {"bound": "hbm", "kernel": "casts of the step: " + " + ".join(cast_labels), "achieved": round(cast_gbs, 1),
                         "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": round(cast_gbs / pk["hbm_gbs"], 4),
                         "traffic": NCU_TRAFFIC_QUANTIZE_CURRENT_BYTES if "quantize_current" in avg else None,
                         "peak_source": pk["source"] + " copy bandwidth", "frac_of_nominal_8000": round(cast_gbs / NOMINAL_HBM_GBS, 4),
                         "algorithmic_bytes": "5 B per bf16 element for amax+quantize (two reads, one write), 3 B per element for dequantize; "
                                              "re-reads served by L2 still count as algorithmic bytes"}
        if "quantize_current" in avg:
            roofline_cast["quantize_current_gbs"] = round(5.0 * n_x / 3 / (avg["quantize_current"] * 1e-3) / 1e9, 1)
        else:
            roofline_cast["amax_gbs"] = round(2.0 * n_x / 3 / (avg["amax"] * 1e-3) / 1e9, 1)
            roofline_cast["quantize_gbs"] = round(3.0 * n_x / 3 / (avg["quantize"] * 1e-3) / 1e9, 1)
        cast = None
        if not args.no_cast_sweep:
            cast = bench_cast_sweep(torch, api, synth, device, args.cast_log2n)
            for v in cast.values():
                v["frac_of_measured_hbm"] = round(v["gbs"] / pk["hbm_gbs"], 4)
        cast_sizes = bench_cast_sizes(torch, api, synth, device, pk) if world == 1 and not args.no_cast_sweep else None
        gemm_alone = bench_gemm_alone(torch, step) if world == 1 and not args.no_next_rows else None
        next_rows = None
        if world == 1 and not args.no_next_rows:
            next_rows = bench_next_rows(torch, api, synth, device, pk)
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            threads = os.cpu_count() or 1
            cpu_tokens = 24                     # about 10-20 s of CPU work on 16 cores
            dt, flops = oracle_step(cpu_tokens, threads)
            cpu = {"value": flops / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": round(dt, 2),
                   "sample": "the same step with %d of the %d tokens (weights at full size), CPU oracle as it stands" % (cpu_tokens, TOKENS)}
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp8 (e4m3/e5m2) operands, f32 accumulate, bf16 out", "data": "synthetic",
            "config": {"workload": WORKLOAD, "tokens": TOKENS, "d_in": D_IN, "d_out": D_OUT, "parallelism": "dp%d" % world,
                       "l2": "inputs larger than L2 (step touches > 1 GB)", "weights_layout": "[d_in, d_out] row-major"},
            "clocks": clocks,
            "e2e": {"value": step.gemm_flops * world / (e2e_ms / e2e_steps * 1e-3) / 1e12, "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
                    "how": "pinned host buffers; upload, kernels and download of consecutive steps overlap on three streams"},
            "gpu_launches": int(launches), "gpu_launches_note": "kernels plus 4-byte memset nodes enqueued by the library in the timed region",
            "roofline": roofline, "roofline_cast": roofline_cast, "kernels": kernels, "cast_sweep_2pow%d" % args.cast_log2n: cast,
            "cast_sizes": cast_sizes,
            "gemm_alone": gemm_alone,
            "next_rows": next_rows,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-cast-sweep", action="store_true")
    ap.add_argument("--no-next-rows", action="store_true")
    ap.add_argument("--config", type=int, default=0, help="run one of the five named workloads (1..5), every call timed alone")
    ap.add_argument("--cast-sizes-only", action="store_true", help="only the cast bandwidth sweep over 2^20 .. 2^30 elements")
    ap.add_argument("--next-rows-only", action="store_true", help="profiling aid: run only the next-row kernels")
    ap.add_argument("--cast-log2n", type=int, default=28)
    ap.add_argument("--unfused-cast", action="store_true", help="amax, scale and quantize as three calls per tensor instead of fp8_quantize_current")
    ap.add_argument("--only", default=None, help="profiling aid: time only the calls with this label (e.g. gemm_fprop, quantize, amax)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
