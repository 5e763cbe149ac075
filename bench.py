#!/usr/bin/env python
"""Benchmark of the FP8 hot path on B200.

One "step" is one pass of the whole hot path over one synthetic batch of the largest workload,
the 175B-class FFN layer (hidden 12288 -> 49152, 8192 tokens): for each of the activations X,
weights W (E4M3) and output gradients dY (E5M2) the two-pass current scaling
amax -> scale -> quantize, one dequantize (the FP8 -> bf16 round trip), then the FP8 GEMMs with
fp32 accumulation and bf16 output with epilogue amax: forward Y = X.W and dgrad dX = dY.W^T.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line.  `value` is whole-job TFLOP/s: GEMM flops of all ranks divided by the
max-over-ranks device time of the K steps, casts included.  With --gpus N > 1 and no torchrun
environment the script starts its N ranks itself (one process per GPU).  `--impl reference`
times the CPU oracle (the slow checker under oracle/) on a bounded sample of the same step.

Two regimes are reported and labelled: the K timed steps (a fraction of a second: the GPU is
still at boost clocks, "burst") and a loop of whole steps lasting at least two seconds under
the power cap ("sustained").  Roofline fractions divide burst figures by the burst peak and
sustained figures by the sustained peak.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
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
NOMINAL_FP8_TFLOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0
FP8_MACS_PER_SM_PER_CLOCK = 8192           # dense 8-bit multiply-adds one SM's tensor pipe retires per clock

# (tokens, d_in, d_out, sigma of the weights, seed, GEMM passes) of the layer workloads
LAYERS = {
    "hidden4096": dict(tokens=8192, d_in=4096, d_out=16384, w_sigma=0.02, seed=3, passes=("fprop", "dgrad", "wgrad")),
    "hidden12288": dict(tokens=8192, d_in=12288, d_out=49152, w_sigma=0.006, seed=5, passes=("fprop", "dgrad")),
}
HEADLINE = "hidden12288"


def workload_text(layer):
    L = LAYERS[layer]
    return ("transformer FFN linear layer, hidden %d->%d, %d tokens: amax+scale+quantize of X, W (E4M3) and dY (E5M2), "
            "one dequantize, %s FP8 GEMMs, bf16 out + epilogue amax" % (L["d_in"], L["d_out"], L["tokens"], "/".join(L["passes"])))


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


def ncu_traffic():
    """DRAM bytes per launch (read + write) of the profiled kernels, from the table the ncu summaries keep:
    lines of `name  bytes  ...`; a name missing from the table gives None."""
    table = {}
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 2 and not line.startswith("#"):
                    table[parts[0]] = float(parts[1])
    except OSError:
        pass
    return table


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
                "samples": len(sm), "samples_under_load": len(busy), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------
# the step on the GPU
# ----------------------------------------------------------------------------

class LinearStep:
    """Buffers and call sequence of one step.  Everything the step computes runs in the library's kernels."""

    def __init__(self, torch, api, synth, device, layer, seed_offset=0, acc=None):
        L = LAYERS[layer]
        self.acc = api.ACC_SPLIT if acc is None else acc          # accumulation mode of the GEMMs (library default)
        self.torch, self.api, self.layer = torch, api, layer
        self.T, self.I, self.O, self.passes = L["tokens"], L["d_in"], L["d_out"], L["passes"]
        T, I, O, seed = self.T, self.I, self.O, L["seed"] + seed_offset
        bf, u8, f32 = torch.bfloat16, torch.uint8, torch.float32
        self.X = synth.activations(T * I, seed, dtype=bf, device=device).view(T, I)
        self.W = synth.weights(I * O, seed, L["w_sigma"], dtype=bf, device=device).view(I, O)
        self.dY = synth.gradients(T * O, seed + (1 if layer == "hidden4096" else 0), dtype=bf, device=device).view(T, O)
        self.Xq = torch.empty(T, I, dtype=u8, device=device)
        self.Wq = torch.empty(I, O, dtype=u8, device=device)
        self.dYq = torch.empty(T, O, dtype=u8, device=device)
        self.Xhat = torch.empty(T, I, dtype=bf, device=device)
        self.Y = torch.empty(T, O, dtype=bf, device=device) if "fprop" in self.passes else None
        self.dX = torch.empty(T, I, dtype=bf, device=device) if "dgrad" in self.passes else None
        self.dW = torch.empty(I, O, dtype=bf, device=device) if "wgrad" in self.passes else None
        self.scal = torch.zeros(16, dtype=f32, device=device)      # amax / scale / scale_inv per tensor, GEMM amaxes
        s = [self.scal[i:i + 1] for i in range(16)]
        self.ax, self.sx, self.six, self.aw, self.sw, self.siw, self.ag, self.sg, self.sig = s[:9]
        self.ay, self.adx, self.adw = s[9:12]
        self.flops_per_gemm = 2.0 * T * I * O
        self.gemm_flops = len(self.passes) * self.flops_per_gemm
        # algorithmic HBM bytes of the cast part: two-pass (read, read, write) = 5 B per bf16 element; dequantize 3 B
        self.n_cast = T * I + I * O + T * O
        self.cast_bytes = 5.0 * self.n_cast + 3.0 * T * I
        self.inputs = (self.X, self.W, self.dY)
        self.outputs = tuple(t for t in (self.Y, self.dX, self.dW) if t is not None)

    def calls(self):
        """(label, thunk) for every library call of one step, in order"""
        a = self.api
        E4, E5, KM, MN = a.E4M3, a.E5M2, a.MAJOR_K, a.MAJOR_MN
        calls = [
            # amax -> scale -> quantize of one tensor in one cooperative launch
            ("quantize_current_X", lambda: a.fp8_quantize_current(self.X, E4, self.Xq, self.ax, self.sx, self.six)),
            ("quantize_current_W", lambda: a.fp8_quantize_current(self.W, E4, self.Wq, self.aw, self.sw, self.siw)),
            ("quantize_current_dY", lambda: a.fp8_quantize_current(self.dY, E5, self.dYq, self.ag, self.sg, self.sig)),
            ("dequantize", lambda: a.fp8_dequantize(self.Xq, E4, self.six, self.Xhat)),
        ]
        if "fprop" in self.passes:      # Y[T,O] = X[T,I] . W[I,O]   (W stored with the output index contiguous)
            calls.append(("gemm_fprop", lambda: a.fp8_gemm(self.Xq, E4, KM, self.Wq, E4, MN, self.Y, self.six, self.siw, self.ay, acc=self.acc)))
        if "dgrad" in self.passes:      # dX[T,I] = dY[T,O] . W^T      (W stored [I,O] is the [N,K] layout here)
            calls.append(("gemm_dgrad", lambda: a.fp8_gemm(self.dYq, E5, KM, self.Wq, E4, KM, self.dX, self.sig, self.siw, self.adx, acc=self.acc)))
        if "wgrad" in self.passes:      # dW[I,O] = X^T . dY           (both operands stored with the contraction index outermost)
            calls.append(("gemm_wgrad", lambda: a.fp8_gemm(self.Xq, E4, MN, self.dYq, E5, MN, self.dW, self.six, self.sig, self.adw, acc=self.acc)))
        return calls

    def cast_elements(self, label):
        return {"quantize_current_X": self.T * self.I, "quantize_current_W": self.I * self.O,
                "quantize_current_dY": self.T * self.O, "dequantize": self.T * self.I}[label]

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


def per_label_ms(events):
    """average device time per call label over the recorded steps"""
    acc = {}
    for row in events:
        for (label, e0), (_, e1) in zip(row[:-1], row[1:]):
            acc.setdefault(label, []).append(e0.elapsed_time(e1))
    return {k: sum(v) / len(v) for k, v in acc.items()}


def step_figures(step, avg):
    """per-kernel figures of a step from its per-label average times: GEMM TFLOP/s, cast GB/s"""
    gemms = {k: round(step.flops_per_gemm / (avg[k] * 1e-3) / 1e12, 1) for k in avg if k.startswith("gemm_")}
    casts = {}
    for k in avg:
        if k.startswith("quantize_current"):
            casts[k] = round(5.0 * step.cast_elements(k) / (avg[k] * 1e-3) / 1e9, 1)
        elif k == "dequantize":
            casts[k] = round(3.0 * step.cast_elements(k) / (avg[k] * 1e-3) / 1e9, 1)
    gemm_ms = sum(avg[k] for k in gemms) / max(1, len(gemms))
    cast_ms = sum(avg[k] for k in casts)
    total = sum(avg.values())
    return {"gemm_tflops": gemms, "cast_gbs": casts,
            "gemm_mean_tflops": step.flops_per_gemm / (gemm_ms * 1e-3) / 1e12,
            "cast_total_gbs": step.cast_bytes / (cast_ms * 1e-3) / 1e9,
            "kernels": {k: {"avg_ms": round(v, 4), "share": round(v / total, 4)} for k, v in avg.items()}}


def bench_cast_sizes(torch, api, synth, device, pk, sizes=(20, 24, 28, 30)):
    """The bandwidth sweep over tensor sizes (bf16, 2^20 .. 2^30 elements).  Each kernel is timed twice:
     - "same_buffer": 20 back-to-back calls on one tensor; below ~126 MB of traffic the tensor stays in L2, so the
       figure is flagged l2_resident and is a latency / L2 number, not an HBM one;
     - "ring": a CUDA graph of calls that walk a ring of distinct tensors totalling more than 512 MB, so that every
       call misses L2: the HBM-honest figure for the small sizes (and the launch cost without host gaps).
    Calls of a few microseconds are bound by launch latency, not by HBM: flagged latency_bound."""
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
            "quantize_e5m2_with_amax": (lambda i: api.fp8_quantize(xs[i], api.E5M2, s, cs[i], api.SATURATE, a), 3.0 * n),
            "quantize_current_e4m3": (lambda i: api.fp8_quantize_current(xs[i], api.E4M3, cs[i], a, s2, si2), 5.0 * n),
            "dequantize_e4m3": (lambda i: api.fp8_dequantize(cs[i], api.E4M3, si, bs[i]), 3.0 * n),
            "fake_quantize_e4m3": (lambda i: api.fp8_fake_quantize(xs[i], api.E4M3, s, si, bs[i]), 4.0 * n),
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
                             "frac_of_measured_hbm": round(nbytes / gms / 1e6 / pk["hbm_gbs"], 4), "calls_in_graph": calls,
                             "latency_bound": bool(gms * 1e3 < 8.0)}
            del graph
            row[name] = entry
        out["2pow%d" % log2n] = row
        del x, codes, back, xs, cs, bs
        torch.cuda.empty_cache()
    return out


def timed_alone(torch, fn, n=20):
    """mean of n back-to-back calls after a short idle and three warm-up calls: a kernel timed by itself (burst)"""
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


def best_single_launch(torch, fn, n=10):
    """the fastest of n individually timed launches after a short idle: how the measured bf16 burst peak was taken"""
    torch.cuda.synchronize()
    time.sleep(0.25)
    best = float("inf")
    for _ in range(n):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    return best


def bench_layer_alone(torch, step, pk, n_gemm=20):
    """Every call of a layer's step timed by itself (burst regime), with its roofline fraction:
    GEMMs against 2 x the measured bf16 burst rate, casts against the measured copy bandwidth."""
    out = {}
    for label, fn in step.calls():
        if label.startswith("gemm_"):
            ms = timed_alone(torch, fn, n_gemm)
            tf = step.flops_per_gemm / ms / 1e9
            out[label] = {"ms": round(ms, 4), "tflops": round(tf, 1), "frac_of_2x_measured_bf16_burst": round(tf / (2 * pk["bf16_burst"]), 4),
                          "frac_of_nominal_4500": round(tf / NOMINAL_FP8_TFLOPS, 4)}
        else:
            ms = timed_alone(torch, fn)
            nbytes = (5.0 if label.startswith("quantize_current") else 3.0) * step.cast_elements(label)
            out[label] = {"ms": round(ms, 4), "gbs": round(nbytes / ms / 1e6, 1), "frac_of_measured_hbm": round(nbytes / ms / 1e6 / pk["hbm_gbs"], 4),
                          "frac_of_nominal_8000": round(nbytes / ms / 1e6 / NOMINAL_HBM_GBS, 4)}
    return out


def bench_tiny(torch, api, synth, device):
    """The 256 x 256 fp32 tensors of the smallest workload: casts and a 256^3 GEMM, every call latency-bound."""
    f32, u8 = torch.float32, torch.uint8
    out = {}
    A = synth.normal_with_scaled_outliers(256 * 256, 0, synth.A_ID, 0.005, 64.0, dtype=f32, device=device).view(256, 256)
    B = synth.normal_with_scaled_outliers(256 * 256, 0, synth.B_ID, 0.005, 64.0, dtype=f32, device=device).view(256, 256)
    q, sc = [], []
    for name, x in (("A", A), ("B", B)):
        c = torch.empty(256, 256, dtype=u8, device=device)
        s = torch.zeros(3, dtype=f32, device=device)
        ms = timed_alone(torch, lambda: api.fp8_quantize_current(x, api.E4M3, c, s[0:1], s[1:2], s[2:3]))
        out["quantize_current_%s_256x256_fp32" % name] = {"us": round(ms * 1e3, 2), "latency_bound": True}
        q.append(c); sc.append(s)
    D = torch.empty(256, 256, dtype=f32, device=device)
    am = torch.zeros(1, dtype=f32, device=device)
    ms = timed_alone(torch, lambda: api.fp8_gemm(q[0], api.E4M3, api.MAJOR_K, q[1], api.E4M3, api.MAJOR_K, D, sc[0][2:3], sc[1][2:3], am))
    out["gemm_256x256x256_fp32_out"] = {"us": round(ms * 1e3, 2), "latency_bound": True,
                                        "note": "host time of one call included: the launches are issued back to back from Python"}
    return out


def bench_next_rows(torch, api, synth, device, pk, iters=5):
    """The rows beyond the core path, each timed alone on workload-shaped tensors: simulated-FP8 round trip,
    per-channel weight scales, FP8-output GEMM, attention-style batched GEMM."""
    def timed(fn):
        return timed_alone(torch, fn, 4 * iters)

    L = LAYERS["hidden4096"]
    TOKENS, D_IN, D_OUT, W_SIGMA = L["tokens"], L["d_in"], L["d_out"], L["w_sigma"]
    out = {}
    f32 = torch.float32
    sc = torch.tensor([3.0, 1.0 / 3.0, 0.0, 0.0], dtype=f32, device=device)
    s, si, a = sc[0:1], sc[1:2], sc[2:3]
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
    # split accumulation (partial sums every 2048 of K added in registers) against one accumulator, same codes:
    # forward K = 4096 and, on the same codes read as dY-shaped operands, the dgrad shape K = 16384
    for name, acc in (("one_accumulator", api.ACC_FAST), ("split_accumulation", api.ACC_SPLIT)):
        ms = timed(lambda: api.fp8_gemm(Xq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_MN, Y, sx[2:3], si, a, acc=acc))
        out["gemm_fprop_K4096_" + name] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1)}
    dX = torch.empty(TOKENS, D_IN, dtype=torch.bfloat16, device=device)
    for name, acc in (("one_accumulator", api.ACC_FAST), ("split_accumulation", api.ACC_SPLIT)):
        ms = timed(lambda: api.fp8_gemm(Yq, api.E4M3, api.MAJOR_K, Wq, api.E4M3, api.MAJOR_K, dX, si, si, a, acc=acc))
        out["gemm_dgrad_K16384_" + name] = {"ms": round(ms, 4), "tflops": round(flops / ms / 1e9, 1)}
    del dX, W, X, Y, Yq
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


def oracle_step(layer: str, sample_tokens: int, threads: int, sample_out: int | None = None, inputs=None):
    """The same step on a bounded sample of the layer: `sample_tokens` tokens and `sample_out` output features
    (W is [d_in, sample_out], same recipe), run by the CPU oracle as it stands.  `inputs` = (X, W, dY) as bf16 bit
    patterns of exactly that sample (the GPU arm passes slices of its own tensors); otherwise they are generated here.
    Returns (seconds, gemm flops of the sample)."""
    import numpy as np
    import torch

    import oracle
    from paper_2209_05433_b200 import synth

    L = LAYERS[layer]
    T, I, O = sample_tokens, L["d_in"], sample_out or L["d_out"]

    def bits(t):
        return t.view(torch.int16).numpy().view(np.uint16)

    key = (layer, T, O)
    if inputs is not None:
        _oracle_inputs.clear()
        _oracle_inputs[key] = inputs
    if key not in _oracle_inputs:                                  # synthetic inputs are made once, outside the timed part
        _oracle_inputs.clear()
        _oracle_inputs[key] = (bits(synth.activations(T * I, L["seed"], dtype=torch.bfloat16)),
                               bits(synth.weights(I * O, L["seed"], L["w_sigma"], dtype=torch.bfloat16)),
                               bits(synth.gradients(T * O, L["seed"], dtype=torch.bfloat16)))
    X, W, dY = _oracle_inputs[key]
    t0 = time.perf_counter()
    q, sinv = {}, {}
    for name, t, fmt in (("x", X, oracle.E4M3), ("w", W, oracle.E4M3), ("g", dY, oracle.E5M2)):
        s, si = oracle.scale_from_amax(oracle.amax(t, threads), fmt)
        q[name], sinv[name] = oracle.quantize(t, s, fmt, threads=threads), si
    oracle.dequantize(q["x"], sinv["x"], oracle.E4M3, "bf16", threads=threads)
    def product(A, fa, a_str, B, fb, b_str, rows, cols, k, sa, sb):
        """every output element of a rows x cols product through the oracle's per-element routine; the element list
        (not the few rows of the sample) is what is split over the host cores"""
        ii, jj = np.repeat(np.arange(rows, dtype=np.int64), cols), np.tile(np.arange(cols, dtype=np.int64), rows)
        return oracle.gemm_samples(A, fa, a_str, B, fb, b_str, k, ii, jj, sa, sb, threads=threads)[0]

    results = []
    if "fprop" in L["passes"]:
        results.append(product(q["x"], oracle.E4M3, (I, 1), q["w"], oracle.E4M3, (O, 1), T, O, I, sinv["x"], sinv["w"]))
    if "dgrad" in L["passes"]:
        results.append(product(q["g"], oracle.E5M2, (O, 1), q["w"], oracle.E4M3, (1, O), T, I, O, sinv["g"], sinv["w"]))
    if "wgrad" in L["passes"]:
        results.append(product(q["x"], oracle.E4M3, (1, I), q["g"], oracle.E5M2, (O, 1), I, O, T, sinv["x"], sinv["g"]))
    for r in results:
        oracle.round_bf16_from_f64(r)
    dt = time.perf_counter() - t0
    return dt, len(results) * 2.0 * T * I * O


def reference_sample(layer: str, steps: int, warmup: int, threads: int):
    """(tokens, output features) of the per-step sample: 4 tokens and as many output features (multiples of
    256) as fit about 150 s for the whole run, at most the full layer.
    Every cost of the step (weight cast, the GEMMs) is linear in the feature count."""
    t_small, _ = oracle_step(layer, 4, threads, 256)               # calibration on the smallest sample
    total = float(os.environ.get("FP8_BENCH_REFERENCE_SECONDS", "150"))      # wall-clock aim for the whole run
    budget = min(8.0, total / max(1, steps + warmup))
    grow = max(1.0, budget / max(t_small, 1e-3))
    sample_out = int(min(LAYERS[layer]["d_out"], 256 * int(grow)))
    return 4, max(256, sample_out // 256 * 256)


def run_reference(args, world, rank):
    if rank != 0:
        return                                                     # the oracle runs once, on rank 0's host cores
    layer = HEADLINE
    L = LAYERS[layer]
    threads = os.cpu_count() or 1
    sample_tokens, sample_out = reference_sample(layer, args.steps, args.warmup, threads)
    for _ in range(args.warmup):
        oracle_step(layer, sample_tokens, threads, sample_out)
    times, flops = [], 0.0
    for _ in range(args.steps):
        dt, flops = oracle_step(layer, sample_tokens, threads, sample_out)
        times.append(dt)
    total = sum(times)
    value = flops * len(times) / total / 1e12
    sample = "the same step on %d of the %d tokens and %d of the %d output features, CPU oracle as it stands" % (
        sample_tokens, L["tokens"], sample_out, L["d_out"])
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64 accumulation over decoded fp8 codes", "data": "synthetic",
        "config": {"workload": workload_text(layer), "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------

def run_only(args, torch, api, synth, device):
    """One call of a layer's step, alone (what the ncu captures under profiles/ run): a full step first to set
    scales and codes, then `--steps` launches of the named call."""
    step = LinearStep(torch, api, synth, device, args.layer, acc=api.ACC_FAST if args.acc == "fast" else api.ACC_SPLIT)
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
    st, detail = api.fp8_async_status()
    if st != 0:
        raise SystemExit("device-side wait expired (code %d)" % detail)
    print(json.dumps({"only": args.only, "layer": args.layer, "steps": args.steps, "ms_per_call": e0.elapsed_time(e1) / args.steps}))


def run_ours(args, world, rank, local):
    import torch
    import torch.distributed as dist

    from paper_2209_05433_b200 import api, synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    if local >= torch.cuda.device_count():
        raise SystemExit("rank %d has no GPU: %d visible" % (local, torch.cuda.device_count()))
    torch.cuda.set_device(local)
    device = "cuda:%d" % local
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(device))
    api.load()
    pk = peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=device)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return ms

    if args.only:
        run_only(args, torch, api, synth, device)
        return
    if args.config:
        if args.config == 1:
            res = bench_tiny(torch, api, synth, device)
        elif args.config == 2:
            res = bench_cast_sizes(torch, api, synth, device, pk)
        elif args.config in (3, 4, 5):
            res = bench_layer_alone(torch, LinearStep(torch, api, synth, device, "hidden12288" if args.config == 5 else "hidden4096"), pk,
                                    n_gemm=5 if args.config == 5 else 20)
        else:
            raise SystemExit("--config takes 1..5")
        print(json.dumps({"config": args.config, "results": res}))
        return

    # independent batches per rank: no data-path collective (per-tensor amax is local to a rank's own tensors)
    layer = HEADLINE
    step = LinearStep(torch, api, synth, device, layer, seed_offset=16 * rank)
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step.run()
    barrier()
    st, detail = api.fp8_async_status()
    if st != 0:
        raise SystemExit("device-side wait expired during warm-up (code %d)" % detail)

    # ---- the K timed steps
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
    total_ms = max_over_ranks(events[0][0][1].elapsed_time(events[-1][-1][1]))
    avg = per_label_ms(events)
    clocks = sampler.stop() if rank == 0 else None
    st, detail = api.fp8_async_status()
    if st != 0:
        raise SystemExit("device-side wait expired during the timed region (code %d)" % detail)

    # ---- sustained: whole steps back to back for at least two seconds, clocks sampled over exactly that loop
    ms_per_step = total_ms / args.steps
    n_sus = max(args.steps, int(args.sustained_seconds * 1e3 / ms_per_step) + 1)
    sampler2 = ClockSampler(local)
    if rank == 0:
        sampler2.start()
    sus_events = []
    # the SM clock as the kernels see it: a one-warp probe kernel on a second stream, a 100 us window every few steps
    # (few and short: while a window is open on an SM, a CTA that needs the whole register file waits for it)
    n_probes = 16
    probe_out = torch.zeros(n_probes, 2, dtype=torch.int64, device=device)
    s_probe = torch.cuda.Stream()
    probe_every = max(1, n_sus // n_probes)
    barrier()
    for i in range(n_sus):
        step.run_timed(sus_events)
        if i % probe_every == 0 and i // probe_every < n_probes and i >= n_sus // 4:
            with torch.cuda.stream(s_probe):
                api.fp8_sm_clock_probe(probe_out[i // probe_every], 100)
    barrier()
    probes = [(int(c), int(t)) for c, t in probe_out.cpu().tolist() if t > 0]
    device_mhz = sorted(c * 1000.0 / t for c, t in probes)
    device_mhz_median = device_mhz[len(device_mhz) // 2] if device_mhz else None
    sus_ms = max_over_ranks(sus_events[0][0][1].elapsed_time(sus_events[-1][-1][1]))
    sus_avg = per_label_ms(sus_events[len(sus_events) // 4:])      # per-kernel figures from the last three quarters: clocks have settled
    sus_clocks = sampler2.stop() if rank == 0 else None
    del events, sus_events

    # ---- end to end: pinned host inputs -> device, the step, results -> pinned host, EVERY step.
    # Three streams (copy in, compute, copy out) and two device buffer sets, so that the upload of step i+1 and
    # the download of step i-1 overlap the kernels of step i; each step still moves all of its own bytes.
    steps2 = [step, LinearStep(torch, api, synth, device, layer, seed_offset=16 * rank)]
    host_in = [torch.empty(t.shape, dtype=t.dtype).pin_memory().copy_(t) for t in step.inputs]
    host_out = [[torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in s_.outputs] for s_ in steps2]
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
        sb = steps2[b]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_comp[b])                  # the previous step on this set has consumed its inputs
            for h, d in zip(host_in, sb.inputs):
                d.copy_(h, non_blocking=True)
            ev_in[b].record(s_in)
        with torch.cuda.stream(s_comp):
            s_comp.wait_event(ev_in[b])
            s_comp.wait_event(ev_out[b])                 # its previous outputs have left the device buffers
            sb.run()
            ev_comp[b].record(s_comp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_comp[b])
            for h, d in zip(host_out[b], sb.outputs):
                h.copy_(d, non_blocking=True)
            host_scal[b].copy_(sb.scal, non_blocking=True)
            ev_out[b].record(s_out)

    e2e_steps = max(2, min(args.steps, 6))
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
    e2e_ms = max_over_ranks(e0.elapsed_time(e1))
    del steps2[1], host_in, host_out
    torch.cuda.empty_cache()

    if rank == 0:
        value = step.gemm_flops * world / (ms_per_step * 1e-3) / 1e12
        burst = step_figures(step, avg)
        sus = step_figures(step, sus_avg)
        sus_ms_per_step = sus_ms / n_sus
        sms = torch.cuda.get_device_properties(local).multi_processor_count
        traffic = ncu_traffic()

        def clock_normalised(tflops, mhz):
            """fraction of the tensor pipes' rate at the clock the loop ran at: flop / (SMs x 8192 MAC x 2 x clock)"""
            if not mhz:
                return None
            return round(tflops * 1e12 / (sms * FP8_MACS_PER_SM_PER_CLOCK * 2.0 * mhz * 1e6), 4)

        # dominant kernel: the FP8 GEMM (launches of 2*T*I*O flops each).  frac: sustained figure / sustained peak.
        fp8_sus, fp8_burst = 2.0 * pk["bf16_sustained"], 2.0 * pk["bf16_burst"]         # fp8 : bf16 nominal ratio is 2
        a_sus, a_burst = sus["gemm_mean_tflops"], burst["gemm_mean_tflops"]
        roofline = {
            "bound": "tensor", "kernel": "k_gemm_fp8", "achieved": round(a_sus, 1), "peak": round(fp8_sus, 1), "unit": "TFLOP/s",
            "frac": round(a_sus / fp8_sus, 4), "traffic": traffic.get("k_gemm_fp8.fprop." + layer),
            "regime": "sustained: per-launch CUDA events inside a loop of %d whole steps (%.2f s), divided by 2 x %s bf16 sustained cuBLAS "
                      "TFLOP/s (fp8:bf16 nominal ratio 2)" % (n_sus, sus_ms / 1e3, pk["source"]),
            "algorithmic_flops_per_launch": step.flops_per_gemm,
            "accumulation": "library default: partial sums every 2048 of K added in registers (1e-5 * sum|a.b| for any data); "
                            "the single-accumulator mode FP8_ACC_FAST is 2.5-4 % faster, see next_rows",
            "per_gemm_tflops": sus["gemm_tflops"],
            "clock_normalised": {"sm_mhz_on_device_median": round(device_mhz_median, 1) if device_mhz_median else None,
                                 "frac_of_tensor_pipe_rate": clock_normalised(a_sus, device_mhz_median),
                                 "probes": len(device_mhz), "sm_mhz_on_device_min_max": [round(device_mhz[0], 1), round(device_mhz[-1], 1)] if device_mhz else None,
                                 "sm_mhz_sampled_median": sus_clocks["sm_mhz"], "frac_with_sampled_clock": clock_normalised(a_sus, sus_clocks["sm_mhz"]),
                                 "formula": "flop / (%d SMs x %d MAC x 2 x SM clock); the clock is read on the device by a one-warp probe kernel on a second "
                                            "stream during the loop (100 us windows, on whichever SM has registers free); the nvidia-smi samples of the same loop are given for comparison"
                                            % (sms, FP8_MACS_PER_SM_PER_CLOCK)},
            "burst": {"achieved": round(a_burst, 1), "peak": round(fp8_burst, 1), "frac": round(a_burst / fp8_burst, 4),
                      "regime": "the %d timed steps (%.3f s), divided by 2 x %s bf16 burst cuBLAS TFLOP/s" % (args.steps, total_ms / 1e3, pk["source"]),
                      "per_gemm_tflops": burst["gemm_tflops"]},
            "frac_of_nominal_4500": round(a_sus / NOMINAL_FP8_TFLOPS, 4), "burst_frac_of_nominal_4500": round(a_burst / NOMINAL_FP8_TFLOPS, 4),
            "traffic_note": "DRAM bytes per launch of the forward GEMM from the ncu capture summarised under profiles/; algorithmic %.3e"
                            % (step.T * step.I + step.I * step.O + 2.0 * step.T * step.O),
        }
        # the memory-bound half: amax + quantize (+ dequantize) of the step against HBM
        c_sus, c_burst = sus["cast_total_gbs"], burst["cast_total_gbs"]
        roofline_cast = {
            "bound": "hbm", "kernel": "casts of the step: current scaling of X (one cooperative k_quantize_current), of W and dY (k_amax + k_scale_from_amax + k_quantize each, tensors of 256 MB and more) + k_dequantize", "achieved": round(c_sus, 1),
            "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": round(c_sus / pk["hbm_gbs"], 4),
            "traffic": traffic.get("cast_W." + layer),
            "traffic_note": "DRAM bytes of one current-scaling call on W (the amax and the quantize kernel together) from the ncu capture "
                            "summarised under profiles/; algorithmic %.3e" % (5.0 * step.I * step.O),
            "peak_source": pk["source"] + " copy bandwidth", "regime": "sustained loop (same as roofline)",
            "per_call_gbs": sus["cast_gbs"], "burst": {"achieved": round(c_burst, 1), "frac": round(c_burst / pk["hbm_gbs"], 4), "per_call_gbs": burst["cast_gbs"]},
            "frac_of_nominal_8000": round(c_sus / NOMINAL_HBM_GBS, 4),
            "algorithmic_bytes": "5 B per bf16 element for amax+quantize (two reads, one write), 3 B per element for dequantize; "
                                 "re-reads served by L2 still count as algorithmic bytes",
        }
        sustained = {"steps": n_sus, "seconds": round(sus_ms / 1e3, 3), "ms_per_step": round(sus_ms_per_step, 4),
                     "value": round(step.gemm_flops * world / (sus_ms_per_step * 1e-3) / 1e12, 1), "unit": UNIT, "clocks": sus_clocks,
                     "kernels": sus["kernels"]}
        per_config = cast_sizes = next_rows = cpu = None
        if world == 1 and not args.quick:
            threads = os.cpu_count() or 1
            cpu_tokens = 4 if threads >= 12 else 2                 # about 20 s of CPU work on 16 cores
            to_bits = lambda t: t.contiguous().cpu().view(torch.int16).numpy().view("uint16").reshape(-1)
            cpu_inputs = (to_bits(step.X[:cpu_tokens]), to_bits(step.W), to_bits(step.dY[:cpu_tokens]))
            best_launch = {}
            for label, fn in step.calls():
                if label.startswith("gemm_"):
                    tf = step.flops_per_gemm / best_single_launch(torch, fn) / 1e9
                    best_launch[label] = {"tflops": round(tf, 1), "frac_of_2x_measured_bf16_burst": round(tf / (2 * pk["bf16_burst"]), 4),
                                          "frac_of_nominal_4500": round(tf / NOMINAL_FP8_TFLOPS, 4)}
            del step
            torch.cuda.empty_cache()
            cast_sizes = bench_cast_sizes(torch, api, synth, device, pk)
            small = LinearStep(torch, api, synth, device, "hidden4096")
            per_config = {
                "1_tiny_256": bench_tiny(torch, api, synth, device),
                "2_cast_sweep": "see cast_sizes",
                "3_4_hidden4096_each_call_alone": bench_layer_alone(torch, small, pk),
                "5_hidden12288": {"burst_in_step": {"gemm_tflops": burst["gemm_tflops"], "cast_gbs": burst["cast_gbs"]},
                                  "sustained_in_step": {"gemm_tflops": sus["gemm_tflops"], "cast_gbs": sus["cast_gbs"]},
                                  "gemm_best_single_launch_of_10_after_idle": best_launch},
            }
            del small
            torch.cuda.empty_cache()
            next_rows = bench_next_rows(torch, api, synth, device, pk)
            dt, flops = oracle_step(layer, cpu_tokens, threads, inputs=cpu_inputs)
            cpu = {"value": flops / dt / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": round(dt, 2),
                   "sample": "the same step with %d of the %d tokens (weights at full size), CPU oracle as it stands" % (cpu_tokens, LAYERS[layer]["tokens"])}
        L = LAYERS[layer]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "fp8 (e4m3/e5m2) operands, f32 accumulate, bf16 out", "data": "synthetic",
            "config": {"workload": workload_text(layer), "tokens": L["tokens"], "d_in": L["d_in"], "d_out": L["d_out"], "parallelism": "dp%d" % world,
                       "l2": "inputs larger than L2 (step touches > 5 GB)", "weights_layout": "[d_in, d_out] row-major",
                       "regime_of_value": "the K timed steps (burst clocks when K steps last well under a second); see `sustained`"},
            "clocks": clocks,
            "e2e": {"value": step_flops_e2e(L, world, e2e_ms / e2e_steps), "unit": UNIT,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
                    "how": "pinned host buffers; upload, kernels and download of consecutive steps overlap on three streams"},
            "gpu_launches": int(launches), "gpu_launches_note": "kernels plus 4-byte memset nodes enqueued by the library in the timed region",
            "roofline": roofline, "roofline_cast": roofline_cast, "sustained": sustained, "kernels": burst["kernels"],
            "per_config": per_config, "cast_sizes": cast_sizes, "next_rows": next_rows, "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def step_flops_e2e(L, world, ms):
    return len(L["passes"]) * 2.0 * L["tokens"] * L["d_in"] * L["d_out"] * world / (ms * 1e-3) / 1e12


def spawn_ranks(n):
    """--gpus N without a torchrun environment: start N ranks of this script, one per GPU"""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n), "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--sustained-seconds", type=float, default=2.0, help="minimum length of the sustained whole-step loop")
    ap.add_argument("--quick", action="store_true", help="the step only: no per-config, cast-size, next-row or CPU-baseline sections")
    ap.add_argument("--config", type=int, default=0, help="run one of the five named workloads (1..5), every call timed alone")
    ap.add_argument("--only", default=None, help="time only the calls with this label of a layer's step (e.g. gemm_fprop, quantize_current_W)")
    ap.add_argument("--layer", choices=sorted(LAYERS), default=HEADLINE, help="layer of --only")
    ap.add_argument("--acc", choices=["split", "fast"], default="split", help="accumulation mode of the GEMMs under --only (split = library default)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args.gpus)
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, world, rank)
    else:
        run_ours(args, world, rank, local)


if __name__ == "__main__":
    main()
