"""Helpers shared by the GPU parity tests (no FP8 arithmetic of their own)."""
import os

import numpy as np
import torch

THREADS = max(1, min(32, os.cpu_count() or 1))


def to_np_bits(t: torch.Tensor) -> np.ndarray:
    """torch tensor -> numpy; bf16 as uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def same_with_nan(got: np.ndarray, want: np.ndarray, wide: str) -> np.ndarray:
    """element-wise equality of wide results where every NaN equals every NaN"""
    if wide == "bf16":
        gn = (got & 0x7FFF) > 0x7F80
        wn = (want & 0x7FFF) > 0x7F80
        return np.where(gn | wn, gn & wn, got == want)
    g, w = got.view(np.uint32), want.view(np.uint32)
    gn = (g & 0x7FFFFFFF) > 0x7F800000
    wn = (w & 0x7FFFFFFF) > 0x7F800000
    return np.where(gn | wn, gn & wn, g == w)


def bf16_order(bits: np.ndarray) -> np.ndarray:
    """bf16 patterns -> integers ordered like the values (both zeros map to 0)"""
    b = bits.astype(np.int64)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


def check_gemm_f32(gpu: np.ndarray, ref: np.ndarray, sabs: np.ndarray, rel: float = 1e-5):
    """|gpu - ref| <= rel * sum|a.b| per element; NaN/Inf must match. Returns (ok mask, worst ratio)."""
    gpu = gpu.astype(np.float64)
    special = ~np.isfinite(ref)
    ok = np.empty(ref.shape, dtype=bool)
    with np.errstate(invalid="ignore"):
        err = np.abs(gpu - ref)
        ok[~special] = err[~special] <= rel * sabs[~special]
    ok[special] = np.where(np.isnan(ref[special]), np.isnan(gpu[special]), gpu[special] == ref[special])
    with np.errstate(invalid="ignore", divide="ignore"):
        ratio = np.where(sabs > 0, err / sabs, 0.0)
    worst = float(np.nanmax(ratio[~special])) if (~special).any() else 0.0
    return ok, worst


def check_gemm_bf16(gpu_bits: np.ndarray, ref: np.ndarray, sabs: np.ndarray, round_bf16, rel: float = 1e-5):
    """bf16 criterion: the stored pattern lies within 1 bf16 ulp of the correctly rounded value of some
    v in [ref - rel*sabs, ref + rel*sabs].  Wherever that interval is narrower than a quarter of a bf16 ulp of
    the reference (no cancellation: the accumulation tolerance cannot move the rounding by a whole step) the
    literal test is required as well: within 1 ulp of the correctly rounded reference.
    Returns (ok mask, literal mask); `literal` is reported for the remaining elements too."""
    special = ~np.isfinite(ref)
    tol = rel * sabs
    lo = bf16_order(round_bf16(np.where(special, 0.0, ref - tol)))
    hi = bf16_order(round_bf16(np.where(special, 0.0, ref + tol)))
    mid = bf16_order(round_bf16(np.where(special, 0.0, ref)))
    g = bf16_order(gpu_bits)
    g_nan = (gpu_bits & 0x7FFF) > 0x7F80
    ok = (g >= lo - 1) & (g <= hi + 1) & ~g_nan
    literal = (np.abs(g - mid) <= 1) & ~g_nan
    # one bf16 ulp of the reference: 2^(exponent - 7), exponent clamped at the smallest normal
    with np.errstate(divide="ignore", invalid="ignore"):
        expo = np.floor(np.log2(np.maximum(np.abs(np.where(special, 1.0, ref)), 2.0 ** -126)))
    ulp = np.exp2(expo - 7)
    must_be_literal = tol < 0.25 * ulp
    ok &= literal | ~must_be_literal
    if special.any():
        gv = (gpu_bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        sp_ok = np.where(np.isnan(ref), g_nan, gv == ref)
        ok = np.where(special, sp_ok, ok)
        literal = np.where(special, sp_ok, literal)
    return ok, literal


def fp8_order(codes: np.ndarray) -> np.ndarray:
    """FP8 codes -> integers ordered like the values (sign-magnitude; both zeros map to 0)"""
    c = codes.astype(np.int64)
    return np.where(c & 0x80, -(c & 0x7F), c & 0x7F)


def check_gemm_fp8out(gpu_codes: np.ndarray, ref: np.ndarray, sabs: np.ndarray, scale_d: float, encode, rel: float = 1e-5):
    """FP8-output criterion: the stored code is encode(v * scale_d) for some v in [ref - rel*sabs, ref + rel*sabs]
    (encode is monotonic, so that set is the code interval between the encodings of the two ends; no further
    slack: the epilogue's own binary32 roundings are ~2^-23 relative, far inside rel*sabs >= rel*|ref|).
    `encode(float32 array) -> codes` is the oracle's conversion.  NaN reference -> NaN code.
    Returns (ok mask, mask of codes equal to encode(ref * scale_d))."""
    special = ~np.isfinite(ref)
    tol = rel * sabs
    sd = np.float64(scale_d)
    with np.errstate(over="ignore", invalid="ignore"):
        lo = fp8_order(encode(np.where(special, 0.0, (ref - tol) * sd).astype(np.float32)))
        hi = fp8_order(encode(np.where(special, 0.0, (ref + tol) * sd).astype(np.float32)))
        want = encode((ref * sd).astype(np.float32))
    g = fp8_order(gpu_codes)
    ok = (g >= lo) & (g <= hi)
    exact = gpu_codes == want
    if special.any():
        ok = np.where(special, exact, ok)
    return ok, exact
