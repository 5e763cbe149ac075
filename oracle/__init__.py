"""CPU oracle for the FP8 hot path (test infrastructure, never the product path).

Thin numpy/ctypes front end over ``fp8_oracle.c`` (plain scalar C, compiled with
gcc on first use).  Only tests, the smoke check and the bench's CPU-baseline leg
may import this package; the CUDA library neither imports nor links it.

Every function takes and returns numpy arrays; bf16 tensors travel as uint16
bit patterns, FP8 tensors as uint8 codes.  ``threads`` only splits the element
range into contiguous chunks handed to the same scalar C routine (ctypes drops
the GIL), it changes no arithmetic.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading
from concurrent.futures import ThreadPoolExecutor

import numpy as np

E4M3, E5M2 = 0, 1
SATURATE, NOSAT = 0, 1
FMT_MAX = {E4M3: 448.0, E5M2: 57344.0}   # Table 1, "Max normal"

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fp8_oracle.c")
_LIB = os.path.join(_HERE, "libfp8_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle next to its source; returns the library path."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-ffp-contract=off", "-fno-fast-math", "-std=c11", "-shared", "-fPIC",
                 "-o", tmp, _SRC, "-lm"])
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    c = ctypes
    u8p, u16p, f32p, f64p, i64p = (c.POINTER(c.c_uint8), c.POINTER(c.c_uint16), c.POINTER(c.c_float),
                                   c.POINTER(c.c_double), c.POINTER(c.c_int64))
    lib.fp8o_decode.restype = c.c_double
    lib.fp8o_decode.argtypes = [c.c_uint8, c.c_int]
    lib.fp8o_decode_table.restype = None
    lib.fp8o_decode_table.argtypes = [c.c_int, f64p]
    lib.fp8o_encode.restype = c.c_uint8
    lib.fp8o_encode.argtypes = [c.c_float, c.c_int, c.c_int]
    lib.fp8o_f32_to_bf16.restype = c.c_uint16
    lib.fp8o_f32_to_bf16.argtypes = [c.c_float]
    lib.fp8o_f64_to_bf16.restype = c.c_uint16
    lib.fp8o_f64_to_bf16.argtypes = [c.c_double]
    lib.fp8o_f64_to_bf16_array.restype = None
    lib.fp8o_f64_to_bf16_array.argtypes = [f64p, c.c_size_t, u16p]
    lib.fp8o_count_double_rounding_f32.restype = c.c_size_t
    lib.fp8o_count_double_rounding_f32.argtypes = [f32p, c.c_size_t, c.c_float, c.c_int, c.c_int]
    lib.fp8o_quantize_f32.restype = None
    lib.fp8o_quantize_f32.argtypes = [f32p, c.c_size_t, c.c_float, c.c_int, c.c_int, u8p]
    lib.fp8o_quantize_bf16.restype = None
    lib.fp8o_quantize_bf16.argtypes = [u16p, c.c_size_t, c.c_float, c.c_int, c.c_int, u8p]
    lib.fp8o_dequantize_f32.restype = None
    lib.fp8o_dequantize_f32.argtypes = [u8p, c.c_size_t, c.c_int, c.c_float, f32p]
    lib.fp8o_dequantize_bf16.restype = None
    lib.fp8o_dequantize_bf16.argtypes = [u8p, c.c_size_t, c.c_int, c.c_float, u16p]
    lib.fp8o_amax_f32.restype = c.c_uint32
    lib.fp8o_amax_f32.argtypes = [f32p, c.c_size_t]
    lib.fp8o_amax_bf16.restype = c.c_uint32
    lib.fp8o_amax_bf16.argtypes = [u16p, c.c_size_t]
    lib.fp8o_scale_from_amax.restype = None
    lib.fp8o_scale_from_amax.argtypes = [c.c_float, c.c_int, f32p, f32p]
    lib.fp8o_scale_pow2_from_amax.restype = None
    lib.fp8o_scale_pow2_from_amax.argtypes = [c.c_float, c.c_int, f32p, f32p]
    gemm_common = [u8p, c.c_int, c.c_int64, c.c_int64, u8p, c.c_int, c.c_int64, c.c_int64]
    lib.fp8o_gemm_rows.restype = None
    lib.fp8o_gemm_rows.argtypes = gemm_common + [c.c_int64, c.c_int64, c.c_int64, c.c_int64,
                                                 c.c_float, c.c_float, f64p, f64p]
    u32p = c.POINTER(c.c_uint32)
    lib.fp8o_amax_channels_f32.restype = None
    lib.fp8o_amax_channels_f32.argtypes = [f32p, c.c_int64, c.c_int64, c.c_int64, c.c_int, u32p]
    lib.fp8o_amax_channels_bf16.restype = None
    lib.fp8o_amax_channels_bf16.argtypes = [u16p, c.c_int64, c.c_int64, c.c_int64, c.c_int, u32p]
    lib.fp8o_quantize_channels_f32.restype = None
    lib.fp8o_quantize_channels_f32.argtypes = [f32p, c.c_int64, c.c_int64, c.c_int64, c.c_int, f32p, c.c_int, c.c_int, u8p, c.c_int64]
    lib.fp8o_quantize_channels_bf16.restype = None
    lib.fp8o_quantize_channels_bf16.argtypes = [u16p, c.c_int64, c.c_int64, c.c_int64, c.c_int, f32p, c.c_int, c.c_int, u8p, c.c_int64]
    lib.fp8o_gemm_rows_colscale.restype = None
    lib.fp8o_gemm_rows_colscale.argtypes = gemm_common + [c.c_int64, c.c_int64, c.c_int64, c.c_int64,
                                                          c.c_float, f32p, f64p, f64p]
    lib.fp8o_gemm_samples.restype = None
    lib.fp8o_gemm_samples.argtypes = gemm_common + [c.c_int64, i64p, i64p, c.c_int64,
                                                    c.c_float, c.c_float, f64p, f64p]
    lib.fp8o_dot_exact.restype = c.c_int
    lib.fp8o_dot_exact.argtypes = [u8p, c.c_int, c.c_int64, u8p, c.c_int, c.c_int64, c.c_int64,
                                   i64p, c.POINTER(c.c_uint64), c.POINTER(c.c_int)]
    _lib = lib
    return lib


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _chunks(n: int, threads: int):
    threads = max(1, min(int(threads), max(1, n)))
    step = -(-n // threads)
    return [(lo, min(n, lo + step)) for lo in range(0, n, step)] if n else []


def _run(jobs, threads):
    if threads <= 1 or len(jobs) <= 1:
        for j in jobs:
            j()
        return
    with ThreadPoolExecutor(max_workers=threads) as ex:
        for f in [ex.submit(j) for j in jobs]:
            f.result()


# ------------------------------------------------------------------ scalars --

def decode(code: int, fmt: int) -> float:
    return float(_load().fp8o_decode(int(code) & 0xFF, fmt))


def decode_table(fmt: int) -> np.ndarray:
    t = np.empty(256, dtype=np.float64)
    _load().fp8o_decode_table(fmt, _ptr(t, ctypes.c_double))
    return t


def encode(y, fmt: int, overflow: int = SATURATE) -> int:
    return int(_load().fp8o_encode(ctypes.c_float(np.float32(y)), fmt, overflow))


def f32_to_bf16(v) -> int:
    return int(_load().fp8o_f32_to_bf16(ctypes.c_float(np.float32(v))))


def f64_to_bf16(v) -> int:
    return int(_load().fp8o_f64_to_bf16(ctypes.c_double(float(v))))


def scale_from_amax(amax, fmt: int):
    s, si = ctypes.c_float(), ctypes.c_float()
    _load().fp8o_scale_from_amax(ctypes.c_float(np.float32(amax)), fmt, ctypes.byref(s), ctypes.byref(si))
    return np.float32(s.value), np.float32(si.value)


def scale_pow2_from_amax(amax, fmt: int):
    s, si = ctypes.c_float(), ctypes.c_float()
    _load().fp8o_scale_pow2_from_amax(ctypes.c_float(np.float32(amax)), fmt, ctypes.byref(s), ctypes.byref(si))
    return np.float32(s.value), np.float32(si.value)


def fake_quantize(x: np.ndarray, scale, scale_inv, fmt: int, overflow: int = SATURATE, threads: int = 1) -> np.ndarray:
    """Simulated FP8 (Section 4): convert to FP8 and straight back, in the type of x."""
    wide = "f32" if _wide_kind(np.ascontiguousarray(x).reshape(-1)) == "f32" else "bf16"
    return dequantize(quantize(x, scale, fmt, overflow, threads), scale_inv, fmt, wide, threads)


# ------------------------------------------------------------------ tensors --

def _wide_kind(x: np.ndarray) -> str:
    if x.dtype == np.float32:
        return "f32"
    if x.dtype == np.uint16:
        return "bf16"
    raise TypeError("wide tensors are float32 arrays or uint16 arrays of bf16 bit patterns")


def quantize(x: np.ndarray, scale, fmt: int, overflow: int = SATURATE, threads: int = 1) -> np.ndarray:
    """codes = encode(fp32(x) * scale), element by element."""
    lib = _load()
    x = np.ascontiguousarray(x).reshape(-1)
    kind = _wide_kind(x)
    out = np.empty(x.size, dtype=np.uint8)
    sc = ctypes.c_float(np.float32(scale))
    jobs = []
    for lo, hi in _chunks(x.size, threads):
        if kind == "f32":
            jobs.append(lambda lo=lo, hi=hi: lib.fp8o_quantize_f32(
                _ptr(x[lo:hi], ctypes.c_float), hi - lo, sc, fmt, overflow, _ptr(out[lo:hi], ctypes.c_uint8)))
        else:
            jobs.append(lambda lo=lo, hi=hi: lib.fp8o_quantize_bf16(
                _ptr(x[lo:hi], ctypes.c_uint16), hi - lo, sc, fmt, overflow, _ptr(out[lo:hi], ctypes.c_uint8)))
    _run(jobs, threads)
    return out


def count_double_rounding(x: np.ndarray, scale, fmt: int, overflow: int = SATURATE) -> int:
    """Diagnostic: elements whose code would differ if the exact product x*scale were rounded once
    (instead of to binary32 first, then to FP8)."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    return int(_load().fp8o_count_double_rounding_f32(_ptr(x, ctypes.c_float), x.size, ctypes.c_float(np.float32(scale)), fmt, overflow))


def dequantize(codes: np.ndarray, scale_inv, fmt: int, wide: str = "f32", threads: int = 1) -> np.ndarray:
    """wide = round(decode(code) * scale_inv); bf16 results are uint16 bit patterns."""
    lib = _load()
    codes = np.ascontiguousarray(codes, dtype=np.uint8).reshape(-1)
    si = ctypes.c_float(np.float32(scale_inv))
    out = np.empty(codes.size, dtype=np.float32 if wide == "f32" else np.uint16)
    jobs = []
    for lo, hi in _chunks(codes.size, threads):
        if wide == "f32":
            jobs.append(lambda lo=lo, hi=hi: lib.fp8o_dequantize_f32(
                _ptr(codes[lo:hi], ctypes.c_uint8), hi - lo, fmt, si, _ptr(out[lo:hi], ctypes.c_float)))
        else:
            jobs.append(lambda lo=lo, hi=hi: lib.fp8o_dequantize_bf16(
                _ptr(codes[lo:hi], ctypes.c_uint8), hi - lo, fmt, si, _ptr(out[lo:hi], ctypes.c_uint16)))
    _run(jobs, threads)
    return out


def amax_bits(x: np.ndarray, threads: int = 1) -> int:
    """binary32 bit pattern of max|x| (0x7FC00000 if any NaN, 0 when empty)."""
    lib = _load()
    x = np.ascontiguousarray(x).reshape(-1)
    kind = _wide_kind(x)
    parts = []
    plock = threading.Lock()

    def job(lo, hi):
        if kind == "f32":
            r = lib.fp8o_amax_f32(_ptr(x[lo:hi], ctypes.c_float), hi - lo)
        else:
            r = lib.fp8o_amax_bf16(_ptr(x[lo:hi], ctypes.c_uint16), hi - lo)
        with plock:
            parts.append(int(r))

    _run([lambda lo=lo, hi=hi: job(lo, hi) for lo, hi in _chunks(x.size, threads)], threads)
    # the maximum of chunk maxima; a NaN chunk (0x7FC00000) is above every non-NaN pattern
    return max(parts) if parts else 0


def amax(x: np.ndarray, threads: int = 1) -> np.float32:
    return np.array([amax_bits(x, threads)], dtype=np.uint32).view(np.float32)[0]


# ------------------------------------------------------- per-channel scales --

def amax_channels(x: np.ndarray, axis: int) -> np.ndarray:
    """float32 amax per channel of a 2-D array: axis 0 = one per column, axis 1 = one per row."""
    lib = _load()
    x = np.ascontiguousarray(x)
    rows, cols = x.shape
    out = np.empty(cols if axis == 0 else rows, dtype=np.uint32)
    if _wide_kind(x.reshape(-1)) == "f32":
        lib.fp8o_amax_channels_f32(_ptr(x, ctypes.c_float), rows, cols, cols, axis, _ptr(out, ctypes.c_uint32))
    else:
        lib.fp8o_amax_channels_bf16(_ptr(x, ctypes.c_uint16), rows, cols, cols, axis, _ptr(out, ctypes.c_uint32))
    return out.view(np.float32)


def scales_from_amax(amax_vec: np.ndarray, fmt: int, pow2: bool = False):
    s = np.empty(amax_vec.size, dtype=np.float32)
    si = np.empty(amax_vec.size, dtype=np.float32)
    for i, a in enumerate(np.asarray(amax_vec, dtype=np.float32).reshape(-1)):
        s[i], si[i] = scale_pow2_from_amax(a, fmt) if pow2 else scale_from_amax(a, fmt)
    return s, si


def quantize_channels(x: np.ndarray, scale_vec: np.ndarray, axis: int, fmt: int, overflow: int = SATURATE) -> np.ndarray:
    lib = _load()
    x = np.ascontiguousarray(x)
    rows, cols = x.shape
    sv = np.ascontiguousarray(scale_vec, dtype=np.float32)
    assert sv.size == (cols if axis == 0 else rows)
    out = np.empty((rows, cols), dtype=np.uint8)
    if _wide_kind(x.reshape(-1)) == "f32":
        lib.fp8o_quantize_channels_f32(_ptr(x, ctypes.c_float), rows, cols, cols, axis, _ptr(sv, ctypes.c_float), fmt, overflow,
                                       _ptr(out, ctypes.c_uint8), cols)
    else:
        lib.fp8o_quantize_channels_bf16(_ptr(x, ctypes.c_uint16), rows, cols, cols, axis, _ptr(sv, ctypes.c_float), fmt, overflow,
                                        _ptr(out, ctypes.c_uint8), cols)
    return out


def gemm_rows_colscale(A, fmt_a, a_strides, B, fmt_b, b_strides, N, K, i0, i1, sa_inv, sb_inv_vec, threads: int = 1):
    """gemm_rows with one inverse scale per column of B (per output channel)."""
    lib = _load()
    A = np.ascontiguousarray(A, dtype=np.uint8).reshape(-1)
    B = np.ascontiguousarray(B, dtype=np.uint8).reshape(-1)
    sv = np.ascontiguousarray(sb_inv_vec, dtype=np.float32)
    assert sv.size == N
    rows = i1 - i0
    ref = np.empty((rows, N), dtype=np.float64)
    sab = np.empty((rows, N), dtype=np.float64)
    sa = ctypes.c_float(np.float32(sa_inv))
    jobs = []
    for lo, hi in _chunks(rows, threads):
        jobs.append(lambda lo=lo, hi=hi: lib.fp8o_gemm_rows_colscale(
            _ptr(A, ctypes.c_uint8), fmt_a, a_strides[0], a_strides[1],
            _ptr(B, ctypes.c_uint8), fmt_b, b_strides[0], b_strides[1],
            N, K, i0 + lo, i0 + hi, sa, _ptr(sv, ctypes.c_float),
            _ptr(ref[lo:hi], ctypes.c_double), _ptr(sab[lo:hi], ctypes.c_double)))
    _run(jobs, threads)
    return ref, sab


# --------------------------------------------------------------------- GEMM --

def gemm_rows(A, fmt_a, a_strides, B, fmt_b, b_strides, N, K, i0, i1, sa_inv, sb_inv, threads: int = 1):
    """Rows [i0,i1) of (A.B)*sa_inv*sb_inv in double, plus sum|a.b|*sa_inv*sb_inv.

    ``a_strides`` = (stride of i, stride of k) and ``b_strides`` = (stride of k,
    stride of j), in elements of the flat uint8 buffers A and B."""
    lib = _load()
    A = np.ascontiguousarray(A, dtype=np.uint8).reshape(-1)
    B = np.ascontiguousarray(B, dtype=np.uint8).reshape(-1)
    rows = i1 - i0
    ref = np.empty((rows, N), dtype=np.float64)
    sab = np.empty((rows, N), dtype=np.float64)
    sa, sb = ctypes.c_float(np.float32(sa_inv)), ctypes.c_float(np.float32(sb_inv))
    jobs = []
    for lo, hi in _chunks(rows, threads):
        jobs.append(lambda lo=lo, hi=hi: lib.fp8o_gemm_rows(
            _ptr(A, ctypes.c_uint8), fmt_a, a_strides[0], a_strides[1],
            _ptr(B, ctypes.c_uint8), fmt_b, b_strides[0], b_strides[1],
            N, K, i0 + lo, i0 + hi, sa, sb,
            _ptr(ref[lo:hi], ctypes.c_double), _ptr(sab[lo:hi], ctypes.c_double)))
    _run(jobs, threads)
    return ref, sab


def gemm_samples(A, fmt_a, a_strides, B, fmt_b, b_strides, K, ii, jj, sa_inv, sb_inv, threads: int = 1):
    """The same quantities at the listed (i, j) positions."""
    lib = _load()
    A = np.ascontiguousarray(A, dtype=np.uint8).reshape(-1)
    B = np.ascontiguousarray(B, dtype=np.uint8).reshape(-1)
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    ref = np.empty(ii.size, dtype=np.float64)
    sab = np.empty(ii.size, dtype=np.float64)
    sa, sb = ctypes.c_float(np.float32(sa_inv)), ctypes.c_float(np.float32(sb_inv))
    jobs = []
    for lo, hi in _chunks(ii.size, threads):
        jobs.append(lambda lo=lo, hi=hi: lib.fp8o_gemm_samples(
            _ptr(A, ctypes.c_uint8), fmt_a, a_strides[0], a_strides[1],
            _ptr(B, ctypes.c_uint8), fmt_b, b_strides[0], b_strides[1],
            K, _ptr(ii[lo:hi], ctypes.c_int64), _ptr(jj[lo:hi], ctypes.c_int64), hi - lo, sa, sb,
            _ptr(ref[lo:hi], ctypes.c_double), _ptr(sab[lo:hi], ctypes.c_double)))
    _run(jobs, threads)
    return ref, sab


def dot_exact(a_codes, fmt_a, b_codes, fmt_b):
    """Exact dot product of two code vectors as a Python integer and a unit exponent:
    value = integer * 2**unit_exp.  Returns None when a code is NaN or Inf."""
    lib = _load()
    a = np.ascontiguousarray(a_codes, dtype=np.uint8).reshape(-1)
    b = np.ascontiguousarray(b_codes, dtype=np.uint8).reshape(-1)
    assert a.size == b.size
    hi, lo, ue = ctypes.c_int64(), ctypes.c_uint64(), ctypes.c_int()
    rc = lib.fp8o_dot_exact(_ptr(a, ctypes.c_uint8), fmt_a, 1, _ptr(b, ctypes.c_uint8), fmt_b, 1, a.size,
                            ctypes.byref(hi), ctypes.byref(lo), ctypes.byref(ue))
    if rc:
        return None
    return (int(hi.value) << 64) + int(lo.value), int(ue.value)


def round_bf16_from_f64(v: np.ndarray) -> np.ndarray:
    """Correctly rounded (single rounding) bf16 bit patterns of double values."""
    lib = _load()
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    lib.fp8o_f64_to_bf16_array(_ptr(v, ctypes.c_double), v.size, _ptr(out, ctypes.c_uint16))
    return out
