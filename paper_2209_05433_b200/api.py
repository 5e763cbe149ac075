"""Python binding of the fp8_b200 C ABI (include/fp8_b200.h).

Argument marshalling only: every function checks dtypes, takes `data_ptr()` of
torch CUDA tensors, passes torch's current stream and calls the entry point of
the same name in ``libfp8_b200.so``.  There is no fallback: if the library is
not built, or a call returns a non-zero status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import _build

E4M3, E5M2 = 0, 1            # fp8_format
F32, BF16 = 0, 1             # fp8_wide
SATURATE, NOSAT = 0, 1       # fp8_overflow
MAJOR_K, MAJOR_MN = 0, 1     # fp8_major
ACC_SPLIT, ACC_FAST = 0, 1    # fp8_accumulate: bounded error for any data (default) / one accumulator

EXPORTS = ["fp8_amax", "fp8_scale_from_amax", "fp8_quantize", "fp8_quantize_current",
           "fp8_quantize_current_workspace_bytes", "fp8_quantize_current_static", "fp8_dequantize", "fp8_fake_quantize",
           "fp8_scale_pow2_from_amax", "fp8_gemm", "fp8_gemm_fp8out", "fp8_amax_channels", "fp8_scales_from_amax",
           "fp8_quantize_channels", "fp8_quantize_transpose", "fp8_gemm_channel_scales", "fp8_gemm_batched",
           "fp8_gemm_splitk", "fp8_gemm_splitk_workspace",
           "fp8_async_status", "fp8_self_test_expire_wait", "fp8_sm_clock_probe", "fp8_status_string", "fp8_launch_count"]


class Fp8Error(RuntimeError):
    pass


class GemmDesc(ctypes.Structure):
    _fields_ = [("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("fa", ctypes.c_int), ("fb", ctypes.c_int), ("ma", ctypes.c_int), ("mb", ctypes.c_int),
                ("lda", ctypes.c_int64), ("ldb", ctypes.c_int64), ("ldd", ctypes.c_int64), ("out", ctypes.c_int), ("acc", ctypes.c_int)]


_lib = None


def library_path() -> str:
    return _build.LIB


def load(build_if_missing: bool = True) -> ctypes.CDLL:
    """Loads libfp8_b200.so (building it with nvcc when it is missing or stale)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if build_if_missing and _build.is_stale():
        try:
            _build.build_library()
        except Exception as e:
            if not os.path.exists(path):     # stale is tolerable, missing is not
                raise Fp8Error("libfp8_b200.so is missing and could not be built: %s" % e) from e
    if not os.path.exists(path):
        raise Fp8Error("libfp8_b200.so not found at %s; run `python -m paper_2209_05433_b200._build`" % path)
    lib = ctypes.CDLL(path)
    vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    lib.fp8_amax.restype = i32
    lib.fp8_amax.argtypes = [vp, i32, sz, vp, vp]
    lib.fp8_scale_from_amax.restype = i32
    lib.fp8_scale_from_amax.argtypes = [vp, i32, vp, vp, vp]
    lib.fp8_quantize.restype = i32
    lib.fp8_quantize.argtypes = [vp, i32, sz, i32, i32, vp, vp, vp, vp]
    lib.fp8_quantize_current.restype = i32
    lib.fp8_quantize_current.argtypes = [vp, i32, sz, i32, i32, vp, vp, vp, vp, vp, vp]
    lib.fp8_quantize_current_workspace_bytes.restype = sz
    lib.fp8_quantize_current_workspace_bytes.argtypes = []
    lib.fp8_quantize_current_static.restype = i32
    lib.fp8_quantize_current_static.argtypes = [vp, i32, sz, i32, i32, vp, vp, vp, vp, vp]
    lib.fp8_dequantize.restype = i32
    lib.fp8_dequantize.argtypes = [vp, sz, i32, vp, vp, i32, vp]
    lib.fp8_fake_quantize.restype = i32
    lib.fp8_fake_quantize.argtypes = [vp, i32, sz, i32, i32, vp, vp, vp, vp]
    lib.fp8_scale_pow2_from_amax.restype = i32
    lib.fp8_scale_pow2_from_amax.argtypes = [vp, i32, vp, vp, vp]
    lib.fp8_gemm.restype = i32
    lib.fp8_gemm.argtypes = [ctypes.POINTER(GemmDesc), vp, vp, vp, vp, vp, vp, vp]
    lib.fp8_gemm_fp8out.restype = i32
    lib.fp8_gemm_fp8out.argtypes = [ctypes.POINTER(GemmDesc), vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
    i64 = ctypes.c_int64
    lib.fp8_amax_channels.restype = i32
    lib.fp8_amax_channels.argtypes = [vp, i32, i64, i64, i64, i32, vp, vp]
    lib.fp8_scales_from_amax.restype = i32
    lib.fp8_scales_from_amax.argtypes = [vp, i64, i32, i32, vp, vp, vp]
    lib.fp8_quantize_channels.restype = i32
    lib.fp8_quantize_channels.argtypes = [vp, i32, i64, i64, i64, i32, i32, i32, vp, vp, i64, vp]
    lib.fp8_quantize_transpose.restype = i32
    lib.fp8_quantize_transpose.argtypes = [vp, i32, i64, i64, i64, i32, i32, vp, vp, i64, vp, i64, vp, vp]
    lib.fp8_gemm_channel_scales.restype = i32
    lib.fp8_gemm_channel_scales.argtypes = [ctypes.POINTER(GemmDesc), vp, vp, vp, vp, vp, vp, vp]
    lib.fp8_gemm_batched.restype = i32
    lib.fp8_gemm_batched.argtypes = [ctypes.POINTER(GemmDesc), i64, vp, i64, vp, i64, vp, i64, vp, vp, vp, vp]
    lib.fp8_gemm_splitk_workspace.restype = i32
    lib.fp8_gemm_splitk_workspace.argtypes = [ctypes.POINTER(GemmDesc), ctypes.POINTER(ctypes.c_int), ctypes.POINTER(sz)]
    lib.fp8_gemm_splitk.restype = i32
    lib.fp8_gemm_splitk.argtypes = [ctypes.POINTER(GemmDesc), vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.fp8_async_status.restype = i32
    lib.fp8_async_status.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
    lib.fp8_self_test_expire_wait.restype = i32
    lib.fp8_self_test_expire_wait.argtypes = [i32, ctypes.c_uint64, vp]
    lib.fp8_sm_clock_probe.restype = i32
    lib.fp8_sm_clock_probe.argtypes = [vp, ctypes.c_uint32, vp]
    lib.fp8_status_string.restype = ctypes.c_char_p
    lib.fp8_status_string.argtypes = [i32]
    lib.fp8_launch_count.restype = ctypes.c_uint64
    lib.fp8_launch_count.argtypes = []
    _lib = lib
    return lib


def _check(status: int, what: str) -> None:
    if status != 0:
        raise Fp8Error("%s failed: %s (status %d)" % (what, load().fp8_status_string(status).decode(), status))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _wide_of(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("wide tensors must be float32 or bfloat16, got %s" % t.dtype)


def _dev(t: torch.Tensor, name: str) -> int:
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor" % name)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return t.data_ptr()


def _scalar(t: torch.Tensor, name: str) -> int:
    if t.dtype != torch.float32 or t.numel() != 1:
        raise TypeError("%s must be a one-element float32 CUDA tensor" % name)
    return _dev(t, name)


def fp8_amax(x: torch.Tensor, amax_out: torch.Tensor) -> None:
    _check(load().fp8_amax(_dev(x, "x"), _wide_of(x), x.numel(), _scalar(amax_out, "amax_out"), _stream()), "fp8_amax")


def fp8_scale_from_amax(amax: torch.Tensor, fmt: int, scale_out: torch.Tensor, scale_inv_out: torch.Tensor) -> None:
    _check(load().fp8_scale_from_amax(_scalar(amax, "amax"), fmt, _scalar(scale_out, "scale_out"),
                                      _scalar(scale_inv_out, "scale_inv_out"), _stream()), "fp8_scale_from_amax")


def fp8_quantize(x: torch.Tensor, fmt: int, scale: torch.Tensor, out: torch.Tensor,
                 overflow: int = SATURATE, amax_out: torch.Tensor | None = None) -> None:
    if out.dtype != torch.uint8 or out.numel() != x.numel():
        raise TypeError("out must be a uint8 tensor with as many elements as x")
    _check(load().fp8_quantize(_dev(x, "x"), _wide_of(x), x.numel(), fmt, overflow, _scalar(scale, "scale"),
                               _dev(out, "out"), None if amax_out is None else _scalar(amax_out, "amax_out"),
                               _stream()), "fp8_quantize")


_workspaces: dict = {}


def current_scaling_workspace(device: torch.device) -> torch.Tensor:
    """A zeroed workspace for fp8_quantize_current on `device`, made once per (device, stream)."""
    key = (device.index if device.index is not None else torch.cuda.current_device(), _stream())
    ws = _workspaces.get(key)
    if ws is None:
        nbytes = int(load().fp8_quantize_current_workspace_bytes())
        ws = torch.zeros(max(nbytes, 16), dtype=torch.uint8, device=device)
        _workspaces[key] = ws
    return ws


def fp8_quantize_current(x: torch.Tensor, fmt: int, out: torch.Tensor, amax_out: torch.Tensor, scale_out: torch.Tensor,
                         scale_inv_out: torch.Tensor, overflow: int = SATURATE, workspace: torch.Tensor | None = None) -> None:
    if out.dtype != torch.uint8 or out.numel() != x.numel():
        raise TypeError("out must be a uint8 tensor with as many elements as x")
    ws = current_scaling_workspace(x.device) if workspace is None else workspace
    _check(load().fp8_quantize_current(_dev(x, "x"), _wide_of(x), x.numel(), fmt, overflow, _dev(out, "out"),
                                       _scalar(amax_out, "amax_out"), _scalar(scale_out, "scale_out"),
                                       _scalar(scale_inv_out, "scale_inv_out"), _dev(ws, "workspace"), _stream()),
           "fp8_quantize_current")


STATIC_MAX_ELEMENTS = 1 << 32


def fp8_quantize_current_static(x: torch.Tensor, fmt: int, out: torch.Tensor, amax_out: torch.Tensor,
                                scale_out: torch.Tensor, scale_inv_out: torch.Tensor, overflow: int = SATURATE) -> None:
    """fp8_quantize_current for callers that cannot allocate a workspace: the kernel's control words
    live in a small array inside the library.  Calls that overlap on the GPU race on that array."""
    if out.dtype != torch.uint8 or out.numel() != x.numel():
        raise TypeError("out must be a uint8 tensor with as many elements as x")
    _check(load().fp8_quantize_current_static(_dev(x, "x"), _wide_of(x), x.numel(), fmt, overflow, _dev(out, "out"),
                                              _scalar(amax_out, "amax_out"), _scalar(scale_out, "scale_out"),
                                              _scalar(scale_inv_out, "scale_inv_out"), _stream()),
           "fp8_quantize_current_static")


def fp8_dequantize(codes: torch.Tensor, fmt: int, scale_inv: torch.Tensor, out: torch.Tensor) -> None:
    if codes.dtype != torch.uint8 or out.numel() != codes.numel():
        raise TypeError("codes must be uint8 and out must have as many elements")
    _check(load().fp8_dequantize(_dev(codes, "codes"), codes.numel(), fmt, _scalar(scale_inv, "scale_inv"),
                                 _dev(out, "out"), _wide_of(out), _stream()), "fp8_dequantize")


def fp8_fake_quantize(x: torch.Tensor, fmt: int, scale: torch.Tensor, scale_inv: torch.Tensor, out: torch.Tensor,
                      overflow: int = SATURATE) -> None:
    if out.dtype != x.dtype or out.numel() != x.numel():
        raise TypeError("out must have the dtype and size of x")
    _check(load().fp8_fake_quantize(_dev(x, "x"), _wide_of(x), x.numel(), fmt, overflow, _scalar(scale, "scale"),
                                    _scalar(scale_inv, "scale_inv"), _dev(out, "out"), _stream()), "fp8_fake_quantize")


def fp8_scale_pow2_from_amax(amax: torch.Tensor, fmt: int, scale_out: torch.Tensor, scale_inv_out: torch.Tensor) -> None:
    _check(load().fp8_scale_pow2_from_amax(_scalar(amax, "amax"), fmt, _scalar(scale_out, "scale_out"),
                                           _scalar(scale_inv_out, "scale_inv_out"), _stream()), "fp8_scale_pow2_from_amax")


def fp8_gemm(A: torch.Tensor, fa: int, ma: int, B: torch.Tensor, fb: int, mb: int, D: torch.Tensor,
             scale_inv_a: torch.Tensor, scale_inv_b: torch.Tensor, amax_out: torch.Tensor | None = None,
             acc: int = ACC_SPLIT) -> None:
    """D[M,N] = (A[M,K] . B[K,N]) * scale_inv_a * scale_inv_b.

    A is a 2-D uint8 tensor stored [M,K] when ``ma == MAJOR_K`` or [K,M] when
    ``ma == MAJOR_MN``; B is stored [N,K] when ``mb == MAJOR_K`` or [K,N] when
    ``mb == MAJOR_MN``.  Row pitches are taken from the tensors' strides.
    ``acc``: ACC_SPLIT (default) adds partial sums every 2048 of K in registers (tolerance met on any data at any
    K); ACC_FAST keeps one accumulator over all of K (a few per cent faster; for zero-mean operands)."""
    d = _gemm_desc_2d(A, ma, B, mb, D, fa, fb, acc)
    _check(load().fp8_gemm(ctypes.byref(d), A.data_ptr(), B.data_ptr(), D.data_ptr(),
                           _scalar(scale_inv_a, "scale_inv_a"), _scalar(scale_inv_b, "scale_inv_b"),
                           None if amax_out is None else _scalar(amax_out, "amax_out"), _stream()), "fp8_gemm")


def _gemm_desc_2d(A, ma, B, mb, D, fa, fb, acc, codes_out=False):
    """descriptor of a 2-D product from the tensors' shapes and strides; D is a wide tensor, or uint8 codes"""
    if A.dtype != torch.uint8 or B.dtype != torch.uint8 or A.dim() != 2 or B.dim() != 2 or D.dim() != 2 or (codes_out and D.dtype != torch.uint8):
        raise TypeError("A and B must be 2-D uint8 tensors and D a 2-D %s tensor" % ("uint8" if codes_out else "float32 or bfloat16"))
    for t, name in ((A, "A"), (B, "B"), (D, "D")):
        if not t.is_cuda or t.stride(1) != 1:
            raise ValueError("%s must be a CUDA tensor with unit inner stride" % name)
    M, K = (A.shape[0], A.shape[1]) if ma == MAJOR_K else (A.shape[1], A.shape[0])
    Kb, N = (B.shape[1], B.shape[0]) if mb == MAJOR_K else (B.shape[0], B.shape[1])
    if K != Kb or tuple(D.shape) != (M, N):
        raise ValueError("shape mismatch: A gives M=%d K=%d, B gives K=%d N=%d, D is %s" % (M, K, Kb, N, tuple(D.shape)))
    return GemmDesc(M, N, K, fa, fb, ma, mb, A.stride(0), B.stride(0), D.stride(0), BF16 if codes_out else _wide_of(D), acc)


def fp8_gemm_splitk_workspace(M: int, N: int, K: int) -> tuple[int, int]:
    """(number of K-slices, workspace bytes) fp8_gemm_splitk uses for this shape on the current device"""
    d = GemmDesc(M, N, K, E4M3, E4M3, MAJOR_K, MAJOR_K, K, K, N, BF16, ACC_FAST)
    splits, nbytes = ctypes.c_int(0), ctypes.c_size_t(0)
    _check(load().fp8_gemm_splitk_workspace(ctypes.byref(d), ctypes.byref(splits), ctypes.byref(nbytes)), "fp8_gemm_splitk_workspace")
    return splits.value, nbytes.value


def fp8_gemm_splitk(A: torch.Tensor, fa: int, ma: int, B: torch.Tensor, fb: int, mb: int, D: torch.Tensor,
                    scale_inv_a: torch.Tensor, scale_inv_b: torch.Tensor, workspace: torch.Tensor | None,
                    amax_out: torch.Tensor | None = None, acc: int = ACC_SPLIT) -> None:
    """fp8_gemm with the contraction cut into slices when the problem has few output tiles; ``workspace`` is a
    CUDA tensor of at least fp8_gemm_splitk_workspace(M, N, K)[1] bytes (None when that is 0)."""
    d = _gemm_desc_2d(A, ma, B, mb, D, fa, fb, acc)
    ws_ptr, ws_bytes = (None, 0) if workspace is None else (workspace.data_ptr(), workspace.numel() * workspace.element_size())
    _check(load().fp8_gemm_splitk(ctypes.byref(d), A.data_ptr(), B.data_ptr(), D.data_ptr(),
                                  _scalar(scale_inv_a, "scale_inv_a"), _scalar(scale_inv_b, "scale_inv_b"),
                                  None if amax_out is None else _scalar(amax_out, "amax_out"), ws_ptr, ws_bytes, _stream()),
           "fp8_gemm_splitk")


def fp8_gemm_fp8out(A: torch.Tensor, fa: int, ma: int, B: torch.Tensor, fb: int, mb: int, D: torch.Tensor, fd: int,
                    scale_inv_a: torch.Tensor, scale_inv_b: torch.Tensor, scale_d: torch.Tensor,
                    amax_out: torch.Tensor | None = None, overflow: int = SATURATE, acc: int = ACC_SPLIT) -> None:
    """D[M,N] (uint8 codes of format fd) = encode((A . B) * scale_inv_a * scale_inv_b * scale_d); amax_out
    receives the amax of the result before the output scale and conversion.  Layout rules as fp8_gemm."""
    d = _gemm_desc_2d(A, ma, B, mb, D, fa, fb, acc, codes_out=True)
    _check(load().fp8_gemm_fp8out(ctypes.byref(d), A.data_ptr(), B.data_ptr(), D.data_ptr(), fd, overflow,
                                  _scalar(scale_inv_a, "scale_inv_a"), _scalar(scale_inv_b, "scale_inv_b"),
                                  _scalar(scale_d, "scale_d"), None if amax_out is None else _scalar(amax_out, "amax_out"),
                                  _stream()), "fp8_gemm_fp8out")


def _vec(t: torch.Tensor, count: int, name: str) -> int:
    if t.dtype != torch.float32 or t.numel() != count:
        raise TypeError("%s must be a float32 CUDA tensor with %d elements" % (name, count))
    return _dev(t, name)


def _rows2d(t: torch.Tensor, name: str):
    if t.dim() != 2 or not t.is_cuda or t.stride(1) != 1:
        raise ValueError("%s must be a 2-D CUDA tensor with unit inner stride" % name)
    return t.shape[0], t.shape[1], t.stride(0)


def fp8_amax_channels(x: torch.Tensor, axis: int, amax_vec: torch.Tensor) -> None:
    rows, cols, ld = _rows2d(x, "x")
    _check(load().fp8_amax_channels(x.data_ptr(), _wide_of(x), rows, cols, ld, axis,
                                    _vec(amax_vec, cols if axis == 0 else rows, "amax_vec"), _stream()), "fp8_amax_channels")


def fp8_scales_from_amax(amax_vec: torch.Tensor, fmt: int, scale_vec: torch.Tensor, scale_inv_vec: torch.Tensor, pow2: bool = False) -> None:
    n = amax_vec.numel()
    _check(load().fp8_scales_from_amax(_vec(amax_vec, n, "amax_vec"), n, fmt, 1 if pow2 else 0, _vec(scale_vec, n, "scale_vec"),
                                       _vec(scale_inv_vec, n, "scale_inv_vec"), _stream()), "fp8_scales_from_amax")


def fp8_quantize_channels(x: torch.Tensor, axis: int, fmt: int, scale_vec: torch.Tensor, out: torch.Tensor, overflow: int = SATURATE) -> None:
    rows, cols, ld = _rows2d(x, "x")
    orows, ocols, ld_out = _rows2d(out, "out")
    if out.dtype != torch.uint8 or (orows, ocols) != (rows, cols):
        raise TypeError("out must be a uint8 tensor of the shape of x")
    _check(load().fp8_quantize_channels(x.data_ptr(), _wide_of(x), rows, cols, ld, axis, fmt, overflow,
                                        _vec(scale_vec, cols if axis == 0 else rows, "scale_vec"), out.data_ptr(), ld_out, _stream()),
           "fp8_quantize_channels")


def fp8_quantize_transpose(x: torch.Tensor, fmt: int, scale: torch.Tensor, out: torch.Tensor | None, out_t: torch.Tensor,
                           amax_out: torch.Tensor | None = None, overflow: int = SATURATE) -> None:
    """codes of the 2-D tensor x in both orientations from one pass: ``out`` [rows, cols] (or None) and
    ``out_t`` [cols, rows]; ``amax_out`` optionally receives amax of x."""
    rows, cols, ldx = _rows2d(x, "x")
    trows, tcols, ldt = _rows2d(out_t, "out_t")
    if out_t.dtype != torch.uint8 or (trows, tcols) != (cols, rows):
        raise TypeError("out_t must be a uint8 tensor of the transposed shape of x")
    ldo = 0
    if out is not None:
        orows, ocols, ldo = _rows2d(out, "out")
        if out.dtype != torch.uint8 or (orows, ocols) != (rows, cols):
            raise TypeError("out must be a uint8 tensor of the shape of x")
    _check(load().fp8_quantize_transpose(x.data_ptr(), _wide_of(x), rows, cols, ldx, fmt, overflow, _scalar(scale, "scale"),
                                         None if out is None else out.data_ptr(), ldo, out_t.data_ptr(), ldt,
                                         None if amax_out is None else _scalar(amax_out, "amax_out"), _stream()),
           "fp8_quantize_transpose")


def fp8_gemm_channel_scales(A: torch.Tensor, fa: int, ma: int, B: torch.Tensor, fb: int, mb: int, D: torch.Tensor,
                            scale_inv_a: torch.Tensor, scale_inv_b_vec: torch.Tensor, amax_out: torch.Tensor | None = None,
                            acc: int = ACC_SPLIT) -> None:
    """fp8_gemm with one inverse scale per column of B (per output channel)."""
    d = _gemm_desc_2d(A, ma, B, mb, D, fa, fb, acc)
    _check(load().fp8_gemm_channel_scales(ctypes.byref(d), A.data_ptr(), B.data_ptr(), D.data_ptr(),
                                          _scalar(scale_inv_a, "scale_inv_a"), _vec(scale_inv_b_vec, d.N, "scale_inv_b_vec"),
                                          None if amax_out is None else _scalar(amax_out, "amax_out"), _stream()),
           "fp8_gemm_channel_scales")


def fp8_gemm_batched(A: torch.Tensor, fa: int, ma: int, B: torch.Tensor, fb: int, mb: int, D: torch.Tensor,
                     scale_inv_a: torch.Tensor, scale_inv_b: torch.Tensor, amax_out: torch.Tensor | None = None,
                     acc: int = ACC_SPLIT) -> None:
    """Batched fp8_gemm: A, B are 3-D uint8 tensors [batch, rows, cols] (layouts per member as fp8_gemm), D is
    [batch, M, N]; the batch strides are taken from the tensors."""
    if A.dtype != torch.uint8 or B.dtype != torch.uint8 or A.dim() != 3 or B.dim() != 3 or D.dim() != 3:
        raise TypeError("A and B must be 3-D uint8 tensors and D a 3-D tensor")
    for t, name in ((A, "A"), (B, "B"), (D, "D")):
        if not t.is_cuda or t.stride(2) != 1:
            raise ValueError("%s must be a CUDA tensor with unit inner stride" % name)
    batch = A.shape[0]
    M, K = (A.shape[1], A.shape[2]) if ma == MAJOR_K else (A.shape[2], A.shape[1])
    Kb, N = (B.shape[2], B.shape[1]) if mb == MAJOR_K else (B.shape[1], B.shape[2])
    if K != Kb or B.shape[0] != batch or tuple(D.shape) != (batch, M, N):
        raise ValueError("shape mismatch")
    d = GemmDesc(M, N, K, fa, fb, ma, mb, A.stride(1), B.stride(1), D.stride(1), _wide_of(D), acc)
    _check(load().fp8_gemm_batched(ctypes.byref(d), batch, A.data_ptr(), A.stride(0), B.data_ptr(), B.stride(0),
                                   D.data_ptr(), D.stride(0), _scalar(scale_inv_a, "scale_inv_a"), _scalar(scale_inv_b, "scale_inv_b"),
                                   None if amax_out is None else _scalar(amax_out, "amax_out"), _stream()), "fp8_gemm_batched")


TIMEOUT = 7                                   # FP8_ERR_TIMEOUT
WAIT_MBARRIER, WAIT_GRID_BARRIER = 0, 1       # fp8_wait_kind


def fp8_async_status() -> tuple[int, int]:
    """(status, detail) of the device-side error latch; synchronises the device.  After a time-out the cached
    current-scaling workspaces are cleared again (the kernel leaves them zeroed; this costs nothing and does not
    rely on it)."""
    detail = ctypes.c_uint32(0)
    s = load().fp8_async_status(ctypes.byref(detail))
    if int(s) == TIMEOUT:
        for ws in _workspaces.values():
            ws.zero_()
        torch.cuda.synchronize()
    return int(s), int(detail.value)


def fp8_self_test_expire_wait(which: int, limit_cycles: int = 2_000_000) -> None:
    """Makes one bounded device-side wait run out on purpose (about a millisecond by default); see the header."""
    _check(load().fp8_self_test_expire_wait(which, limit_cycles, _stream()), "fp8_self_test_expire_wait")


def fp8_sm_clock_probe(out: torch.Tensor, duration_us: int = 200) -> None:
    """Enqueues the one-warp clock probe on the current stream; `out` is a 2-element int64 CUDA tensor that receives
    (SM clocks, nanoseconds) of a window of `duration_us` microseconds."""
    if out.dtype != torch.int64 or out.numel() != 2:
        raise TypeError("out must be a 2-element int64 CUDA tensor")
    _check(load().fp8_sm_clock_probe(_dev(out, "out"), duration_us, _stream()), "fp8_sm_clock_probe")


def fp8_launch_count() -> int:
    return int(load().fp8_launch_count())
