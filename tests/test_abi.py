"""The C-ABI library builds, loads, and exports every entry point the header declares.
Runs without a GPU: only calls that return before touching the device are made."""
import ctypes
import os
import re

import pytest

from paper_2209_05433_b200 import api

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "fp8_b200.h")


_keep = []


def _addresses():
    """(an aligned address, one that is not 16-byte aligned) for the argument-error calls.  Every such call fails
    validation before anything is enqueued, so the addresses are never dereferenced; on a machine with a GPU they
    still point into a real device buffer, so that even a library bug that enqueued work could not touch memory
    this process does not own."""
    try:
        import torch
        if torch.cuda.is_available():
            buf = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
            _keep.append(buf)
            return ctypes.c_void_p(buf.data_ptr()), ctypes.c_void_p(buf.data_ptr() + 8)
    except Exception:
        pass
    return ctypes.c_void_p(16), ctypes.c_void_p(24)


def _declared():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fp8_[a-z_0-9]+)\s*\(", text)))


def test_header_and_binding_name_the_same_entry_points():
    assert _declared() == sorted(api.EXPORTS)
    for name in ("fp8_amax", "fp8_scale_from_amax", "fp8_quantize", "fp8_dequantize", "fp8_gemm"):
        assert callable(getattr(api, name))


def test_library_exports_every_declared_symbol():
    lib = api.load()
    for name in _declared():
        assert hasattr(lib, name), name
    assert lib.fp8_status_string(0) == b"ok"
    assert lib.fp8_status_string(4) == b"operand not 16-byte aligned"
    assert lib.fp8_status_string(99) == b"unknown status"


def test_argument_errors_are_reported_before_any_launch():
    lib = api.load()
    one, odd = _addresses()            # never dereferenced: every call below fails validation first
    assert lib.fp8_amax(one, 0, 4, None, None) == 1                      # FP8_ERR_NULL
    assert lib.fp8_amax(one, 7, 4, one, None) == 2                       # FP8_ERR_ENUM
    assert lib.fp8_scale_from_amax(None, 0, one, one, None) == 1
    assert lib.fp8_scale_from_amax(one, 5, one, one, None) == 2
    assert lib.fp8_quantize(one, 1, 4, 0, 0, None, one, None, None) == 1
    assert lib.fp8_quantize(one, 1, 4, 3, 0, one, one, None, None) == 2
    assert lib.fp8_quantize(one, 1, 4, 0, 2, one, one, None, None) == 2
    assert lib.fp8_dequantize(one, 4, 0, None, one, 1, None) == 1
    assert lib.fp8_dequantize(one, 4, 9, one, one, 1, None) == 2
    d = api.GemmDesc(128, 128, 128, 0, 0, 0, 0, 128, 128, 128, 1)
    assert lib.fp8_gemm(None, one, one, one, one, one, None, None) == 1
    assert lib.fp8_gemm(ctypes.byref(d), one, one, one, None, one, None, None) == 1
    d.fa = 4
    assert lib.fp8_gemm(ctypes.byref(d), one, one, one, one, one, None, None) == 2
    d.fa = 0
    d.acc = 2                                                                           # not an fp8_accumulate
    assert lib.fp8_gemm(ctypes.byref(d), one, one, one, one, one, None, None) == 2
    d.acc = api.ACC_SPLIT
    d.M = -1
    assert lib.fp8_gemm(ctypes.byref(d), one, one, one, one, one, None, None) == 3       # FP8_ERR_SHAPE
    d.M = 128
    d.lda = 64                                                                          # smaller than K
    assert lib.fp8_gemm(ctypes.byref(d), one, one, one, one, one, None, None) == 3
    d.lda = 136                                                                         # not a multiple of 16
    assert lib.fp8_gemm(ctypes.byref(d), one, one, one, one, one, None, None) == 4       # FP8_ERR_ALIGN
    d.lda = 128
    assert lib.fp8_gemm(ctypes.byref(d), odd, one, one, one, one, None, None) == 4
    d.ldd = 100                                                                         # smaller than N
    assert lib.fp8_gemm(ctypes.byref(d), one, one, one, one, one, None, None) == 3


def test_argument_errors_of_the_wider_entry_points():
    lib = api.load()
    one, odd = _addresses()
    # one-launch current scaling: null pointers, enums, workspace alignment
    assert lib.fp8_quantize_current(one, 1, 4, 0, 0, one, None, one, one, one, None) == 1
    assert lib.fp8_quantize_current(one, 1, 4, 0, 0, one, one, one, one, None, None) == 1
    assert lib.fp8_quantize_current(one, 1, 4, 5, 0, one, one, one, one, one, None) == 2
    assert lib.fp8_quantize_current(one, 1, 4, 0, 0, one, one, one, one, odd, None) == 4
    assert lib.fp8_quantize_current_workspace_bytes() == 16
    assert lib.fp8_quantize_current_static(one, 1, 4, 0, 0, one, None, one, one, None) == 1
    assert lib.fp8_quantize_current_static(one, 9, 4, 0, 0, one, one, one, one, None) == 2
    # simulated FP8, power-of-two scale
    assert lib.fp8_fake_quantize(one, 1, 4, 0, 0, None, one, one, None) == 1
    assert lib.fp8_fake_quantize(one, 1, 4, 0, 7, one, one, one, None) == 2
    assert lib.fp8_scale_pow2_from_amax(one, 0, None, one, None) == 1
    assert lib.fp8_scale_pow2_from_amax(one, 3, one, one, None) == 2
    # per-channel
    assert lib.fp8_amax_channels(one, 1, 4, 4, 4, 0, None, None) == 1
    assert lib.fp8_amax_channels(one, 1, 4, 4, 4, 2, one, None) == 2
    assert lib.fp8_amax_channels(one, 1, 4, 8, 4, 0, one, None) == 3            # pitch smaller than the row
    assert lib.fp8_scales_from_amax(None, 4, 0, 0, one, one, None) == 1
    assert lib.fp8_scales_from_amax(one, -1, 0, 0, one, one, None) == 3
    assert lib.fp8_quantize_channels(one, 1, 4, 4, 4, 0, 0, 0, None, one, 4, None) == 1
    assert lib.fp8_quantize_channels(one, 1, 4, 4, 4, 0, 0, 0, one, one, 2, None) == 3
    assert lib.fp8_quantize_channels(one, 1, 4, 4, 4, 1, 4, 0, one, one, 4, None) == 2
    # quantize + transposed copy
    assert lib.fp8_quantize_transpose(one, 1, 4, 4, 4, 0, 0, one, one, 4, None, 4, None, None) == 1      # no out_t
    assert lib.fp8_quantize_transpose(one, 1, 4, 4, 4, 0, 0, None, one, 4, one, 4, None, None) == 1      # no scale
    assert lib.fp8_quantize_transpose(one, 3, 4, 4, 4, 0, 0, one, one, 4, one, 4, None, None) == 2
    assert lib.fp8_quantize_transpose(one, 1, 4, 4, 4, 0, 2, one, one, 4, one, 4, None, None) == 2
    assert lib.fp8_quantize_transpose(one, 1, 4, 8, 4, 0, 0, one, one, 8, one, 4, None, None) == 3       # ldx < cols
    assert lib.fp8_quantize_transpose(one, 1, 4, 8, 8, 0, 0, one, one, 4, one, 4, None, None) == 3       # ldo < cols
    assert lib.fp8_quantize_transpose(one, 1, 4, 8, 8, 0, 0, one, None, 0, one, 2, None, None) == 3      # ldt < rows
    assert lib.fp8_quantize_transpose(None, 1, 0, 8, 8, 0, 0, one, None, 0, None, 0, None, None) == 0    # empty: nothing touched
    # GEMM variants
    d = api.GemmDesc(256, 256, 128, 0, 0, 0, 0, 128, 128, 256, 1)
    assert lib.fp8_gemm_fp8out(ctypes.byref(d), one, one, one, 0, 0, one, one, None, None, None) == 1
    assert lib.fp8_gemm_fp8out(ctypes.byref(d), one, one, one, 2, 0, one, one, one, None, None) == 2
    assert lib.fp8_gemm_fp8out(ctypes.byref(d), one, one, one, 0, 3, one, one, one, None, None) == 2
    assert lib.fp8_gemm_channel_scales(ctypes.byref(d), one, one, one, one, None, None, None) == 1
    # split-K: null outputs, enum and shape checks come before any device work
    assert lib.fp8_gemm_splitk_workspace(ctypes.byref(d), None, None) == 1
    assert lib.fp8_gemm_splitk(None, one, one, one, one, one, None, None, 0, None) == 1
    d.acc = 7
    assert lib.fp8_gemm_splitk(ctypes.byref(d), one, one, one, one, one, None, None, 0, None) == 2
    assert lib.fp8_gemm_fp8out(ctypes.byref(d), one, one, one, 0, 0, one, one, one, None, None) == 2
    assert lib.fp8_gemm_channel_scales(ctypes.byref(d), one, one, one, one, one, None, None) == 2
    assert lib.fp8_gemm_batched(ctypes.byref(d), 1, one, 0, one, 0, one, 0, one, one, None, None) == 2
    d.acc = api.ACC_FAST
    assert lib.fp8_gemm_batched(ctypes.byref(d), -1, one, 0, one, 0, one, 0, one, one, None, None) == 3
    assert lib.fp8_gemm_batched(ctypes.byref(d), 4, one, 256 * 128, one, 256 * 128, one, 100, one, one, None, None) == 3   # members of D overlap
    assert lib.fp8_gemm_batched(ctypes.byref(d), 4, one, 0, one, 256 * 128, one, 256 * 256, one, one, None, None) == 3
    assert lib.fp8_gemm_batched(ctypes.byref(d), 4, one, 256 * 128 + 8, one, 256 * 128, one, 256 * 256, one, one, None, None) == 4
    assert lib.fp8_gemm_batched(ctypes.byref(d), 70000, one, 256 * 128, one, 256 * 128, one, 256 * 256, one, one, None, None) == 5


def test_header_is_plain_c_and_the_struct_layout_matches_the_binding(tmp_path):
    """the boundary is a C ABI: the header compiles as C11 on its own, and a C program links against the
    library by symbol name; sizes and offsets of fp8_gemm_desc equal those of the ctypes mirror"""
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    src = tmp_path / "abi_probe.c"
    src.write_text(
        '#include <stddef.h>\n#include <stdio.h>\n#include "fp8_b200.h"\n'
        "int main(void) {\n"
        "    fp8_gemm_desc d;\n"
        '    printf("%zu %zu %zu %zu %zu %zu %zu\\n", sizeof d, offsetof(fp8_gemm_desc, K), offsetof(fp8_gemm_desc, fa),\n'
        "           offsetof(fp8_gemm_desc, mb), offsetof(fp8_gemm_desc, lda), offsetof(fp8_gemm_desc, out), offsetof(fp8_gemm_desc, acc));\n"
        '    printf("%s\\n", fp8_status_string(FP8_ERR_ALIGN));\n'
        "    return fp8_amax(NULL, FP8_BF16, 4, NULL, NULL) == FP8_ERR_NULL ? 0 : 1;\n"
        "}\n")
    exe = tmp_path / "abi_probe"
    lib_dir = os.path.dirname(api.library_path())
    api.load()                                  # builds the library if it is missing
    subprocess.check_call([gcc, "-std=c11", "-Wall", "-Werror", "-pedantic", "-I", os.path.join(ROOT, "include"), str(src),
                           "-o", str(exe), "-L", lib_dir, "-l:libfp8_b200.so", "-Wl,-rpath," + lib_dir])
    out = subprocess.run([str(exe)], capture_output=True, text=True)
    assert out.returncode == 0, out.stderr
    sizes, msg = out.stdout.strip().split("\n")
    G = api.GemmDesc
    assert [int(v) for v in sizes.split()] == [ctypes.sizeof(G), G.K.offset, G.fa.offset, G.mb.offset, G.lda.offset, G.out.offset, G.acc.offset]
    assert msg == "operand not 16-byte aligned"
