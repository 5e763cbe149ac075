"""fp8_quantize_current_static: the one-launch current-scaling conversion for callers that cannot
allocate device memory (its control words live in a small array inside the library).

Collected last on purpose: if this file fails, a run that stops at the first failure has already run
every other test.  The check is against the existing entry point fp8_quantize_current, bit for bit
(the tolerance every cast test uses), on two calls in a row, through the C ABI; one case is also compared
directly with the CPU oracle."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, to_np_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _scalars():
    return [torch.full((1,), -1.0, dtype=torch.float32, device=DEV) for _ in range(3)]


def _run_pair(x, fmt, overflow):
    n = x.numel()
    ref_codes = torch.empty(n, dtype=torch.uint8, device=DEV)
    ra, rs, rsi = _scalars()
    api.fp8_quantize_current(x, fmt, ref_codes, ra, rs, rsi, overflow)
    codes = torch.full((n + 32,), 0x5A, dtype=torch.uint8, device=DEV)
    a, s, si = _scalars()
    api.fp8_quantize_current_static(x, fmt, codes[:n], a, s, si, overflow)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert torch.equal(codes[:n], ref_codes)
    assert bool((codes[n:] == 0x5A).all())
    for got, want in ((a, ra), (s, rs), (si, rsi)):
        assert got.view(torch.int32).item() == want.view(torch.int32).item()


@pytest.mark.parametrize("wide", [torch.bfloat16, torch.float32])
def test_static_scratch_variant_matches_workspace_variant_twice_in_a_row(wide):
    x1 = synth.activations((1 << 22) + 5, 3, dtype=wide, device=DEV)
    x2 = synth.gradients(777777, 4, dtype=wide, device=DEV)          # a different tensor, size and amax
    _run_pair(x1, api.E4M3, api.SATURATE)
    _run_pair(x2, api.E5M2, api.SATURATE)                            # second call right after the first
    _run_pair(x1, api.E4M3, api.NOSAT)
    # back-to-back on one stream without any host synchronisation in between
    n = x2.numel()
    outs = [torch.empty(n, dtype=torch.uint8, device=DEV) for _ in range(2)]
    sc = [_scalars() for _ in range(2)]
    for o, (a, s, si) in zip(outs, sc):
        api.fp8_quantize_current_static(x2, api.E5M2, o, a, s, si)
    ref = torch.empty(n, dtype=torch.uint8, device=DEV)
    ra, rs, rsi = _scalars()
    api.fp8_quantize_current(x2, api.E5M2, ref, ra, rs, rsi)
    torch.cuda.synchronize()
    for o, (a, s, si) in zip(outs, sc):
        assert torch.equal(o, ref) and a.item() == ra.item() and s.item() == rs.item() and si.item() == rsi.item()


def test_static_scratch_variant_matches_the_oracle():
    x = synth.gradients((1 << 21) + 3, 9, dtype=torch.bfloat16, device=DEV)
    codes = torch.empty(x.numel(), dtype=torch.uint8, device=DEV)
    a, s, si = _scalars()
    api.fp8_quantize_current_static(x, api.E5M2, codes, a, s, si)
    torch.cuda.synchronize()
    xh = to_np_bits(x)
    want_amax = oracle.amax(xh, THREADS)
    ws, wsi = oracle.scale_from_amax(want_amax, oracle.E5M2)
    assert a.item() == want_amax and s.item() == ws and si.item() == wsi
    assert np.array_equal(codes.cpu().numpy(), oracle.quantize(xh, ws, oracle.E5M2, threads=THREADS))


def test_static_scratch_variant_edge_sizes_and_limit():
    for n in (0, 1, 9, 4099):
        x = synth.activations(n, 5, dtype=torch.bfloat16, device=DEV)
        _run_pair(x, api.E4M3, api.SATURATE)
    # beyond the stated maximum: refused on the host, nothing is enqueued or dereferenced
    lib = api.load()
    buf = torch.zeros(4096, dtype=torch.uint8, device=DEV)              # a real buffer: the call is refused before it is used
    one = ctypes.c_void_p(buf.data_ptr())
    too_many = ctypes.c_size_t(api.STATIC_MAX_ELEMENTS + 1)
    status = lib.fp8_quantize_current_static(one, api.BF16, too_many, api.E4M3, api.SATURATE, one, one, one, one, None)
    assert status == 5 and lib.fp8_status_string(status) == b"unsupported size"
