"""The library's bounded device-side waits, made to run out on purpose.

Every wait a kernel of the library performs (the mbarrier waits of the GEMM roles, the grid barrier of the
one-launch current scaling) counts SM clocks and gives up after a limit.  The self-test entry point launches
a kernel whose wait can never be satisfied, with a limit of about a millisecond: the kernel returns by
itself, the host reads FP8_ERR_TIMEOUT with the code of the wait, the latch clears, and the same stream goes
on to produce bit-exact results.  Nothing here faults, traps or waits without a limit."""
import time

import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, to_np_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
LIMIT = 2_000_000           # SM clocks: about a millisecond


def _scalars(k=3):
    return [torch.zeros(1, dtype=torch.float32, device=DEV) for _ in range(k)]


def _expire(which, code):
    torch.cuda.synchronize()
    assert api.fp8_async_status() == (0, 0)
    t0 = time.perf_counter()
    api.fp8_self_test_expire_wait(which, LIMIT)
    st, detail = api.fp8_async_status()                  # synchronises: the kernel has returned by itself
    dt = time.perf_counter() - t0
    assert (st, detail) == (api.TIMEOUT, code)
    assert dt < 1.0, "a wait of about a millisecond took %.3f s" % dt
    assert api.fp8_async_status() == (0, 0)              # the latch was cleared by the read


def _cast_is_bit_exact(entry):
    x = synth.activations((1 << 20) + 13, 11, dtype=torch.bfloat16, device=DEV)
    codes = torch.empty(x.numel(), dtype=torch.uint8, device=DEV)
    a, s, si = _scalars()
    entry(x, api.E4M3, codes, a, s, si)
    torch.cuda.synchronize()
    xh = to_np_bits(x)
    ws, wsi = oracle.scale_from_amax(oracle.amax(xh, THREADS), oracle.E4M3)
    assert s.item() == ws and si.item() == wsi
    assert np.array_equal(codes.cpu().numpy(), oracle.quantize(xh, ws, oracle.E4M3, threads=THREADS))


def test_mbarrier_wait_gives_up_and_the_gemm_still_works():
    _expire(api.WAIT_MBARRIER, 9)
    # the next GEMM on the same stream: exact against the oracle (small integers: every sum is exact in fp32)
    rng = np.random.default_rng(5)
    M, N, K = 384, 512, 640
    A = oracle.quantize(rng.integers(-4, 5, size=(M, K)).astype(np.float32), 1.0, oracle.E4M3).reshape(M, K)
    B = oracle.quantize(rng.integers(-4, 5, size=(N, K)).astype(np.float32), 1.0, oracle.E4M3).reshape(N, K)
    D = torch.empty(M, N, dtype=torch.float32, device=DEV)
    one = torch.ones(1, dtype=torch.float32, device=DEV)
    api.fp8_gemm(torch.from_numpy(A).to(DEV), api.E4M3, api.MAJOR_K, torch.from_numpy(B).to(DEV), api.E4M3, api.MAJOR_K, D, one, one)
    torch.cuda.synchronize()
    assert api.fp8_async_status() == (0, 0)
    ref, _ = oracle.gemm_rows(A, oracle.E4M3, (K, 1), B, oracle.E4M3, (1, K), N, K, 0, M, 1.0, 1.0, threads=THREADS)
    assert np.array_equal(D.cpu().numpy().astype(np.float64), ref)


def test_grid_barrier_gives_up_and_both_one_launch_variants_still_work():
    # a normal call first, so that the cached workspace of this stream exists and is in use
    _cast_is_bit_exact(api.fp8_quantize_current)
    _expire(api.WAIT_GRID_BARRIER, 16)
    # the variant that shares the control words with the self-test clears them itself before every call
    _cast_is_bit_exact(api.fp8_quantize_current_static)
    # the caller-workspace variant: its workspace was not involved; and had it been, the kernel leaves it zeroed
    ws = api.current_scaling_workspace(torch.device(DEV, torch.cuda.current_device()))
    assert int(ws.view(torch.int32).abs().sum().item()) == 0
    _cast_is_bit_exact(api.fp8_quantize_current)
    _expire(api.WAIT_GRID_BARRIER, 16)                   # and again: the self-test is repeatable
    _cast_is_bit_exact(api.fp8_quantize_current_static)


def test_self_test_rejects_bad_arguments():
    lib = api.load()
    assert lib.fp8_self_test_expire_wait(2, LIMIT, None) == 2            # not an fp8_wait_kind
    assert lib.fp8_self_test_expire_wait(0, 0, None) == 5                # no limit
    assert lib.fp8_self_test_expire_wait(1, 3_000_000_000, None) == 5    # longer than about a second
    torch.cuda.synchronize()
    assert api.fp8_async_status() == (0, 0)


def test_sm_clock_probe_reports_a_plausible_clock_and_is_bounded():
    out = torch.zeros(2, dtype=torch.int64, device=DEV)
    t0 = time.perf_counter()
    api.fp8_sm_clock_probe(out, 300)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0
    clocks, ns = (int(v) for v in out.cpu())
    assert 250_000 <= ns <= 5_000_000, ns                       # about the 300 us asked for
    mhz = clocks * 1000.0 / ns
    assert 100.0 < mhz < 3000.0, mhz
    lib = api.load()
    assert lib.fp8_sm_clock_probe(None, 100, None) == 1
    assert lib.fp8_sm_clock_probe(out.data_ptr(), 0, None) == 5 and lib.fp8_sm_clock_probe(out.data_ptr(), 200000, None) == 5
