"""Extreme extents: tensors of more than 2^32 elements through the cast kernels (64-bit indexing end to end),
a contraction of 2^20 terms and an output of 2^20 rows through the GEMM.  Checked against the oracle on
slices and samples it can compute one by one, and through properties that hold at any size."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, check_gemm_f32, same_with_nan, to_np_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
E4, E5 = oracle.E4M3, oracle.E5M2


def _scalar(v=0.0):
    return torch.tensor([v], dtype=torch.float32, device=DEV)


def test_casts_on_more_than_2pow32_elements():
    """n = 2^32 + 4099 bf16 elements (8.6 GB): the value that decides amax sits beyond index 2^32, and the
    slices compared with the oracle are the first 2^20 elements, a block at 2^31 and everything from 2^32 - 2^19
    to the ragged end"""
    n = (1 << 32) + 4099
    x = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    blk = 1 << 28
    for lo in range(0, n, blk):                                    # same recipe as the bandwidth sweep, block by block
        m = min(blk, n - lo)
        x[lo:lo + m] = synth.normal_laplace_mixture(m, 100 + lo // blk, synth.T_ID, device=DEV)
    big = (1 << 32) + 1234
    x[big] = -3.0e6                                                # decides amax; beyond the 32-bit index range
    slices = [(0, 1 << 20), (1 << 31, (1 << 31) + (1 << 18)), ((1 << 32) - (1 << 19), n)]
    x_host = [to_np_bits(x[lo:hi]) for lo, hi in slices]
    want_amax = oracle.amax_bits(to_np_bits(x[big:big + 1]))
    amax, s, si = _scalar(-1.0), _scalar(), _scalar()
    api.fp8_amax(x, amax)
    assert amax.cpu().numpy().view(np.uint32)[0] == want_amax
    api.fp8_scale_from_amax(amax, api.E5M2, s, si)
    ws, wsi = oracle.scale_from_amax(np.uint32(want_amax).view(np.float32), E5)
    assert s.item() == ws and si.item() == wsi
    codes = torch.full((n + 64,), 0xA5, dtype=torch.uint8, device=DEV)
    amax2 = _scalar(-1.0)
    api.fp8_quantize(x, api.E5M2, s, codes[:n], api.SATURATE, amax2)
    torch.cuda.synchronize()
    assert amax2.cpu().numpy().view(np.uint32)[0] == want_amax
    assert bool((codes[n:] == 0xA5).all())
    for (lo, hi), xh in zip(slices, x_host):
        assert np.array_equal(codes[lo:hi].cpu().numpy(), oracle.quantize(xh, ws, E5, threads=THREADS)), (lo, hi)
    # one-launch current scaling gives the same codes and scalars
    codes2 = torch.empty(n, dtype=torch.uint8, device=DEV)
    a3, s3, si3 = _scalar(-1.0), _scalar(), _scalar()
    api.fp8_quantize_current(x, api.E5M2, codes2, a3, s3, si3)
    torch.cuda.synchronize()
    assert a3.cpu().numpy().view(np.uint32)[0] == want_amax and s3.item() == ws and si3.item() == wsi
    for lo, hi in slices + [(big - 4096, n)]:
        assert torch.equal(codes2[lo:hi], codes[lo:hi]), (lo, hi)
    del codes2
    # dequantize back over the input buffer (the input is no longer needed)
    api.fp8_dequantize(codes[:n], api.E5M2, si, x)
    torch.cuda.synchronize()
    for lo, hi in slices:
        want = oracle.dequantize(codes[lo:hi].cpu().numpy(), wsi, E5, "bf16", threads=THREADS)
        assert same_with_nan(to_np_bits(x[lo:hi]), want, "bf16").all(), (lo, hi)


@pytest.mark.parametrize("acc", [api.ACC_FAST, api.ACC_SPLIT])
def test_gemm_contraction_of_2pow20_terms(acc):
    """K = 2^20: 8192 K-blocks per tile (512 chunks with split accumulation); sampled outputs against the oracle.
    Split accumulation holds 1e-5 * sum|ab|.  One accumulator over a million terms of heavy-tailed codes
    (magnitudes uniform over the code space) is outside what it is specified for (K <= 2048 on any data, the
    workloads' K <= 49152 on their data): its truncating additions reach about 1.2e-5 here, checked against 5e-5."""
    rng = np.random.default_rng(5)
    M, N, K = 128, 256, 1 << 20
    gen = torch.Generator(device=DEV)
    gen.manual_seed(11)
    A = torch.randint(0, 0x70, (M, K), dtype=torch.uint8, device=DEV, generator=gen) | (torch.randint(0, 2, (M, K), dtype=torch.uint8, device=DEV, generator=gen) << 7)
    B = torch.randint(0, 0x70, (N, K), dtype=torch.uint8, device=DEV, generator=gen) | (torch.randint(0, 2, (N, K), dtype=torch.uint8, device=DEV, generator=gen) << 7)
    D = torch.empty(M, N, dtype=torch.float32, device=DEV)
    api.fp8_gemm(A, api.E5M2, api.MAJOR_K, B, api.E4M3, api.MAJOR_K, D, _scalar(2.0 ** -10), _scalar(2.0 ** -4), acc=acc)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    ii = np.concatenate([rng.integers(0, M, 60), [0, 0, M - 1, M - 1]])
    jj = np.concatenate([rng.integers(0, N, 60), [0, N - 1, 0, N - 1]])
    ref, sabs = oracle.gemm_samples(A.cpu().numpy(), E5, (K, 1), B.cpu().numpy(), E4, (1, K), K, ii, jj, 2.0 ** -10, 2.0 ** -4, threads=THREADS)
    got = to_np_bits(D)[ii, jj]
    ok, worst = check_gemm_f32(got, ref, sabs, rel=1e-5 if acc == api.ACC_SPLIT else 5e-5)
    assert ok.all(), worst


def test_gemm_output_of_2pow20_rows():
    """M = 2^20 + 3 rows (4097 row tiles of 256), N = 24, K = 48: every row against the fp64 matmul of the decoded
    codes (E4M3 x E4M3: exact), so that a tile-coordinate or store-address overflow anywhere would show"""
    rng = np.random.default_rng(6)
    M, N, K = (1 << 20) + 3, 24, 48
    t = oracle.decode_table(E4)
    A_np = rng.integers(0, 0x78, size=(M, K), dtype=np.uint8) | (rng.integers(0, 2, size=(M, K), dtype=np.uint8) << 7)
    B_np = rng.integers(0, 0x78, size=(N, K), dtype=np.uint8) | (rng.integers(0, 2, size=(N, K), dtype=np.uint8) << 7)
    A, B = torch.from_numpy(A_np).to(DEV), torch.from_numpy(B_np).to(DEV)
    D_full = torch.full((M + 1, N), 777.0, dtype=torch.float32, device=DEV)
    amax = _scalar(-1.0)
    api.fp8_gemm(A, api.E4M3, api.MAJOR_K, B, api.E4M3, api.MAJOR_K, D_full[:M], _scalar(0.5), _scalar(0.25), amax)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0 and bool((D_full[M:] == 777.0).all())
    ref = (t[A_np] @ t[B_np].T) * 0.125
    sabs = (np.abs(t[A_np]) @ np.abs(t[B_np]).T) * 0.125
    got = to_np_bits(D_full[:M])
    ok, worst = check_gemm_f32(got, ref, sabs)
    assert ok.all(), (worst, np.argwhere(~ok)[:4].tolist())
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1), THREADS)
