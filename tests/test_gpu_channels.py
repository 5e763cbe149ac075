"""Per-channel scale factors (per-channel weights, per-tensor activations): amax per row / column,
vector scales, quantize with a scale vector (bit-exact), and the GEMM with one inverse scale per output
channel (tolerance of the per-tensor GEMM)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, check_gemm_bf16, check_gemm_f32, to_np_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
E4, E5 = oracle.E4M3, oracle.E5M2


def _scalar(v):
    return torch.tensor([v], dtype=torch.float32, device=DEV)


@pytest.mark.parametrize("wide", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("axis", [0, 1])
@pytest.mark.parametrize("shape,pitch", [((1, 1), 1), ((37, 53), 53), ((64, 128), 128), ((300, 520), 528), ((1024, 4096), 4096),
                                          ((5, 4099), 4099), ((513, 72), 80), ((3, 16405), 16416), ((2000, 264), 264), ((700, 1300), 1312)])
def test_amax_scales_quantize_per_channel(wide, axis, shape, pitch):
    rows, cols = shape
    base = synth.weights(rows * pitch + 8, 13, 0.02, dtype=wide, device=DEV)
    x = base[: rows * pitch].view(rows, pitch)[:, :cols]
    if rows * cols > 100:
        x[3 % rows, 5 % cols] = float("nan")
        x[1 % rows, 9 % cols] = float("inf")
        x[2 % rows, 2 % cols] = 40.0
    x_np = to_np_bits(x)
    channels = cols if axis == 0 else rows
    amax = torch.full((channels,), -1.0, dtype=torch.float32, device=DEV)
    api.fp8_amax_channels(x, axis, amax)
    want_amax = oracle.amax_channels(x_np, axis)
    assert np.array_equal(amax.cpu().numpy().view(np.uint32), want_amax.view(np.uint32))
    for fmt, pow2 in ((E4, False), (E5, True)):
        s = torch.empty(channels, dtype=torch.float32, device=DEV)
        si = torch.empty(channels, dtype=torch.float32, device=DEV)
        api.fp8_scales_from_amax(amax, fmt, s, si, pow2)
        ws, wsi = oracle.scales_from_amax(want_amax, fmt, pow2)
        assert np.array_equal(s.cpu().numpy().view(np.uint32), ws.view(np.uint32))
        assert np.array_equal(si.cpu().numpy().view(np.uint32), wsi.view(np.uint32))
        for overflow in (api.SATURATE, api.NOSAT):
            out_pitch = (cols + 15) // 16 * 16
            out_full = torch.full((rows + 1, out_pitch), 0xA5, dtype=torch.uint8, device=DEV)
            out = out_full[:rows, :cols]
            api.fp8_quantize_channels(x, axis, fmt, s, out, overflow)
            torch.cuda.synchronize()
            want = oracle.quantize_channels(x_np, ws, axis, fmt, overflow)
            got = out.cpu().numpy()
            bad = np.argwhere(got != want)
            assert bad.size == 0, bad[:5].tolist()
            assert bool((out_full[rows:, :] == 0xA5).all()) and bool((out_full[:rows, cols:] == 0xA5).all())


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("shape", [(384, 768, 640), (129, 257, 129), (100, 40, 48)])
def test_gemm_with_per_channel_weight_scales(out_dtype, shape):
    """weights W[K,N] quantized with one scale per output channel (column), activations per tensor"""
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    n_pitch = (N + 15) // 16 * 16
    w = synth.weights(K * n_pitch, 21, 0.02, dtype=torch.bfloat16, device=DEV).view(K, n_pitch)[:, :N]
    w = w * torch.exp2(torch.randint(-3, 4, (N,), device=DEV).float()).to(torch.bfloat16)      # channels of different magnitude
    xa = synth.activations(M * K, 22, dtype=torch.bfloat16, device=DEV).view(M, K)
    w = w.contiguous() if N == n_pitch else w
    # library: per-channel path for W, per-tensor path for X
    amax_w = torch.empty(N, dtype=torch.float32, device=DEV)
    sw, siw = torch.empty(N, dtype=torch.float32, device=DEV), torch.empty(N, dtype=torch.float32, device=DEV)
    wq_full = torch.full((K, n_pitch), 0x7F, dtype=torch.uint8, device=DEV)     # NaN codes in the padding
    wq = wq_full[:, :N]
    wc = w.contiguous()
    api.fp8_amax_channels(wc, 0, amax_w)
    api.fp8_scales_from_amax(amax_w, api.E4M3, sw, siw)
    api.fp8_quantize_channels(wc, 0, api.E4M3, sw, wq)
    ax, sx, six = _scalar(0.0), _scalar(0.0), _scalar(0.0)
    k_pitch = (K + 15) // 16 * 16
    xq_full = torch.full((M, k_pitch), 0x7F, dtype=torch.uint8, device=DEV)
    xq = xq_full[:, :K]
    xq_dense = torch.empty(M * K, dtype=torch.uint8, device=DEV)
    api.fp8_quantize_current(xa, api.E4M3, xq_dense, ax, sx, six)
    xq.copy_(xq_dense.view(M, K))
    ldd = (N * (2 if out_dtype == torch.bfloat16 else 4) + 15) // 16 * 16 // (2 if out_dtype == torch.bfloat16 else 4)
    D_full = torch.full((M + 1, ldd), 777.0, dtype=out_dtype, device=DEV)
    D = D_full[:M, :N]
    amax_d = _scalar(-1.0)
    api.fp8_gemm_channel_scales(xq, api.E4M3, api.MAJOR_K, wq, api.E4M3, api.MAJOR_MN, D, six, siw, amax_d)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert bool((D_full[M:, :] == 777.0).all()) and bool((D_full[:M, N:] == 777.0).all())
    # oracle from the same wide inputs
    w_np, x_np = to_np_bits(wc), to_np_bits(xa)
    o_siw = oracle.scales_from_amax(oracle.amax_channels(w_np, 0), E4)
    Wq = oracle.quantize_channels(w_np, o_siw[0], 0, E4)
    o_sx = oracle.scale_from_amax(oracle.amax(x_np.reshape(-1)), E4)
    Xq = oracle.quantize(x_np.reshape(-1), o_sx[0], E4).reshape(M, K)
    assert np.array_equal(wq.cpu().numpy(), Wq) and np.array_equal(xq.cpu().numpy(), Xq)
    ref, sabs = oracle.gemm_rows_colscale(Xq, E4, (K, 1), Wq, E4, (N, 1), N, K, 0, M, o_sx[1], o_siw[1], threads=THREADS)
    got = to_np_bits(D)
    if out_dtype == torch.float32:
        ok, worst = check_gemm_f32(got, ref, sabs)
    else:
        ok, _ = check_gemm_bf16(got, ref, sabs, oracle.round_bf16_from_f64)
    assert ok.all(), np.argwhere(~ok)[:4].tolist()
    a2 = _scalar(-1.0)
    api.fp8_amax(D.contiguous(), a2)
    assert amax_d.cpu().numpy().view(np.uint32)[0] == a2.cpu().numpy().view(np.uint32)[0]


def test_quantize_per_column_at_the_size_where_the_slabs_become_short():
    """From 256 MB on the per-column conversion runs 64-row slabs: a tensor just above that size, with a row count that
    is no multiple of the slab, a row pitch wider than the row, and special values, against the oracle bit for bit;
    the bytes around the output stay untouched."""
    rows, cols, pitch = 16400 + 37, 8192, 8208                      # 269 MB of bf16
    base = synth.weights(rows * pitch, 17, 0.02, dtype=torch.bfloat16, device=DEV)
    x = base.view(rows, pitch)[:, :cols]
    x[rows - 1, cols - 1] = float("nan")
    x[rows - 2, 3] = float("inf")
    x[77, 4100] = 11.0
    x_np = to_np_bits(x)
    amax = torch.empty(cols, dtype=torch.float32, device=DEV)
    api.fp8_amax_channels(x, 0, amax)
    want_amax = oracle.amax_channels(x_np, 0)
    assert np.array_equal(amax.cpu().numpy().view(np.uint32), want_amax.view(np.uint32))
    s, si = torch.empty(cols, dtype=torch.float32, device=DEV), torch.empty(cols, dtype=torch.float32, device=DEV)
    api.fp8_scales_from_amax(amax, E4, s, si)
    ws, _ = oracle.scales_from_amax(want_amax, E4)
    out_full = torch.full((rows + 1, cols + 16), 0xA5, dtype=torch.uint8, device=DEV)
    out = out_full[:rows, :cols]
    api.fp8_quantize_channels(x, 0, E4, s, out)
    torch.cuda.synchronize()
    want = oracle.quantize_channels(x_np, ws, 0, E4, api.SATURATE)
    got = out.cpu().numpy()
    bad = np.argwhere(got != want)
    assert bad.size == 0, bad[:5].tolist()
    assert bool((out_full[rows:, :] == 0xA5).all()) and bool((out_full[:rows, cols:] == 0xA5).all())
