"""Randomised shapes, layouts, formats, pitches, output types and accumulation modes through the GEMM entry
points.  The reference is the plain definition evaluated with library routines: the oracle's decode table
indexed by the codes, then a binary64 matrix product on the device (exact for E4M3 x E4M3, within 1e-12 of
sum|a.b| otherwise), with sum|a.b| from the product of the absolute values.  Fixed seeds: the cases are the same
on every run."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api
from tests._util import check_gemm_bf16, check_gemm_f32, to_np_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
TABLES = {}


def _table(fmt):
    if fmt not in TABLES:
        TABLES[fmt] = torch.from_numpy(oracle.decode_table(fmt)).to(DEV)
    return TABLES[fmt]


def _operand(rng, rows, cols, fmt):
    """finite random codes in a buffer whose pitch is a multiple of 16 plus a random number of 16-byte pads;
    the padding holds NaN codes, so that a read outside the logical extent poisons the result"""
    pitch = (cols + 15) // 16 * 16 + 16 * int(rng.integers(0, 3))
    top = 0x7E if fmt == oracle.E4M3 else 0x7B
    buf = np.full((rows, pitch), 0x7F, dtype=np.uint8)
    buf[:, :cols] = rng.integers(0, top + 1, size=(rows, cols), dtype=np.uint8) | (rng.integers(0, 2, size=(rows, cols), dtype=np.uint8) << 7)
    t = torch.from_numpy(buf).to(DEV)
    return t[:, :cols]


def _reference(A, fa, ma, B, fb, mb, alpha):
    a = _table(fa)[A.long()]
    b = _table(fb)[B.long()]
    a = a if ma == api.MAJOR_K else a.t()                 # [M, K]
    b = b.t() if mb == api.MAJOR_K else b                 # [K, N]
    ref = (a @ b) * alpha
    sabs = (a.abs() @ b.abs()) * alpha
    return ref.cpu().numpy(), sabs.cpu().numpy()


@pytest.mark.parametrize("seed", range(48))
def test_random_gemm_case(seed):
    rng = np.random.default_rng(9000 + seed)
    big = seed % 6 == 0
    M = int(rng.integers(1, 1200 if big else 400))
    N = int(rng.integers(1, 1500 if big else 500))
    K = int(rng.integers(1, 6000 if big else 1500))
    fa, fb = (int(rng.integers(0, 2)), int(rng.integers(0, 2)))
    ma, mb = (int(rng.integers(0, 2)), int(rng.integers(0, 2)))
    acc = int(rng.integers(0, 2))
    out_dtype = torch.float32 if rng.integers(0, 2) else torch.bfloat16
    A = _operand(rng, M if ma == api.MAJOR_K else K, K if ma == api.MAJOR_K else M, fa)
    B = _operand(rng, N if mb == api.MAJOR_K else K, K if mb == api.MAJOR_K else N, fb)
    sa, sb = float(2.0 ** rng.integers(-12, -2)), float(2.0 ** rng.integers(-6, 0))
    esz = 4 if out_dtype == torch.float32 else 2
    ldd = (N * esz + 15) // 16 * 16 // esz + (16 // esz) * int(rng.integers(0, 3))
    D_full = torch.full((M + 1, ldd), 777.0, dtype=out_dtype, device=DEV)
    D = D_full[:M, :N]
    amax = torch.full((1,), -1.0, device=DEV)
    api.fp8_gemm(A, fa, ma, B, fb, mb, D, torch.tensor([sa], device=DEV), torch.tensor([sb], device=DEV), amax, acc=acc)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert bool((D_full[M:, :] == 777.0).all()) and bool((D_full[:M, N:] == 777.0).all()), "wrote outside D"
    ref, sabs = _reference(A, fa, ma, B, fb, mb, np.float64(np.float32(sa)) * np.float64(np.float32(sb)))
    got = to_np_bits(D)
    what = (M, N, K, fa, fb, ma, mb, acc, str(out_dtype))
    if out_dtype == torch.float32:
        ok, worst = check_gemm_f32(got, ref, sabs)
        assert ok.all(), (what, worst, np.argwhere(~ok)[:4].tolist())
    else:
        ok, _ = check_gemm_bf16(got, ref, sabs, oracle.round_bf16_from_f64)
        assert ok.all(), (what, np.argwhere(~ok)[:4].tolist())
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1)), what


@pytest.mark.parametrize("seed", range(32))
def test_random_fp8_output_case(seed):
    from tests._util import check_gemm_fp8out
    rng = np.random.default_rng(7000 + seed)
    M, N, K = int(rng.integers(1, 500)), int(rng.integers(1, 600)), int(rng.integers(1, 3000))
    fa, fb, fd = int(rng.integers(0, 2)), int(rng.integers(0, 2)), int(rng.integers(0, 2))
    ma, mb, acc = int(rng.integers(0, 2)), int(rng.integers(0, 2)), int(rng.integers(0, 2))
    overflow = int(rng.integers(0, 2))
    A = _operand(rng, M if ma == api.MAJOR_K else K, K if ma == api.MAJOR_K else M, fa)
    B = _operand(rng, N if mb == api.MAJOR_K else K, K if mb == api.MAJOR_K else N, fb)
    sa, sb = float(2.0 ** rng.integers(-12, -2)), float(2.0 ** rng.integers(-6, 0))
    ref, sabs = _reference(A, fa, ma, B, fb, mb, np.float64(np.float32(sa)) * np.float64(np.float32(sb)))
    # an output scale that puts the largest result near the top of the format, or (non-saturating runs) beyond it
    peak = max(float(np.abs(ref).max()), 1e-30)
    fmax = 448.0 if fd == oracle.E4M3 else 57344.0
    scale_d = float(np.float32(fmax / peak * (4.0 if overflow == api.NOSAT and seed % 2 else 0.9)))
    ldd = (N + 15) // 16 * 16 + 16 * int(rng.integers(0, 3))
    D_full = torch.full((M + 1, ldd), 0xA5, dtype=torch.uint8, device=DEV)
    D = D_full[:M, :N]
    amax = torch.full((1,), -1.0, device=DEV)
    dev = lambda v: torch.tensor([v], dtype=torch.float32, device=DEV)
    api.fp8_gemm_fp8out(A, fa, ma, B, fb, mb, D, fd, dev(sa), dev(sb), dev(scale_d), amax, overflow, acc=acc)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert bool((D_full[M:, :] == 0xA5).all()) and bool((D_full[:M, N:] == 0xA5).all()), "wrote outside D"
    enc = lambda y: oracle.quantize(y.reshape(-1), 1.0, fd, overflow).reshape(y.shape)
    ok, _ = check_gemm_fp8out(D.cpu().numpy(), ref, sabs, scale_d, enc)
    assert ok.all(), ((M, N, K, fa, fb, fd, ma, mb, acc, overflow), np.argwhere(~ok)[:4].tolist())
    lo = np.max(np.abs(ref) - 1e-5 * sabs) * (1 - 2.0 ** -22)
    hi = np.max(np.abs(ref) + 1e-5 * sabs) * (1 + 2.0 ** -22)
    assert lo <= float(amax.item()) <= hi


@pytest.mark.parametrize("seed", range(24))
def test_random_batched_and_splitk_case(seed):
    rng = np.random.default_rng(5000 + seed)
    fa, fb = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    dev = lambda v: torch.tensor([v], dtype=torch.float32, device=DEV)
    sa, sb = float(2.0 ** rng.integers(-12, -2)), float(2.0 ** rng.integers(-6, 0))
    alpha = np.float64(np.float32(sa)) * np.float64(np.float32(sb))
    if seed % 2 == 0:
        # batched: heads side by side inside the rows of [S, H*d] operands
        H, S, T, Dh = int(rng.integers(1, 6)), int(rng.integers(1, 300)), int(rng.integers(1, 300)), 16 * int(rng.integers(1, 9))
        Qf = _operand(rng, S, H * Dh, fa)
        Kf = _operand(rng, T, H * Dh, fb)
        Q = Qf.as_strided((H, S, Dh), (Dh, Qf.stride(0), 1))
        Kt = Kf.as_strided((H, T, Dh), (Dh, Kf.stride(0), 1))
        ldd = (T + 3) // 4 * 4
        D = torch.full((H, S + 1, ldd), 777.0, dtype=torch.float32, device=DEV)
        amax = torch.full((1,), -1.0, device=DEV)
        api.fp8_gemm_batched(Q, fa, api.MAJOR_K, Kt, fb, api.MAJOR_K, D[:, :S, :T], dev(sa), dev(sb), amax)
        torch.cuda.synchronize()
        assert api.fp8_async_status()[0] == 0
        assert bool((D[:, S:, :] == 777.0).all()) and bool((D[:, :S, T:] == 777.0).all())
        got = to_np_bits(D[:, :S, :T])
        for h in range(H):
            ref, sabs = _reference(Qf[:, h * Dh:(h + 1) * Dh], fa, api.MAJOR_K, Kf[:, h * Dh:(h + 1) * Dh], fb, api.MAJOR_K, alpha)
            ok, worst = check_gemm_f32(got[h], ref, sabs)
            assert ok.all(), (h, worst)
        assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1))
    else:
        # split-K: few rows, long contraction
        M, N, K = int(rng.integers(1, 260)), 4 * int(rng.integers(1, 300)), 256 * int(rng.integers(8, 80))
        mb = int(rng.integers(0, 2))
        A = _operand(rng, M, K, fa)
        B = _operand(rng, N if mb == api.MAJOR_K else K, K if mb == api.MAJOR_K else N, fb)
        splits, nbytes = api.fp8_gemm_splitk_workspace(M, N, K)
        ws = torch.empty(max(nbytes // 4, 4), dtype=torch.float32, device=DEV)
        out_dtype = torch.float32 if seed % 4 == 1 else torch.bfloat16
        esz = 4 if out_dtype == torch.float32 else 2
        ldd = (N * esz + 15) // 16 * 16 // esz
        D_full = torch.full((M + 1, ldd), 777.0, dtype=out_dtype, device=DEV)
        amax = torch.full((1,), -1.0, device=DEV)
        api.fp8_gemm_splitk(A, fa, api.MAJOR_K, B, fb, mb, D_full[:M, :N], dev(sa), dev(sb), ws if nbytes else None, amax)
        torch.cuda.synchronize()
        assert api.fp8_async_status()[0] == 0
        assert bool((D_full[M:, :] == 777.0).all()) and bool((D_full[:M, N:] == 777.0).all())
        ref, sabs = _reference(A, fa, api.MAJOR_K, B, fb, mb, alpha)
        got = to_np_bits(D_full[:M, :N])
        if out_dtype == torch.float32:
            ok, worst = check_gemm_f32(got, ref, sabs)
        else:
            ok, _ = check_gemm_bf16(got, ref, sabs, oracle.round_bf16_from_f64)
        assert ok.all(), ((M, N, K, mb, splits), np.argwhere(~ok)[:4].tolist())
        assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1))


@pytest.mark.parametrize("seed", range(64))
def test_random_cast_case(seed):
    """random length, pointer offsets, wide type, format, overflow mode and scale, special values sprinkled in:
    quantize (+ amax), one-launch current scaling, dequantize and the simulated round trip against the oracle,
    bit for bit, with guard elements around every output"""
    from tests._util import same_with_nan
    rng = np.random.default_rng(3000 + seed)
    n = int(rng.integers(0, 1 << int(rng.integers(1, 20))))
    wide = torch.float32 if rng.integers(0, 2) else torch.bfloat16
    name = "f32" if wide == torch.float32 else "bf16"
    fmt, overflow = int(rng.integers(0, 2)), int(rng.integers(0, 2))
    off_in, off_out = int(rng.integers(0, 16)), int(rng.integers(0, 16))
    scale = float(np.float32(2.0 ** rng.uniform(-20, 20)))
    vals = rng.standard_normal(n).astype(np.float32) * np.exp2(rng.uniform(-12, 12, size=n)).astype(np.float32)
    if n:
        specials = np.array([np.nan, -np.nan, np.inf, -np.inf, 0.0, -0.0, 448.0, 464.0, 465.0, 57344.0, 61440.0, 3e38, -3e38, 1e-40, 2.0 ** -9, 2.0 ** -17],
                            dtype=np.float32)
        where = rng.integers(0, n, size=max(1, n // 50))
        vals[where] = specials[rng.integers(0, specials.size, size=where.size)]
    base = torch.zeros(n + 32, dtype=wide, device=DEV)
    x = base[off_in:off_in + n]
    x.copy_(torch.from_numpy(vals).to(DEV).to(wide))
    xh = to_np_bits(x)
    dev = lambda v: torch.tensor([v], dtype=torch.float32, device=DEV)
    # quantize + amax
    out_full = torch.full((n + 48,), 0xA5, dtype=torch.uint8, device=DEV)
    out = out_full[off_out:off_out + n]
    amax = dev(-1.0)
    api.fp8_quantize(x, fmt, dev(scale), out, overflow, amax)
    want = oracle.quantize(xh, np.float32(scale), fmt, overflow)
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), want), (n, name, fmt, overflow, off_in, off_out, scale)
    assert bool((out_full[:off_out] == 0xA5).all()) and bool((out_full[off_out + n:] == 0xA5).all())
    want_amax = oracle.amax_bits(xh) if n else 0
    assert amax.cpu().numpy().view(np.uint32)[0] == want_amax
    # one-launch current scaling
    out_full.fill_(0xA5)
    a2, s2, si2 = dev(-1.0), dev(-1.0), dev(-1.0)
    api.fp8_quantize_current(x, fmt, out, a2, s2, si2, overflow)
    ws, wsi = oracle.scale_from_amax(np.uint32(want_amax).view(np.float32), fmt)
    torch.cuda.synchronize()
    assert a2.cpu().numpy().view(np.uint32)[0] == want_amax and s2.item() == ws and si2.item() == wsi
    want2 = oracle.quantize(xh, ws, fmt, overflow)
    assert np.array_equal(out.cpu().numpy(), want2)
    assert bool((out_full[:off_out] == 0xA5).all()) and bool((out_full[off_out + n:] == 0xA5).all())
    # dequantize of those codes, and the simulated round trip
    back_full = torch.full((n + 48,), 7.0, dtype=wide, device=DEV)
    back = back_full[off_out:off_out + n]
    api.fp8_dequantize(out, fmt, si2, back)
    torch.cuda.synchronize()
    assert same_with_nan(to_np_bits(back), oracle.dequantize(want2, wsi, fmt, name), name).all()
    assert bool((back_full[:off_out] == 7.0).all()) and bool((back_full[off_out + n:] == 7.0).all())
    back_full.fill_(7.0)
    api.fp8_fake_quantize(x, fmt, s2, si2, back, overflow)
    torch.cuda.synchronize()
    assert same_with_nan(to_np_bits(back), oracle.fake_quantize(xh, ws, wsi, fmt, overflow), name).all()
    assert bool((back_full[:off_out] == 7.0).all()) and bool((back_full[off_out + n:] == 7.0).all())


@pytest.mark.parametrize("seed", range(48))
def test_random_channel_and_transpose_case(seed):
    """random 2-D shapes, pitches and base offsets through the per-channel kernels (both axes) and the transposing
    quantizer, with special values sprinkled in; everything bit-exact against the oracle"""
    rng = np.random.default_rng(1000 + seed)
    rows, cols = int(rng.integers(1, 700)), int(rng.integers(1, 900))
    if seed % 3 == 0:                                       # shapes the vector paths accept
        rows, cols = 4 * int(rng.integers(1, 200)), 8 * int(rng.integers(1, 150))
    wide = torch.float32 if rng.integers(0, 2) else torch.bfloat16
    fmt, overflow, axis = int(rng.integers(0, 2)), int(rng.integers(0, 2)), int(rng.integers(0, 2))
    pitch = cols + (8 * int(rng.integers(0, 3)) if seed % 3 == 0 else int(rng.integers(0, 9)))
    off = 0 if seed % 3 == 0 else int(rng.integers(0, 8))
    vals = rng.standard_normal(rows * pitch).astype(np.float32) * np.exp2(rng.uniform(-8, 8, size=rows * pitch)).astype(np.float32)
    specials = np.array([np.nan, -np.nan, np.inf, -np.inf, 0.0, -0.0, 448.0, 465.0, 61440.0, 3e38, 1e-40], dtype=np.float32)
    where = rng.integers(0, vals.size, size=max(1, vals.size // 200))
    vals[where] = specials[rng.integers(0, specials.size, size=where.size)]
    base = torch.zeros(rows * pitch + 16, dtype=wide, device=DEV)
    base[off:off + rows * pitch] = torch.from_numpy(vals).to(DEV).to(wide)
    x = base[off:off + rows * pitch].view(rows, pitch)[:, :cols]
    xh = to_np_bits(x)
    # per-channel amax -> scales -> quantize
    nch = cols if axis == 0 else rows
    am = torch.full((nch,), -1.0, device=DEV)
    sv, siv = torch.empty(nch, device=DEV), torch.empty(nch, device=DEV)
    api.fp8_amax_channels(x, axis, am)
    api.fp8_scales_from_amax(am, fmt, sv, siv)
    opitch = cols + int(rng.integers(0, 3)) * (8 if seed % 3 == 0 else 1)
    q_full = torch.full((rows + 1, opitch), 0xA5, dtype=torch.uint8, device=DEV)
    api.fp8_quantize_channels(x, axis, fmt, sv, q_full[:rows, :cols], overflow)
    torch.cuda.synchronize()
    want_am = oracle.amax_channels(xh, axis)
    assert np.array_equal(am.cpu().numpy().view(np.uint32), want_am.view(np.uint32)), (rows, cols, axis, str(wide))
    ws, wsi = oracle.scales_from_amax(want_am, fmt)
    assert np.array_equal(sv.cpu().numpy(), ws) and np.array_equal(siv.cpu().numpy(), wsi)
    assert np.array_equal(q_full[:rows, :cols].cpu().numpy(), oracle.quantize_channels(xh, ws, axis, fmt, overflow))
    assert bool((q_full[rows:, :] == 0xA5).all()) and bool((q_full[:rows, cols:] == 0xA5).all())
    # quantize + transposed copy with one scale
    scale = float(np.float32(2.0 ** rng.uniform(-6, 6)))
    tpitch = rows + int(rng.integers(0, 3)) * (4 if seed % 3 == 0 else 1)
    q_full.fill_(0xA5)
    t_full = torch.full((cols + 1, tpitch), 0xA5, dtype=torch.uint8, device=DEV)
    amax = torch.full((1,), -1.0, device=DEV)
    api.fp8_quantize_transpose(x, fmt, torch.tensor([scale], device=DEV), q_full[:rows, :cols], t_full[:cols, :rows], amax, overflow)
    torch.cuda.synchronize()
    want = oracle.quantize(xh.reshape(-1), np.float32(scale), fmt, overflow).reshape(rows, cols)
    assert np.array_equal(q_full[:rows, :cols].cpu().numpy(), want) and np.array_equal(t_full[:cols, :rows].cpu().numpy(), want.T)
    assert bool((q_full[rows:, :] == 0xA5).all()) and bool((q_full[:rows, cols:] == 0xA5).all())
    assert bool((t_full[cols:, :] == 0xA5).all()) and bool((t_full[:cols, rows:] == 0xA5).all())
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(xh.reshape(-1))
