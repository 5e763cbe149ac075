"""GPU parity of fp8_gemm against the CPU oracle (fp64 accumulation over decoded codes).
fp32 output: |gpu - ref| <= 1e-5 * sum_k |a.b| per element.  bf16 output: within 1 bf16 ulp of the
correctly rounded value of some v inside that interval (equal to "1 ulp of the rounded reference"
whenever the accumulation error is far below one bf16 ulp of the result)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2209_05433_b200 import api, synth
from tests._util import THREADS, check_gemm_bf16, check_gemm_f32, check_gemm_fp8out, to_np_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"
E4, E5 = oracle.E4M3, oracle.E5M2
ROLES = {"fprop": (E4, E4), "dgrad": (E5, E4), "wgrad": (E4, E5)}


def _scalar(v):
    return torch.tensor([v], dtype=torch.float32, device=DEV)


def _codes(rng, fmt, shape, spread=6.0):
    """finite random codes with magnitudes spread over a few binades around 1"""
    x = rng.standard_normal(shape).astype(np.float32) * np.exp2(rng.uniform(-spread, 2, size=shape)).astype(np.float32)
    return oracle.quantize(x, 1.0, fmt).reshape(shape)


def _pad_cols(a_np, mult=16, fill=0x7F):
    """copy into a buffer whose row pitch is a multiple of 16 bytes; padding holds NaN codes
    so that any read outside the logical extent would poison the result"""
    r, c = a_np.shape
    pitch = (c + mult - 1) // mult * mult
    buf = np.full((r, pitch), fill, dtype=np.uint8)
    buf[:, :c] = a_np
    return buf


def _run(A_np, fa, ma, B_np, fb, mb, M, N, K, out_dtype, sa_inv=0.013, sb_inv=0.5, want_amax=True, acc=api.ACC_FAST):
    """A_np is the stored array ([M,K] or [K,M]); B_np the stored array ([N,K] or [K,N])."""
    A_buf, B_buf = _pad_cols(A_np), _pad_cols(B_np)
    A = torch.from_numpy(A_buf).to(DEV)[:, : A_np.shape[1]]
    B = torch.from_numpy(B_buf).to(DEV)[:, : B_np.shape[1]]
    esz = 2 if out_dtype == torch.bfloat16 else 4
    ldd = (N * esz + 15) // 16 * 16 // esz
    D_full = torch.full((M + 1, ldd), 777.0, dtype=out_dtype, device=DEV)       # guard row and pad columns
    D = D_full[:M, :N]
    amax = _scalar(-1.0) if want_amax else None
    api.fp8_gemm(A, fa, ma, B, fb, mb, D, _scalar(sa_inv), _scalar(sb_inv), amax, acc=acc)
    torch.cuda.synchronize()
    st, detail = api.fp8_async_status()
    assert st == 0, "device-side wait expired, code %d" % detail
    assert bool((D_full[M:, :] == 777.0).all()) and bool((D_full[:M, N:] == 777.0).all()), "wrote outside D"
    a_str = (A_buf.shape[1], 1) if ma == api.MAJOR_K else (1, A_buf.shape[1])
    b_str = (1, B_buf.shape[1]) if mb == api.MAJOR_K else (B_buf.shape[1], 1)
    ref, sabs = oracle.gemm_rows(A_buf, fa, a_str, B_buf, fb, b_str, N, K, 0, M, sa_inv, sb_inv, threads=THREADS)
    got = to_np_bits(D)
    if out_dtype == torch.float32:
        ok, worst = check_gemm_f32(got, ref, sabs)
        assert ok.all(), "fp32: %d of %d outside 1e-5*sum|ab| (worst ratio %.3g) at %s" % (
            (~ok).sum(), ok.size, worst, np.argwhere(~ok)[:4].tolist())
    else:
        ok, literal = check_gemm_bf16(got, ref, sabs, oracle.round_bf16_from_f64)
        assert ok.all(), "bf16: %d of %d fail at %s" % ((~ok).sum(), ok.size, np.argwhere(~ok)[:4].tolist())
    if want_amax:
        # epilogue amax is the amax of D as stored: the library's own fp8_amax and the oracle's amax of
        # the stored values must both reproduce it bit for bit
        dense = D.contiguous()
        a2 = _scalar(-1.0)
        api.fp8_amax(dense, a2)
        bits = amax.cpu().numpy().view(np.uint32)[0]
        assert bits == a2.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(to_np_bits(dense).reshape(-1))
    return got, ref, sabs


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_config1_tiny_gemm(out_dtype):
    """fp32 A, B [256x256] N(0,1) with 0.5% x64 outliers, amax-derived scales, E4M3 x E4M3, M=N=K=256"""
    M = N = K = 256
    xa = synth.normal_with_scaled_outliers(M * K, 0, synth.A_ID, 0.005, 64.0, device=DEV)
    xb = synth.normal_with_scaled_outliers(K * N, 0, synth.B_ID, 0.005, 64.0, device=DEV)
    qa = torch.empty(M * K, dtype=torch.uint8, device=DEV)
    qb = torch.empty(K * N, dtype=torch.uint8, device=DEV)
    sinv = []
    for x, q in ((xa, qa), (xb, qb)):
        a, s, si = _scalar(0.0), _scalar(0.0), _scalar(0.0)
        api.fp8_amax(x, a)
        api.fp8_scale_from_amax(a, api.E4M3, s, si)
        api.fp8_quantize(x, api.E4M3, s, q)
        sinv.append(si)
    # oracle side from the same wide inputs
    wa = oracle.scale_from_amax(oracle.amax(to_np_bits(xa)), E4)
    wb = oracle.scale_from_amax(oracle.amax(to_np_bits(xb)), E4)
    A_np = oracle.quantize(to_np_bits(xa), wa[0], E4).reshape(M, K)
    B_np = oracle.quantize(to_np_bits(xb), wb[0], E4).reshape(K, N)      # stored [K,N]: N contiguous
    assert np.array_equal(qa.cpu().numpy().reshape(M, K), A_np) and np.array_equal(qb.cpu().numpy().reshape(K, N), B_np)
    D = torch.empty(M, N, dtype=out_dtype, device=DEV)
    api.fp8_gemm(qa.view(M, K), api.E4M3, api.MAJOR_K, qb.view(K, N), api.E4M3, api.MAJOR_MN, D, sinv[0], sinv[1])
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    ref, sabs = oracle.gemm_rows(A_np, E4, (K, 1), B_np, E4, (N, 1), N, K, 0, M, wa[1], wb[1], threads=THREADS)
    if out_dtype == torch.float32:
        ok, worst = check_gemm_f32(to_np_bits(D), ref, sabs)
        assert ok.all(), worst
    else:
        ok, literal = check_gemm_bf16(to_np_bits(D), ref, sabs, oracle.round_bf16_from_f64)
        assert ok.all()


@pytest.mark.parametrize("role", list(ROLES))
@pytest.mark.parametrize("ma", [api.MAJOR_K, api.MAJOR_MN])
@pytest.mark.parametrize("mb", [api.MAJOR_K, api.MAJOR_MN])
@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_layouts_formats_and_outputs(role, ma, mb, out_dtype):
    """several tiles in each direction, several K blocks, every operand layout and format pair"""
    fa, fb = ROLES[role]
    M, N, K = 384, 768, 640
    rng = np.random.default_rng(1000 + list(ROLES).index(role) * 4 + ma * 2 + mb)
    A_np = _codes(rng, fa, (M, K) if ma == api.MAJOR_K else (K, M))
    B_np = _codes(rng, fb, (N, K) if mb == api.MAJOR_K else (K, N))
    _run(A_np, fa, ma, B_np, fb, mb, M, N, K, out_dtype)


@pytest.mark.parametrize("M,N,K", [(1, 8, 16), (100, 40, 48), (129, 257, 129), (300, 520, 200), (128, 256, 128),
                                    (257, 8, 1000), (5, 1000, 33)])
@pytest.mark.parametrize("ma,mb", [(api.MAJOR_K, api.MAJOR_K), (api.MAJOR_K, api.MAJOR_MN), (api.MAJOR_MN, api.MAJOR_MN)])
def test_ragged_edges(M, N, K, ma, mb):
    """sizes that are not multiples of the tile; padding columns of A and B hold NaN codes"""
    rng = np.random.default_rng(M * 1000003 + N * 1009 + K)
    A_np = _codes(rng, E5, (M, K) if ma == api.MAJOR_K else (K, M))
    B_np = _codes(rng, E4, (N, K) if mb == api.MAJOR_K else (K, N))
    for out_dtype in (torch.float32, torch.bfloat16):
        _run(A_np, E5, ma, B_np, E4, mb, M, N, K, out_dtype)


def test_long_k_accumulation_error():
    """K as long as the workloads' longest contraction (49152), operands of both signs like every
    tensor of the workloads: the binary32 accumulation of the tensor cores stays inside 1e-5*sum|ab|"""
    rng = np.random.default_rng(77)
    M, N, K = 128, 256, 49152
    for fa, fb in ((E4, E4), (E5, E4)):
        A_np = _codes(rng, fa, (M, K), spread=3.0)
        B_np = _codes(rng, fb, (N, K), spread=3.0)
        _run(A_np, fa, api.MAJOR_K, B_np, fb, api.MAJOR_K, M, N, K, torch.float32)
        _run(A_np, fa, api.MAJOR_K, B_np, fb, api.MAJOR_K, M, N, K, torch.bfloat16)


def test_same_sign_accumulation_bound():
    """All-positive operands: no cancellation, |sum| = sum|ab|, the worst case for an accumulator that
    truncates.  The tensor core adds each K=32 block product into the binary32 accumulator with
    truncation, so the error grows like (K/32) * 2^-23 * sum|ab|: inside 1e-5 up to K = 2048 for any
    data, and inside that derived bound beyond."""
    rng = np.random.default_rng(78)
    M, N = 128, 256
    for K in (2048, 49152):
        A_np = _codes(rng, E4, (M, K), spread=1.0) & 0x7F
        B_np = _codes(rng, E4, (N, K), spread=1.0) & 0x7F
        A = torch.from_numpy(A_np).to(DEV)
        B = torch.from_numpy(B_np).to(DEV)
        D = torch.empty(M, N, dtype=torch.float32, device=DEV)
        api.fp8_gemm(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, D, _scalar(1.0), _scalar(1.0))
        torch.cuda.synchronize()
        assert api.fp8_async_status()[0] == 0
        ref, sabs = oracle.gemm_rows(A_np, E4, (K, 1), B_np, E4, (1, K), N, K, 0, M, 1.0, 1.0, threads=THREADS)
        rel = np.abs(to_np_bits(D).astype(np.float64) - ref) / sabs
        bound = 1e-5 if K <= 2048 else (K / 32) * 2.0 ** -23
        assert rel.max() <= bound, (K, rel.max(), bound)
        assert np.all(to_np_bits(D).astype(np.float64) <= ref * (1 + 2.0 ** -23))     # truncation never overshoots


@pytest.mark.parametrize("M,K,ma,mb", [(128, 2048, api.MAJOR_K, api.MAJOR_K), (384, 2064, api.MAJOR_MN, api.MAJOR_MN),
                                        (128, 4096, api.MAJOR_K, api.MAJOR_MN), (384, 6176, api.MAJOR_K, api.MAJOR_K),
                                        (384, 16384, api.MAJOR_MN, api.MAJOR_MN), (128, 49152, api.MAJOR_K, api.MAJOR_K)])
def test_split_accumulation_same_sign(M, K, ma, mb):
    """ACC_SPLIT on all-positive operands (the accumulator's worst case): partial sums every 2048 of K are
    added with round-to-nearest, so 1e-5 * sum|ab| holds at every K (M = 128: one CTA per tile; 384: CTA
    pairs, the second pair half empty)"""
    rng = np.random.default_rng(1000 + K + M)
    N = 264
    A_np = _codes(rng, E4, (M, K) if ma == api.MAJOR_K else (K, M), spread=1.0) & 0x7F
    B_np = _codes(rng, E5, (N, K) if mb == api.MAJOR_K else (K, N), spread=1.0) & 0x7F
    _run(A_np, E4, ma, B_np, E5, mb, M, N, K, torch.float32, sa_inv=1.0, sb_inv=1.0, acc=api.ACC_SPLIT)   # checks 1e-5 * sum|ab|
    if K <= 6176:
        _run(A_np, E4, ma, B_np, E5, mb, M, N, K, torch.bfloat16, sa_inv=1.0, sb_inv=1.0, acc=api.ACC_SPLIT)


@pytest.mark.parametrize("M,N,K", [(129, 257, 2048 + 129), (300, 520, 4096 + 200), (128, 256, 8192), (1, 8, 2064)])
@pytest.mark.parametrize("ma,mb", [(api.MAJOR_K, api.MAJOR_MN), (api.MAJOR_K, api.MAJOR_K), (api.MAJOR_MN, api.MAJOR_K)])
def test_split_accumulation_mixed_sign_ragged(M, N, K, ma, mb):
    """ACC_SPLIT on the usual mixed-sign codes: ragged M, N and K (a last chunk shorter than 2048, a last
    K-block shorter than 128)"""
    rng = np.random.default_rng(M * 7 + N * 3 + K)
    A_np = _codes(rng, E5, (M, K) if ma == api.MAJOR_K else (K, M))
    B_np = _codes(rng, E4, (N, K) if mb == api.MAJOR_K else (K, N))
    _run(A_np, E5, ma, B_np, E4, mb, M, N, K, torch.float32, acc=api.ACC_SPLIT)
    if mb == api.MAJOR_MN:
        _run(A_np, E5, ma, B_np, E4, mb, M, N, K, torch.bfloat16, acc=api.ACC_SPLIT)


def test_split_accumulation_many_tiles():
    """more tile pairs than SM pairs with two chunks per tile: the two TMEM accumulators change owner
    (chunk parity) from tile to tile"""
    rng = np.random.default_rng(6)
    M, N, K = 2600, 3904, 2304                   # 11 x 16 = 176 tile pairs
    A_np = _codes(rng, E4, (M, K)) & 0x7F
    B_np = _codes(rng, E4, (K, N)) & 0x7F
    D = torch.empty(M, N, dtype=torch.float32, device=DEV)
    amax = _scalar(0.0)
    api.fp8_gemm(torch.from_numpy(A_np).to(DEV), E4, api.MAJOR_K, torch.from_numpy(B_np).to(DEV), E4, api.MAJOR_MN, D,
                 _scalar(0.25), _scalar(0.125), amax, acc=api.ACC_SPLIT)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    t = oracle.decode_table(E4)
    ref = (t[A_np] @ t[B_np]) * (0.25 * 0.125)   # all terms positive: ref is also sum|ab| (library fp64 matmul as reference)
    got = to_np_bits(D)
    assert (np.abs(got.astype(np.float64) - ref) / ref).max() < 1e-5
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1))


def test_split_equals_fast_up_to_2048():
    """within one 2048-wide chunk both modes run the same additions: identical bits"""
    rng = np.random.default_rng(5)
    for K in (512, 1024, 1040, 2048):
        M, N = 256, 512
        A = torch.from_numpy(_codes(rng, E4, (M, K))).to(DEV)
        B = torch.from_numpy(_codes(rng, E4, (N, K))).to(DEV)
        D0 = torch.empty(M, N, dtype=torch.float32, device=DEV)
        D1 = torch.empty_like(D0)
        api.fp8_gemm(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, D0, _scalar(1.0), _scalar(1.0), acc=api.ACC_FAST)
        api.fp8_gemm(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, D1, _scalar(1.0), _scalar(1.0), acc=api.ACC_SPLIT)
        torch.cuda.synchronize()
        assert torch.equal(D0.view(torch.int32), D1.view(torch.int32))


def test_split_accumulation_other_entry_points():
    """ACC_SPLIT through the FP8-output, per-channel-scale and batched entry points on all-positive codes at
    K = 6144 + 64 (three full chunks and a short one)"""
    rng = np.random.default_rng(4242)
    M, N, K = 384, 520, 6144 + 64
    A_np = _codes(rng, E4, (M, K), spread=1.0) & 0x7F
    B_np = _codes(rng, E4, (N, K), spread=1.0) & 0x7F
    A, B = torch.from_numpy(A_np).to(DEV), torch.from_numpy(B_np).to(DEV)
    ref, sabs = oracle.gemm_rows(A_np, E4, (K, 1), B_np, E4, (1, K), N, K, 0, M, 0.5, 0.25, threads=THREADS)
    # FP8 output
    scale_d = float(oracle.scale_from_amax(np.float32(np.abs(ref).max()), E4)[0])
    ldd = (N + 15) // 16 * 16
    D8_full = torch.full((M + 1, ldd), 0xA5, dtype=torch.uint8, device=DEV)
    amax = _scalar(-1.0)
    api.fp8_gemm_fp8out(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, D8_full[:M, :N], E4, _scalar(0.5), _scalar(0.25), _scalar(scale_d),
                        amax, acc=api.ACC_SPLIT)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert bool((D8_full[M:, :] == 0xA5).all()) and bool((D8_full[:M, N:] == 0xA5).all())
    enc = lambda y: oracle.quantize(y.reshape(-1), 1.0, E4, threads=THREADS).reshape(y.shape)
    assert check_gemm_fp8out(D8_full[:M, :N].cpu().numpy(), ref, sabs, scale_d, enc)[0].all()
    assert abs(amax.item() - np.abs(ref).max()) <= 1e-5 * np.abs(ref).max()
    # per-channel inverse scales of B
    sv = np.exp2(rng.integers(-3, 3, size=N)).astype(np.float32) * np.float32(0.3)
    refc, sabsc = oracle.gemm_rows_colscale(A_np, E4, (K, 1), B_np, E4, (1, K), N, K, 0, M, 0.5, sv, threads=THREADS)
    Dc = torch.empty(M, N, dtype=torch.float32, device=DEV)
    api.fp8_gemm_channel_scales(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, Dc, _scalar(0.5), torch.from_numpy(sv).to(DEV), acc=api.ACC_SPLIT)
    torch.cuda.synchronize()
    assert (np.abs(to_np_bits(Dc).astype(np.float64) - refc) / sabsc).max() < 1e-5
    # batched: three members, the same B for each, A rolled by member
    Ab = torch.stack([A.roll(b, 0) for b in range(3)])
    Bb = torch.stack([B, B, B])
    Db = torch.empty(3, M, N, dtype=torch.float32, device=DEV)
    api.fp8_gemm_batched(Ab, E4, api.MAJOR_K, Bb, E4, api.MAJOR_K, Db, _scalar(0.5), _scalar(0.25), acc=api.ACC_SPLIT)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    got = to_np_bits(Db).astype(np.float64)
    for b in range(3):
        assert (np.abs(got[b] - np.roll(ref, b, 0)) / np.roll(sabs, b, 0)).max() < 1e-5, b


def test_many_tiles_persistent_schedule():
    """more tiles than SMs so that every CTA walks several tiles and both accumulators wrap"""
    rng = np.random.default_rng(3)
    M, N, K = 128 * 21, 256 * 15, 256            # 315 tiles
    A_np = _codes(rng, E4, (M, K))
    B_np = _codes(rng, E4, (K, N))
    A = torch.from_numpy(A_np).to(DEV)
    B = torch.from_numpy(B_np).to(DEV)
    D = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    amax = _scalar(0.0)
    api.fp8_gemm(A, E4, api.MAJOR_K, B, E4, api.MAJOR_MN, D, _scalar(0.25), _scalar(0.125), amax)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    # E4M3 x E4M3: the fp64 matmul of the decoded operands is the exact sum (library routine as reference)
    t = oracle.decode_table(E4)
    ref = (t[A_np] @ t[B_np]) * (0.25 * 0.125)
    sabs = (np.abs(t[A_np]) @ np.abs(t[B_np])) * (0.25 * 0.125)
    got = to_np_bits(D)
    ok, literal = check_gemm_bf16(got, ref, sabs, oracle.round_bf16_from_f64)
    assert ok.all(), np.argwhere(~ok)[:4].tolist()
    assert literal.mean() > 0.999
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1))


def test_special_codes_and_degenerate_shapes():
    rng = np.random.default_rng(5)
    M, N, K = 128, 256, 256
    A_np = _codes(rng, E5, (M, K))
    B_np = _codes(rng, E4, (N, K))
    A_np[3, 7] = 0x7C          # +Inf
    A_np[9, 1] = 0xFC          # -Inf
    A_np[20, 2] = 0x7E         # E5M2 NaN
    B_np[40, 100] = 0x7F       # E4M3 NaN
    A_np[50, 5] = 0x7C
    B_np[:, 5] = np.where(np.arange(N) % 2 == 0, 0x00, B_np[:, 5])      # Inf * 0 on even columns of row 50
    got, ref, _ = _run(A_np, E5, api.MAJOR_K, B_np, E4, api.MAJOR_K, M, N, K, torch.float32, want_amax=False)
    assert np.isnan(ref[20]).all() and np.isnan(ref[:, 40]).all() and np.isinf(ref[3]).any()
    # K = 0 writes zeros, amax 0; M*N = 0 is a no-op
    D = torch.full((64, 64), 5.0, dtype=torch.bfloat16, device=DEV)
    amax = _scalar(9.0)
    A0 = torch.empty((64, 0), dtype=torch.uint8, device=DEV)
    B0 = torch.empty((64, 0), dtype=torch.uint8, device=DEV)
    api.fp8_gemm(A0, E4, api.MAJOR_K, B0, E4, api.MAJOR_K, D, _scalar(1.0), _scalar(1.0), amax)
    assert bool((D == 0).all()) and amax.item() == 0.0
    amax.fill_(9.0)
    Dz = torch.empty((0, 64), dtype=torch.bfloat16, device=DEV)
    Az = torch.empty((0, 32), dtype=torch.uint8, device=DEV)
    Bz = torch.empty((64, 32), dtype=torch.uint8, device=DEV)
    api.fp8_gemm(Az, E4, api.MAJOR_K, Bz, E4, api.MAJOR_K, Dz, _scalar(1.0), _scalar(1.0), amax)
    assert amax.item() == 0.0


# ------------------------------------------------ FP8-output epilogue --

@pytest.mark.parametrize("role", list(ROLES))
@pytest.mark.parametrize("fd", [E4, E5])
@pytest.mark.parametrize("shape", [(384, 768, 640), (129, 257, 129), (100, 40, 48), (300, 520, 200)])
def test_fp8_output_epilogue(role, fd, shape):
    """results converted to FP8 before they are written; amax reported before the output scale"""
    fa, fb = ROLES[role]
    M, N, K = shape
    rng = np.random.default_rng(2000 + list(ROLES).index(role) * 8 + fd * 4 + M)
    ma, mb = (api.MAJOR_K, api.MAJOR_MN) if role == "fprop" else (api.MAJOR_K, api.MAJOR_K) if role == "dgrad" else (api.MAJOR_MN, api.MAJOR_MN)
    A_np = _codes(rng, fa, (M, K) if ma == api.MAJOR_K else (K, M))
    B_np = _codes(rng, fb, (N, K) if mb == api.MAJOR_K else (K, N))
    A_buf, B_buf = _pad_cols(A_np), _pad_cols(B_np)
    A = torch.from_numpy(A_buf).to(DEV)[:, : A_np.shape[1]]
    B = torch.from_numpy(B_buf).to(DEV)[:, : B_np.shape[1]]
    ldd = (N + 15) // 16 * 16
    sa_inv, sb_inv = 0.013, 0.5
    a_str = (A_buf.shape[1], 1) if ma == api.MAJOR_K else (1, A_buf.shape[1])
    b_str = (1, B_buf.shape[1]) if mb == api.MAJOR_K else (B_buf.shape[1], 1)
    ref, sabs = oracle.gemm_rows(A_buf, fa, a_str, B_buf, fb, b_str, N, K, 0, M, sa_inv, sb_inv, threads=THREADS)
    want_amax = np.abs(ref).max()
    # a scale chosen as the method would: from (an estimate of) the output's own maximum; and one that overflows
    for scale_d, overflow in ((float(oracle.scale_from_amax(np.float32(want_amax), fd)[0]), api.SATURATE),
                              (float(oracle.scale_from_amax(np.float32(want_amax), fd)[0]) * 8.0, api.SATURATE),
                              (float(oracle.scale_from_amax(np.float32(want_amax), fd)[0]) * 8.0, api.NOSAT)):
        D_full = torch.full((M + 1, ldd), 0xA5, dtype=torch.uint8, device=DEV)
        D = D_full[:M, :N]
        amax = _scalar(-1.0)
        api.fp8_gemm_fp8out(A, fa, ma, B, fb, mb, D, fd, _scalar(sa_inv), _scalar(sb_inv), _scalar(scale_d), amax, overflow)
        torch.cuda.synchronize()
        assert api.fp8_async_status()[0] == 0
        assert bool((D_full[M:, :] == 0xA5).all()) and bool((D_full[:M, N:] == 0xA5).all()), "wrote outside D"
        enc = lambda y: oracle.quantize(y.reshape(-1), 1.0, fd, overflow, threads=THREADS).reshape(y.shape)
        ok, exact = check_gemm_fp8out(D.cpu().numpy(), ref, sabs, scale_d, enc)
        assert ok.all(), "%d of %d codes out of tolerance at %s" % ((~ok).sum(), ok.size, np.argwhere(~ok)[:4].tolist())
        assert exact.mean() > 0.99, "only %.4f of the codes equal the conversion of the reference itself" % exact.mean()
        # amax of the unscaled, unconverted result: within the accumulation tolerance of the oracle's
        got_amax = float(amax.item())
        lo = np.max(np.abs(ref) - 1e-5 * sabs) * (1 - 2.0 ** -22)
        hi = np.max(np.abs(ref) + 1e-5 * sabs) * (1 + 2.0 ** -22)
        assert lo <= got_amax <= hi, (got_amax, lo, hi)


def test_fp8_output_special_values_and_k0():
    rng = np.random.default_rng(31)
    M, N, K = 256, 256, 128
    A_np = _codes(rng, E5, (M, K))
    B_np = _codes(rng, E4, (N, K))
    A_np[3, 7] = 0x7C          # +Inf  -> row 3 is +-Inf or NaN
    B_np[40, 100] = 0x7F       # NaN   -> column 40 is NaN
    A = torch.from_numpy(A_np).to(DEV)
    B = torch.from_numpy(B_np).to(DEV)
    ref, sabs = oracle.gemm_rows(A_np, E5, (K, 1), B_np, E4, (1, K), N, K, 0, M, 1.0, 1.0, threads=THREADS)
    for fd in (E4, E5):
        D = torch.empty(M, N, dtype=torch.uint8, device=DEV)
        api.fp8_gemm_fp8out(A, E5, api.MAJOR_K, B, E4, api.MAJOR_K, D, fd, _scalar(1.0), _scalar(1.0), _scalar(0.01))
        enc = lambda y: oracle.quantize(y.reshape(-1), 1.0, fd, threads=THREADS).reshape(y.shape)
        ok, _ = check_gemm_fp8out(D.cpu().numpy(), ref, sabs, 0.01, enc)
        assert ok.all(), np.argwhere(~ok)[:4].tolist()
        got = D.cpu().numpy()
        assert ((got[:, 40] & 0x7F) == 0x7F).all()                      # NaN codes
        inf_row = got[3, np.isinf(ref[3])]
        assert ((inf_row & 0x7F) == (0x7F if fd == E4 else 0x7C)).all()  # Inf -> NaN (E4M3) / Inf (E5M2), never the maximum
    D = torch.full((64, 64), 0x11, dtype=torch.uint8, device=DEV)
    amax = _scalar(3.0)
    A0 = torch.empty((64, 0), dtype=torch.uint8, device=DEV)
    api.fp8_gemm_fp8out(A0, E4, api.MAJOR_K, A0, E4, api.MAJOR_K, D, E4, _scalar(1.0), _scalar(1.0), _scalar(1.0), amax)
    assert bool((D == 0).all()) and amax.item() == 0.0


# ------------------------------------------------------ batched (attention-style) products --

@pytest.mark.parametrize("case", ["scores", "context", "ragged"])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_batched_gemm(case, out_dtype):
    """the two attention products: scores = Q.K^T (both operands K-major, K = head dim) and
    context = P.V (V stored [S, d]: N contiguous), batch = heads; plus a ragged case with padded pitches"""
    rng = np.random.default_rng({"scores": 1, "context": 2, "ragged": 3}[case])
    if case == "scores":
        batch, M, N, K, ma, mb = 6, 320, 320, 128, api.MAJOR_K, api.MAJOR_K
    elif case == "context":
        batch, M, N, K, ma, mb = 5, 256, 128, 384, api.MAJOR_K, api.MAJOR_MN
    else:
        batch, M, N, K, ma, mb = 3, 130, 72, 100, api.MAJOR_MN, api.MAJOR_K
    a_shape = (M, K) if ma == api.MAJOR_K else (K, M)
    b_shape = (N, K) if mb == api.MAJOR_K else (K, N)
    A_np = np.stack([_pad_cols(_codes(rng, E4, a_shape)) for _ in range(batch)])
    B_np = np.stack([_pad_cols(_codes(rng, E4, b_shape)) for _ in range(batch)])
    A = torch.from_numpy(A_np).to(DEV)[:, :, : a_shape[1]]
    B = torch.from_numpy(B_np).to(DEV)[:, :, : b_shape[1]]
    esz = 2 if out_dtype == torch.bfloat16 else 4
    ldd = (N * esz + 15) // 16 * 16 // esz
    D_full = torch.full((batch, M + 1, ldd), 777.0, dtype=out_dtype, device=DEV)
    D = D_full[:, :M, :N]
    amax = _scalar(-1.0)
    api.fp8_gemm_batched(A, E4, ma, B, E4, mb, D, _scalar(0.25), _scalar(0.5), amax)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert bool((D_full[:, M:, :] == 777.0).all()) and bool((D_full[:, :M, N:] == 777.0).all()), "wrote outside D"
    a_str = (A_np.shape[2], 1) if ma == api.MAJOR_K else (1, A_np.shape[2])
    b_str = (1, B_np.shape[2]) if mb == api.MAJOR_K else (B_np.shape[2], 1)
    got = to_np_bits(D)
    for b in range(batch):
        ref, sabs = oracle.gemm_rows(A_np[b], E4, a_str, B_np[b], E4, b_str, N, K, 0, M, 0.25, 0.5, threads=THREADS)
        if out_dtype == torch.float32:
            ok, worst = check_gemm_f32(got[b], ref, sabs)
        else:
            ok, _ = check_gemm_bf16(got[b], ref, sabs, oracle.round_bf16_from_f64)
        assert ok.all(), (b, np.argwhere(~ok)[:4].tolist())
    a2 = _scalar(-1.0)
    api.fp8_amax(D.contiguous(), a2)
    assert amax.cpu().numpy().view(np.uint32)[0] == a2.cpu().numpy().view(np.uint32)[0]


def test_batched_gemm_interleaved_heads():
    """attention heads stored side by side inside a row ([S, H, d] tensors): the batch stride of the read-only
    operands is the head width, smaller than a matrix; scores = Q_h . K_h^T for every head in one launch"""
    rng = np.random.default_rng(17)
    S, H, Dh = 200, 5, 64
    Q_np = _codes(rng, E4, (S, H * Dh))
    K_np = _codes(rng, E4, (S, H * Dh))
    Q = torch.from_numpy(Q_np).to(DEV).view(S, H, Dh).permute(1, 0, 2)        # [H, S, Dh] view, strides (Dh, H*Dh, 1)
    Kt = torch.from_numpy(K_np).to(DEV).view(S, H, Dh).permute(1, 0, 2)
    ldd = 200
    D = torch.empty(H, S, ldd, dtype=torch.float32, device=DEV)[:, :, :S]
    amax = _scalar(-1.0)
    api.fp8_gemm_batched(Q, E4, api.MAJOR_K, Kt, E4, api.MAJOR_K, D, _scalar(0.25), _scalar(0.5), amax)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    got = to_np_bits(D)
    for h in range(H):
        qa = np.ascontiguousarray(Q_np[:, h * Dh:(h + 1) * Dh])
        ka = np.ascontiguousarray(K_np[:, h * Dh:(h + 1) * Dh])
        ref, sabs = oracle.gemm_rows(qa, E4, (Dh, 1), ka, E4, (1, Dh), S, Dh, 0, S, 0.25, 0.5, threads=THREADS)
        ok, worst = check_gemm_f32(got[h], ref, sabs)
        assert ok.all(), (h, worst)
    assert amax.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1))


# ------------------------------------------------------------------ split-K (few output tiles) --

@pytest.mark.parametrize("M,N,K", [(16, 2048, 16384), (128, 1024, 8192), (200, 512, 4096), (1, 256, 65536), (64, 260, 4096)])
@pytest.mark.parametrize("ma,mb", [(api.MAJOR_K, api.MAJOR_K), (api.MAJOR_K, api.MAJOR_MN), (api.MAJOR_MN, api.MAJOR_K)])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_splitk_gemm(M, N, K, ma, mb, out_dtype):
    """a few rows against a wide weight matrix: K is cut into slices (the library says how many), partial
    products are summed in slice order; same tolerance as fp8_gemm, amax of the stored output, guard bands"""
    rng = np.random.default_rng(M + N + K)
    A_np = _codes(rng, E5, (M, K) if ma == api.MAJOR_K else (K, M), spread=3.0)
    B_np = _codes(rng, E4, (N, K) if mb == api.MAJOR_K else (K, N), spread=3.0)
    A_buf, B_buf = _pad_cols(A_np), _pad_cols(B_np)                # row pitches that are multiples of 16 bytes
    A = torch.from_numpy(A_buf).to(DEV)[:, : A_np.shape[1]]
    B = torch.from_numpy(B_buf).to(DEV)[:, : B_np.shape[1]]
    splits, nbytes = api.fp8_gemm_splitk_workspace(M, N, K)
    assert splits >= 1 and nbytes == (splits * M * N * 4 if splits > 1 else 0)
    if (M, N, K) != (64, 260, 4096):
        assert splits > 1, "these shapes leave most SMs idle without slices"
    ws = torch.full((nbytes // 4 + 64,), float("nan"), dtype=torch.float32, device=DEV)
    ldd = N + 3                                                   # only element alignment is needed with slices
    if splits == 1:
        esz = 2 if out_dtype == torch.bfloat16 else 4
        ldd = (N * esz + 15) // 16 * 16 // esz
    D_full = torch.full((M + 1, ldd), 777.0, dtype=out_dtype, device=DEV)
    D = D_full[:M, :N]
    amax = _scalar(-1.0)
    api.fp8_gemm_splitk(A, E5, ma, B, E4, mb, D, _scalar(0.013), _scalar(0.5), ws[: nbytes // 4] if nbytes else None, amax)
    torch.cuda.synchronize()
    assert api.fp8_async_status()[0] == 0
    assert bool((D_full[M:, :] == 777.0).all()) and bool((D_full[:M, N:] == 777.0).all()), "wrote outside D"
    assert bool(torch.isnan(ws[nbytes // 4:]).all()), "wrote past the workspace"
    a_str = (A_buf.shape[1], 1) if ma == api.MAJOR_K else (1, A_buf.shape[1])
    b_str = (1, B_buf.shape[1]) if mb == api.MAJOR_K else (B_buf.shape[1], 1)
    ref, sabs = oracle.gemm_rows(A_buf, E5, a_str, B_buf, E4, b_str, N, K, 0, M, 0.013, 0.5, threads=THREADS)
    got = to_np_bits(D)
    if out_dtype == torch.float32:
        ok, worst = check_gemm_f32(got, ref, sabs)
    else:
        ok, _ = check_gemm_bf16(got, ref, sabs, oracle.round_bf16_from_f64)
    assert ok.all(), np.argwhere(~ok)[:4].tolist()
    a2 = _scalar(-1.0)
    api.fp8_amax(D.contiguous(), a2)
    assert amax.cpu().numpy().view(np.uint32)[0] == a2.cpu().numpy().view(np.uint32)[0] == oracle.amax_bits(got.reshape(-1))


def test_splitk_workspace_errors_and_large_problems_take_the_plain_path():
    assert api.fp8_gemm_splitk_workspace(8192, 16384, 4096) == (1, 0)       # tiles fill the GPU: no slices
    assert api.fp8_gemm_splitk_workspace(16, 4096, 1024) == (1, 0)          # short contraction
    assert api.fp8_gemm_splitk_workspace(16, 4098, 16384) == (1, 0)         # N not a multiple of 4
    M, N, K = 16, 2048, 8192
    splits, nbytes = api.fp8_gemm_splitk_workspace(M, N, K)
    assert splits > 1
    A = torch.zeros(M, K, dtype=torch.uint8, device=DEV)
    B = torch.zeros(N, K, dtype=torch.uint8, device=DEV)
    D = torch.empty(M, N, dtype=torch.bfloat16, device=DEV)
    one = _scalar(1.0)
    with pytest.raises(api.Fp8Error, match="status 1"):
        api.fp8_gemm_splitk(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, D, one, one, None)
    small = torch.empty(nbytes // 4 - 4, dtype=torch.float32, device=DEV)
    with pytest.raises(api.Fp8Error, match="status 3"):
        api.fp8_gemm_splitk(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, D, one, one, small)
    odd = torch.empty(nbytes // 4 + 4, dtype=torch.float32, device=DEV)[1:]
    with pytest.raises(api.Fp8Error, match="status 4"):
        api.fp8_gemm_splitk(A, E4, api.MAJOR_K, B, E4, api.MAJOR_K, D, one, one, odd)
