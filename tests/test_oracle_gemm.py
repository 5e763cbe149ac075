"""Pins for the oracle's FP8 GEMM: exact rational brute force on tiny inputs,
numpy's float64 matmul where the sum is exact, structured operands with closed
forms, and special-value propagation."""
from fractions import Fraction

import numpy as np
import pytest

import oracle
from oracle import E4M3, E5M2


def _finite_codes(rng, fmt, shape):
    c = rng.integers(0, 256, size=shape, dtype=np.uint16).astype(np.uint8)
    t = oracle.decode_table(fmt)
    bad = ~np.isfinite(t[c])
    c[bad] = 0x38 if fmt == E4M3 else 0x3C        # 1.0
    return c


def _frac_table(fmt):
    t = oracle.decode_table(fmt)
    return [Fraction(float(v)) if np.isfinite(v) else None for v in t]


ROLES = [(E4M3, E4M3), (E5M2, E4M3), (E4M3, E5M2)]     # forward, dgrad, wgrad operand formats


@pytest.mark.parametrize("fa,fb", ROLES)
def test_gemm_equals_exact_rational_brute_force(fa, fb):
    rng = np.random.default_rng(100 + fa * 2 + fb)
    M, N, K = 5, 7, 33
    A = _finite_codes(rng, fa, (M, K))
    B = _finite_codes(rng, fb, (K, N))
    ta, tb = _frac_table(fa), _frac_table(fb)
    sa_inv, sb_inv = np.float32(0.0371), np.float32(1.0 / 3.0)
    ref, sab = oracle.gemm_rows(A, fa, (K, 1), B, fb, (N, 1), N, K, 0, M, sa_inv, sb_inv)
    alpha = Fraction(float(sa_inv)) * Fraction(float(sb_inv))
    for i in range(M):
        for j in range(N):
            exact = sum(ta[A[i, k]] * tb[B[k, j]] for k in range(K)) * alpha
            exabs = sum(abs(ta[A[i, k]] * tb[B[k, j]]) for k in range(K)) * alpha
            assert abs(Fraction(float(ref[i, j])) - exact) <= Fraction(1, 10 ** 14) * exabs
            assert abs(Fraction(float(sab[i, j])) - exabs) <= Fraction(1, 10 ** 14) * exabs
            # the 128-bit fixed-point dot product is the exact sum
            integer, ue = oracle.dot_exact(A[i, :], fa, B[:, j].copy(), fb)
            assert Fraction(integer) * Fraction(2) ** ue * alpha == exact


def test_e4m3_gemm_is_exact_and_equals_numpy_float64_matmul():
    rng = np.random.default_rng(5)
    M, N, K = 16, 24, 512
    A = _finite_codes(rng, E4M3, (M, K))
    B = _finite_codes(rng, E4M3, (K, N))
    t = oracle.decode_table(E4M3)
    ref, sab = oracle.gemm_rows(A, E4M3, (K, 1), B, E4M3, (N, 1), N, K, 0, M, 1.0, 1.0)
    # every product is a multiple of 2^-18 and the sum stays far below 2^53 units: any order is exact
    assert np.array_equal(ref, t[A] @ t[B])
    assert np.array_equal(sab, np.abs(t[A]) @ np.abs(t[B]))


@pytest.mark.parametrize("fa,fb", ROLES)
def test_operand_layouts_give_the_same_numbers(fa, fb):
    rng = np.random.default_rng(9)
    M, N, K = 6, 10, 40
    A = _finite_codes(rng, fa, (M, K))
    B = _finite_codes(rng, fb, (K, N))
    base, _ = oracle.gemm_rows(A, fa, (K, 1), B, fb, (N, 1), N, K, 0, M, 0.5, 0.25)
    At = np.ascontiguousarray(A.T)          # stored [K, M]: the row index is the contiguous one
    Bt = np.ascontiguousarray(B.T)          # stored [N, K]: the contraction index is the contiguous one
    alt, _ = oracle.gemm_rows(At, fa, (1, M), Bt, fb, (1, K), N, K, 0, M, 0.5, 0.25)
    assert np.array_equal(base, alt)
    ii = np.array([0, 5, 3, 2], dtype=np.int64)
    jj = np.array([9, 0, 4, 4], dtype=np.int64)
    s, _ = oracle.gemm_samples(At, fa, (1, M), Bt, fb, (1, K), K, ii, jj, 0.5, 0.25)
    assert np.array_equal(s, base[ii, jj])
    part, _ = oracle.gemm_rows(A, fa, (K, 1), B, fb, (N, 1), N, K, 2, 5, 0.5, 0.25, threads=2)
    assert np.array_equal(part, base[2:5])


def test_structured_operands_closed_forms():
    rng = np.random.default_rng(12)
    K = 64
    A = _finite_codes(rng, E5M2, (8, K))
    ta = oracle.decode_table(E5M2)
    one, zero = 0x38, 0x00
    eye = np.where(np.eye(K, dtype=bool), one, zero).astype(np.uint8)
    ref, _ = oracle.gemm_rows(A, E5M2, (K, 1), eye, E4M3, (K, 1), K, K, 0, 8, 0.125, 2.0)
    assert np.array_equal(ref, ta[A] * 0.25)                 # identity B returns the decoded A, unscaled once
    ones = np.full((K, 1), one, dtype=np.uint8)
    ref, sab = oracle.gemm_rows(A, E5M2, (K, 1), ones, E4M3, (1, 1), 1, K, 0, 8, 1.0, 1.0)
    assert np.allclose(ref[:, 0], ta[A].sum(axis=1), rtol=1e-15, atol=0)
    assert np.allclose(sab[:, 0], np.abs(ta[A]).sum(axis=1), rtol=1e-15, atol=0)
    ref, sab = oracle.gemm_rows(A, E5M2, (K, 1), eye, E4M3, (K, 1), K, 0, 0, 8, 1.0, 1.0)   # K = 0
    assert np.all(ref == 0) and np.all(sab == 0)


def test_special_codes_propagate():
    K = 8
    one = 0x38
    A = np.full((1, K), 0x3C, dtype=np.uint8)        # E5M2 ones
    B = np.full((K, 1), one, dtype=np.uint8)
    A[0, 3] = 0x7C                                   # +Inf
    ref, _ = oracle.gemm_rows(A, E5M2, (K, 1), B, E4M3, (1, 1), 1, K, 0, 1, 1.0, 1.0)
    assert ref[0, 0] == np.inf
    B[3, 0] = 0x00                                   # Inf * 0
    ref, _ = oracle.gemm_rows(A, E5M2, (K, 1), B, E4M3, (1, 1), 1, K, 0, 1, 1.0, 1.0)
    assert np.isnan(ref[0, 0])
    A[0, 3] = 0x3C
    B[5, 0] = 0x7F                                   # E4M3 NaN
    ref, _ = oracle.gemm_rows(A, E5M2, (K, 1), B, E4M3, (1, 1), 1, K, 0, 1, 1.0, 1.0)
    assert np.isnan(ref[0, 0])
    assert oracle.dot_exact(A[0], E5M2, B[:, 0].copy(), E4M3) is None


def test_per_channel_scales_reduce_to_per_tensor_routines():
    """Section 4.2: per-channel weight scales.  Channel by channel the functions equal the per-tensor
    ones (pinned separately), and a column-scaled GEMM is the per-tensor GEMM column by column."""
    rng = np.random.default_rng(40)
    x = (rng.standard_normal((37, 53)) * np.exp2(rng.uniform(-4, 4, size=(37, 53)))).astype(np.float32)
    x[5, 7] = np.nan
    for axis in (0, 1):
        am = oracle.amax_channels(x, axis)
        chans = x.T if axis == 0 else x
        want = np.array([oracle.amax_bits(np.ascontiguousarray(ch)) for ch in chans], dtype=np.uint32)
        assert np.array_equal(am.view(np.uint32), want)
        am = np.where(np.isnan(am), 1.0, am).astype(np.float32)
        s, si = oracle.scales_from_amax(am, E4M3)
        assert np.array_equal(s, np.float32(448.0) / am)                 # numpy float32 division
        q = oracle.quantize_channels(x, s, axis, E4M3)
        for ci, ch in enumerate(chans):
            got = q[:, ci] if axis == 0 else q[ci]
            assert np.array_equal(got, oracle.quantize(np.ascontiguousarray(ch), s[ci], E4M3))
    M, N, K = 6, 9, 40
    A = _finite_codes(rng, E4M3, (M, K))
    B = _finite_codes(rng, E4M3, (K, N))
    sv = np.exp2(rng.uniform(-6, 2, size=N)).astype(np.float32)
    ref, sab = oracle.gemm_rows_colscale(A, E4M3, (K, 1), B, E4M3, (N, 1), N, K, 0, M, 0.5, sv)
    for j in range(N):
        r1, s1 = oracle.gemm_rows(A, E4M3, (K, 1), B, E4M3, (N, 1), N, K, 0, M, 0.5, sv[j])
        assert np.array_equal(ref[:, j], r1[:, j]) and np.array_equal(sab[:, j], s1[:, j])


def _nearest_code(y32, fmt):
    """Saturating round-to-nearest-even by exhaustive search over the decode table (reads only the table,
    pinned separately against Table 1): the lowest code among the nearest magnitudes, moved up one when the
    next magnitude is equally near and the found one is odd; beyond the midpoint past the maximum, the maximum."""
    t = oracle.decode_table(fmt)
    maxmag = 0x7E if fmt == E4M3 else 0x7B
    ext = np.concatenate([t[: maxmag + 1], [480.0 if fmt == E4M3 else 65536.0]])
    a = np.abs(y32.astype(np.float64)).reshape(-1)
    d = np.abs(a[:, None] - ext[None, :])
    best = np.argmin(d, axis=1)
    nxt = np.minimum(best + 1, ext.size - 1)
    rows = np.arange(a.size)
    tie = (d[rows, nxt] == d[rows, best]) & (nxt != best)
    best = np.where(tie & (best % 2 == 1), nxt, best)
    best = np.minimum(best, maxmag)
    sign = ((y32.reshape(-1).view(np.uint32) >> 31) << 7).astype(np.uint8)
    return (sign | best.astype(np.uint8)).reshape(y32.shape)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_per_channel_routines_equal_numpy_closed_forms(fmt):
    """Section 4.2, per-channel scales, against definitions written with numpy alone: the per-channel amax is
    np.abs(x).max along the other axis; the codes are the nearest-code search applied to x * s broadcast along
    the channel axis (one binary32 multiply); the column-scaled product is the plain float64 matmul of the
    decoded operands times sa_inv * sb_inv[j].  A row/column mix-up, a wrong pitch or a scale applied along the
    wrong axis fails here on the non-square shapes."""
    rng = np.random.default_rng(77 + fmt)
    rows, cols = 29, 45
    x = (rng.standard_normal((rows, cols)) * np.exp2(rng.uniform(-5, 5, size=(rows, cols)))).astype(np.float32)
    x[:, 3] *= 64.0                                  # a column and a row that dominate their channels
    x[11, :] *= 32.0
    for axis in (0, 1):
        am = oracle.amax_channels(x, axis)
        assert am.shape == ((cols,) if axis == 0 else (rows,))
        assert np.array_equal(am, np.abs(x).max(axis=axis))
        s = (np.float32(oracle.FMT_MAX[fmt]) / am).astype(np.float32)
        y = x * (s[None, :] if axis == 0 else s[:, None])          # binary32 multiply, broadcast along the channel axis
        assert np.array_equal(oracle.quantize_channels(x, s, axis, fmt), _nearest_code(y, fmt))
        # the same through bf16 inputs (exact widening)
        xb = (x.view(np.uint32) >> 16).astype(np.uint16)
        xw = (xb.astype(np.uint32) << 16).view(np.float32)
        amb = oracle.amax_channels(xb, axis)
        assert np.array_equal(amb, np.abs(xw).max(axis=axis))
        yb = xw * (s[None, :] if axis == 0 else s[:, None])
        assert np.array_equal(oracle.quantize_channels(xb, s, axis, fmt), _nearest_code(yb, fmt))
    # NaN propagates per channel only
    xn = x.copy()
    xn[5, 7] = np.nan
    a0, a1 = oracle.amax_channels(xn, 0), oracle.amax_channels(xn, 1)
    assert np.isnan(a0[7]) and np.isnan(a1[5]) and np.isnan(a0).sum() == 1 and np.isnan(a1).sum() == 1
    # column-scaled GEMM = float64 matmul of the decoded codes, column j times sa_inv * sb_inv[j]
    M, N, K = 7, 10, 48
    A = _finite_codes(rng, E4M3, (M, K))
    B = _finite_codes(rng, fmt, (K, N))
    sv = np.exp2(rng.uniform(-6, 2, size=N)).astype(np.float32)
    sa_inv = np.float32(0.37)
    ref, sab = oracle.gemm_rows_colscale(A, E4M3, (K, 1), B, fmt, (N, 1), N, K, 0, M, sa_inv, sv)
    da, db = oracle.decode_table(E4M3)[A], oracle.decode_table(fmt)[B]
    alpha = np.float64(sa_inv) * sv.astype(np.float64)
    want, want_abs = (da @ db) * alpha[None, :], (np.abs(da) @ np.abs(db)) * alpha[None, :]
    assert np.allclose(ref, want, rtol=1e-13, atol=0) and np.allclose(sab, want_abs, rtol=1e-13, atol=0)
    # with B stored transposed ([N, K], strides (1, K)) the same numbers come out
    ref_t, _ = oracle.gemm_rows_colscale(A, E4M3, (K, 1), np.ascontiguousarray(B.T), fmt, (1, K), N, K, 0, M, sa_inv, sv)
    assert np.array_equal(ref_t, ref)
