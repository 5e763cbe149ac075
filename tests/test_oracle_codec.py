"""Pins for the CPU oracle's codec, cast, amax and scale functions.

Nothing here compares the oracle with itself: each check is against a value the
paper prints (tests/golden/table1_fp8_formats.txt), a library routine (numpy
float16 / float32 arithmetic, torch's float8 and bfloat16 casts), a brute-force
nearest-value search, or a closed form.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import E4M3, E5M2, NOSAT, SATURATE

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_fp8_formats.txt")
FMT = {"E4M3": E4M3, "E5M2": E5M2}


def _parse_value(tok):
    if tok in ("inf", "nan"):
        return float(tok)
    if "*2^" in tok:
        m, e = tok.split("*2^")
        return float(m) * 2.0 ** int(e)
    return float(tok)


def _golden_rows():
    rows = []
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        fmt, what, pattern, value = line.split()
        rows.append((fmt, what, pattern, value))
    return rows


def _code_of(pattern):
    return int(pattern.replace(".", ""), 2)


# ------------------------------------------------------------------ decode --

@pytest.mark.parametrize("fmt,what,pattern,value", [r for r in _golden_rows() if r[2] != "-"])
def test_decode_matches_paper_table(fmt, what, pattern, value):
    code = _code_of(pattern)
    want = _parse_value(value)
    for sign in (0, 0x80):
        got = oracle.decode(code | sign, FMT[fmt])
        if np.isnan(want):
            assert np.isnan(got)
        else:
            assert got == (-want if sign else want)
            if want == 0:
                assert np.signbit(got) == bool(sign)


def test_bias_and_binades_match_paper():
    rows = {(f, w): v for f, w, p, v in _golden_rows() if p == "-"}
    for name, fmt, mbits in (("E4M3", E4M3, 3), ("E5M2", E5M2, 2)):
        bias = int(rows[(name, "bias")])
        # code with exponent field == bias and mantissa 0 is 1.0
        assert oracle.decode(bias << mbits, fmt) == 1.0
        t = oracle.decode_table(fmt)[:128]
        finite = t[np.isfinite(t) & (t > 0)]
        binades = set(np.floor(np.log2(finite)).astype(int).tolist())
        assert len(binades) == int(rows[(name, "binades")])
    # without the exponent-1111 normals E4M3 would span one binade less (Section 3.1: 17)
    t = oracle.decode_table(E4M3)[:0x78]
    assert len(set(np.floor(np.log2(t[t > 0])).astype(int).tolist())) == 17


def test_e5m2_is_truncated_half_precision():
    codes = np.arange(256, dtype=np.uint16)
    half = (codes << 8).astype(np.uint16).view(np.float16).astype(np.float64)
    t = oracle.decode_table(E5M2)
    nan = np.isnan(half)
    assert np.array_equal(np.isnan(t), nan)
    assert np.array_equal(t[~nan], half[~nan])
    assert np.array_equal(np.signbit(t[~nan]), np.signbit(half[~nan]))


def test_decode_agrees_with_torch_float8_views():
    codes = torch.arange(256, dtype=torch.uint8)
    for fmt, dt in ((E4M3, torch.float8_e4m3fn), (E5M2, torch.float8_e5m2)):
        lib = codes.view(dt).to(torch.float64).numpy()
        t = oracle.decode_table(fmt)
        assert np.array_equal(np.isnan(t), np.isnan(lib))
        ok = ~np.isnan(t)
        assert np.array_equal(t[ok], lib[ok])


def test_decode_structure():
    for fmt, nfinite in ((E4M3, 126), (E5M2, 123)):
        t = oracle.decode_table(fmt)
        pos = t[:128]
        finite = pos[np.isfinite(pos)]
        assert finite.size == nfinite + 1            # + the zero code
        assert np.all(np.diff(finite) > 0)           # codes order like their values (Section 3.1)
        neg = t[128:]
        same = np.isfinite(pos)
        assert np.array_equal(neg[same], -pos[same])
        assert np.array_equal(np.isnan(neg), np.isnan(pos))
    t4 = oracle.decode_table(E4M3)
    assert 480.0 not in t4 and np.nanmax(t4) == 448.0
    assert np.isnan(t4[0x7F]) and np.isnan(t4[0xFF]) and np.isfinite(t4[:0x7F]).all()
    t5 = oracle.decode_table(E5M2)
    assert t5[0x7C] == np.inf and t5[0xFC] == -np.inf
    assert np.isnan(t5[[0x7D, 0x7E, 0x7F, 0xFD, 0xFE, 0xFF]]).all()


# ------------------------------------------------------------------ encode --

def _brute_force_encode(y32, fmt, overflow):
    """Nearest representable value by exhaustive search over the decode table,
    ties to the even code, then the overflow rule.  Shares no logic with the
    oracle's shift-and-round encoder: it only reads the (separately pinned)
    decode table and compares distances in float64, where they are exact."""
    t = oracle.decode_table(fmt)
    maxmag = 0x7E if fmt == E4M3 else 0x7B
    mags = t[: maxmag + 1].copy()
    # one virtual magnitude past the maximum: where the format would continue
    # (E4M3: 480 at mantissa 111; E5M2: 2^16 in the next binade)
    virtual = 480.0 if fmt == E4M3 else 65536.0
    ext = np.concatenate([mags, [virtual]])
    with np.errstate(invalid="ignore"):       # signalling NaN patterns among the inputs
        y = y32.astype(np.float64)
    a = np.abs(y)
    sign = (y32.view(np.uint32) >> 31).astype(np.uint8) << 7
    out = np.zeros(y.shape, dtype=np.uint8)
    CH = 1 << 16
    for lo in range(0, a.size, CH):
        aa = a[lo:lo + CH]
        with np.errstate(invalid="ignore"):
            d = np.abs(aa[:, None] - ext[None, :])
        best = np.argmin(d, axis=1)                    # lowest code among equals
        dmin = d[np.arange(aa.size), best]
        nxt = np.minimum(best + 1, ext.size - 1)
        tie = (d[np.arange(aa.size), nxt] == dmin) & (nxt != best)
        best = np.where(tie & (best % 2 == 1), nxt, best)
        over = (best > maxmag) | (aa > virtual)
        if overflow == SATURATE:
            code = np.where(over, maxmag, best)
        else:
            code = np.where(over, 0x7F if fmt == E4M3 else 0x7C, best)
        out[lo:lo + CH] = code.astype(np.uint8)
    isnan = np.isnan(y)
    isinf = np.isinf(y)
    out = np.where(isinf, 0x7F if fmt == E4M3 else 0x7C, out)
    out = np.where(isnan, 0x7F, out)
    return (out | sign).astype(np.uint8)


def _oracle_encode(y32, fmt, overflow):
    return oracle.quantize(np.ascontiguousarray(y32, dtype=np.float32), 1.0, fmt, overflow)


def _all_bf16_as_f32():
    return (np.arange(1 << 16, dtype=np.uint32) << 16).view(np.float32)


def _tie_neighbourhood(fmt):
    """every midpoint between neighbouring magnitudes (and past the maximum), +-2 fp32 ulps"""
    t = oracle.decode_table(fmt)
    maxmag = 0x7E if fmt == E4M3 else 0x7B
    mags = np.concatenate([t[: maxmag + 1], [480.0 if fmt == E4M3 else 65536.0]])
    mids = ((mags[:-1] + mags[1:]) / 2).astype(np.float32)
    pts = []
    for m in np.concatenate([mids, mags.astype(np.float32)]):
        b = np.array([m], dtype=np.float32).view(np.uint32)[0].astype(np.int64)
        for d in range(-2, 3):
            if b + d >= 0:
                pts.append(b + d)
    v = np.array(pts, dtype=np.uint32).view(np.float32)
    return np.concatenate([v, -v])


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
@pytest.mark.parametrize("overflow", [SATURATE, NOSAT])
def test_encode_equals_brute_force_nearest(fmt, overflow):
    rng = np.random.default_rng(20220912 + fmt)
    rand_bits = rng.integers(0, 1 << 32, size=1 << 20, dtype=np.uint64).astype(np.uint32).view(np.float32)
    # log-uniform magnitudes across the whole FP8 range incl. subnormals and overflow
    logu = np.exp2(rng.uniform(-20, 18, size=1 << 19)).astype(np.float32) * rng.choice([-1, 1], size=1 << 19).astype(np.float32)
    tiny = np.array([0.0, -0.0, 1e-45, -1e-45, 1e-40, 2.0 ** -126, np.inf, -np.inf, np.nan, 3.4e38, -3.4e38], dtype=np.float32)
    neg_nan = np.array([0xFFC00000, 0x7F800001, 0xFF800001], dtype=np.uint32).view(np.float32)
    y = np.concatenate([_all_bf16_as_f32(), _tie_neighbourhood(fmt), rand_bits, logu, tiny, neg_nan])
    got = _oracle_encode(y, fmt, overflow)
    want = _brute_force_encode(y, fmt, overflow)
    bad = np.nonzero(got != want)[0]
    assert bad.size == 0, [(float(y[i]), hex(got[i]), hex(want[i])) for i in bad[:8]]


def test_encode_named_ties_and_thresholds():
    # midpoints go to the code with an even last bit
    e4 = {2.0 ** -10: 0x00, 3 * 2.0 ** -10: 0x02, 15 * 2.0 ** -10: 0x08, 1.0625: 0x38, 1.1875: 0x3A}
    e5 = {2.0 ** -17: 0x00, 3 * 2.0 ** -17: 0x02, 7 * 2.0 ** -17: 0x04, 1.125: 0x3C, 1.375: 0x3E}
    for y, c in e4.items():
        assert oracle.encode(y, E4M3) == c and oracle.encode(-y, E4M3) == c | 0x80
    for y, c in e5.items():
        assert oracle.encode(y, E5M2) == c and oracle.encode(-y, E5M2) == c | 0x80
    # overflow (Section 2): saturate, or NaN / Inf in the non-saturating mode
    assert oracle.encode(1e6, E4M3, SATURATE) == 0x7E and oracle.encode(-1e6, E4M3, SATURATE) == 0xFE
    assert oracle.encode(1e6, E5M2, SATURATE) == 0x7B and oracle.encode(-1e6, E5M2, SATURATE) == 0xFB
    assert oracle.encode(464.0, E4M3, NOSAT) == 0x7E
    assert oracle.encode(np.nextafter(np.float32(464), np.float32(1e9)), E4M3, NOSAT) == 0x7F
    assert oracle.encode(np.nextafter(np.float32(61440), np.float32(0)), E5M2, NOSAT) == 0x7B
    assert oracle.encode(61440.0, E5M2, NOSAT) == 0x7C
    # special values convert to special values in both modes; E4M3 has no Inf (Section 2)
    for ovf in (SATURATE, NOSAT):
        assert oracle.encode(np.inf, E4M3, ovf) == 0x7F and oracle.encode(-np.inf, E4M3, ovf) == 0xFF
        assert oracle.encode(np.inf, E5M2, ovf) == 0x7C and oracle.encode(-np.inf, E5M2, ovf) == 0xFC
        assert oracle.encode(np.nan, E4M3, ovf) & 0x7F == 0x7F and oracle.encode(np.nan, E5M2, ovf) & 0x7F == 0x7F
    # signed zero, also for values that round to zero
    assert oracle.encode(-0.0, E4M3) == 0x80 and oracle.encode(-1e-30, E4M3) == 0x80 and oracle.encode(-1e-30, E5M2) == 0x80


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_encode_round_trip_every_code(fmt):
    t = oracle.decode_table(fmt).astype(np.float32)
    for ovf in (SATURATE, NOSAT):
        got = _oracle_encode(t, fmt, ovf)
        for c in range(256):
            if np.isnan(t[c]):
                assert got[c] == (c & 0x80) | 0x7F
            else:
                assert got[c] == c, (c, t[c], got[c])


@pytest.mark.parametrize("fmt,dt", [(E4M3, torch.float8_e4m3fn), (E5M2, torch.float8_e5m2)])
def test_encode_agrees_with_torch_cast_in_range(fmt, dt):
    rng = np.random.default_rng(7 + fmt)
    fmax = oracle.FMT_MAX[fmt]
    y = (np.exp2(rng.uniform(-20, np.log2(fmax), size=1 << 18)) * rng.choice([-1, 1], size=1 << 18)).astype(np.float32)
    y = np.concatenate([y, _tie_neighbourhood(fmt)])
    y = y[np.abs(y) <= fmax]
    lib = torch.from_numpy(y).to(dt).view(torch.uint8).numpy()
    assert np.array_equal(_oracle_encode(y, fmt, SATURATE), lib)


def test_e5m2_encode_is_rne_of_half_bits():
    # textbook: for a value that is exactly a float16, E5M2 is the float16 pattern rounded
    # (nearest even) to its top byte; the carry may run into the exponent, up to Inf.
    h = np.arange(1 << 16, dtype=np.uint16)
    hv = h.view(np.float16)
    keep = np.isfinite(hv)
    h, hv = h[keep], hv[keep]
    mag = (h & 0x7FFF).astype(np.uint32)
    low, top = mag & 0xFF, mag >> 8
    up = (low > 0x80) | ((low == 0x80) & (top & 1 == 1))
    want_mag = top + up
    want = (want_mag | ((h >> 15).astype(np.uint32) << 7)).astype(np.uint8)      # 0x7C when it carries to Inf
    got = _oracle_encode(hv.astype(np.float32), E5M2, NOSAT)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_encode_monotonic(fmt):
    rng = np.random.default_rng(3)
    y = np.sort((rng.standard_normal(1 << 18) * np.exp2(rng.uniform(-18, 17, size=1 << 18))).astype(np.float32))
    c = _oracle_encode(y, fmt, SATURATE).astype(np.int32)
    key = np.where(c & 0x80, -(c & 0x7F), c & 0x7F)       # sign-magnitude order
    assert np.all(np.diff(key) >= 0)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_power_of_two_scale_is_an_exponent_bias(fmt):
    # Section 3.2: a programmable exponent bias is the same as a power-of-two scale factor
    rng = np.random.default_rng(11)
    x = (rng.standard_normal(1 << 16) * np.exp2(rng.uniform(-12, 6, size=1 << 16))).astype(np.float32)
    for k in (-3, 1, 3):
        a = oracle.quantize(x, np.float32(2.0 ** k), fmt)
        b = oracle.quantize(np.ldexp(x, k).astype(np.float32), 1.0, fmt)
        assert np.array_equal(a, b)


# ------------------------------------------------- quantize / dequantize --

@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_quantize_is_fp32_multiply_then_encode(fmt):
    rng = np.random.default_rng(5)
    x = (rng.standard_normal(1 << 16) * np.exp2(rng.uniform(-30, 30, size=1 << 16))).astype(np.float32)
    scale = np.float32(37.123)
    y = x * scale                                  # numpy float32 multiply: IEEE, no flush to zero
    assert np.array_equal(oracle.quantize(x, scale, fmt), _brute_force_encode(y, fmt, SATURATE))
    # subnormal products are kept (no flush-to-zero before the conversion)
    xs = np.array([1e-30, -1e-30, 3e-38], dtype=np.float32)
    ys = xs * np.float32(1e-10)
    assert np.array_equal(oracle.quantize(xs, np.float32(1e-10), fmt), _brute_force_encode(ys, fmt, SATURATE))
    # a NaN element keeps its own sign, whatever the multiply would make of it
    nans = np.array([0x7FC00000, 0xFFC00000, 0xFF800001, 0x7FFFFFFF], dtype=np.uint32).view(np.float32)
    assert oracle.quantize(nans, scale, fmt).tolist() == [0x7F, 0xFF, 0xFF, 0x7F]
    assert oracle.quantize(nans, np.float32(-2.0), fmt).tolist() == [0x7F, 0xFF, 0xFF, 0x7F]
    # bf16 input widens exactly
    xb = torch.from_numpy(x).to(torch.bfloat16)
    bits = xb.view(torch.int16).numpy().view(np.uint16)
    yb = xb.to(torch.float32).numpy() * scale
    assert np.array_equal(oracle.quantize(bits, scale, fmt), _brute_force_encode(yb, fmt, SATURATE))


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_dequantize_is_table_lookup_times_inverse_scale(fmt):
    codes = np.arange(256, dtype=np.uint8)
    t = oracle.decode_table(fmt).astype(np.float32)
    si = np.float32(0.0123)
    with np.errstate(invalid="ignore"):
        want = t * si
    got = oracle.dequantize(codes, si, fmt, "f32")
    assert np.array_equal(np.isnan(got), np.isnan(want))
    assert np.array_equal(got[~np.isnan(want)], want[~np.isnan(want)])
    assert np.array_equal(np.signbit(got[~np.isnan(want)]), np.signbit(want[~np.isnan(want)]))
    # bf16 output: torch's float32 -> bfloat16 cast is round-to-nearest-even
    gotb = oracle.dequantize(codes, si, fmt, "bf16")
    wantb = torch.from_numpy(want).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    ok = ~np.isnan(want)
    assert np.array_equal(gotb[ok], wantb[ok])
    assert np.all((gotb[~ok] & 0x7FFF) > 0x7F80)


@pytest.mark.parametrize("fmt,mbits", [(E4M3, 3), (E5M2, 2)])
def test_round_trip_error_bound(fmt, mbits):
    # a normal-range value comes back within half a unit in the last mantissa place
    rng = np.random.default_rng(9)
    amax = 3.0
    x = rng.uniform(-amax, amax, size=1 << 16).astype(np.float32)
    scale, scale_inv = oracle.scale_from_amax(np.float32(np.abs(x).max()), fmt)
    xh = oracle.dequantize(oracle.quantize(x, scale, fmt), scale_inv, fmt, "f32")
    min_normal = (2.0 ** -6 if fmt == E4M3 else 2.0 ** -14) / float(scale)
    big = np.abs(x) >= min_normal
    rel = np.abs(xh[big].astype(np.float64) - x[big]) / np.abs(x[big])
    assert rel.max() <= 2.0 ** -(mbits + 1) * (1 + 1e-5)
    small = ~big
    quantum = (2.0 ** -9 if fmt == E4M3 else 2.0 ** -16) / float(scale)
    assert np.all(np.abs(xh[small].astype(np.float64) - x[small]) <= quantum / 2 * (1 + 1e-5))


def test_double_rounding_diagnostic():
    # two roundings (binary32 product, then FP8) against one rounding of the exact product: they can only
    # differ when the binary32 rounding lands on an FP8 tie, which is rare but real
    rng = np.random.default_rng(33)
    x = rng.standard_normal(1 << 20).astype(np.float32)
    for fmt in (E4M3, E5M2):
        n = oracle.count_double_rounding(x, np.float32(37.123), fmt)
        assert 0 <= n < x.size // 10000
        assert oracle.count_double_rounding(x, np.float32(2.0), fmt) == 0        # a power-of-two scale multiplies exactly
    # a constructed case: x*scale exactly just above the E4M3 tie 1.0625, its binary32 rounding exactly on the tie
    xs = np.array([np.float32(1.0625) + np.float32(2.0 ** -23)], dtype=np.float32)   # 1.0625 + 1 ulp
    sc = np.float32(1.0 - 2.0 ** -24)                                                 # product = 1.0625 + ~2^-23 - 2^-24*1.0625...
    exact = float(xs[0]) * float(sc)
    assert exact > 1.0625 and np.float32(exact) == np.float32(1.0625)
    assert oracle.count_double_rounding(xs, sc, E4M3) == 1                            # exact -> 0x39, twice rounded -> tie -> 0x38
    assert oracle.quantize(xs, sc, E4M3)[0] == 0x38


# ------------------------------------------------------------ amax / scale --

def test_amax_closed_form_and_nan():
    rng = np.random.default_rng(1)
    x = rng.standard_normal(100003).astype(np.float32) * 17
    assert oracle.amax(x) == np.abs(x).max()
    assert oracle.amax(x, threads=4) == np.abs(x).max()
    assert oracle.amax(rng.permutation(x)) == np.abs(x).max()
    assert oracle.amax(np.zeros(0, dtype=np.float32)) == 0 and oracle.amax_bits(np.zeros(0, dtype=np.float32)) == 0
    # equals the integer maximum of the magnitude bit patterns (sign-magnitude ordering, Section 3.1)
    assert oracle.amax_bits(x) == int((x.view(np.uint32) & 0x7FFFFFFF).max())
    x[777] = np.nan
    assert oracle.amax_bits(x) == 0x7FC00000
    x[777] = -np.inf
    assert oracle.amax(x) == np.inf
    xb = torch.from_numpy(rng.standard_normal(4097).astype(np.float32)).to(torch.bfloat16)
    bits = xb.view(torch.int16).numpy().view(np.uint16)
    assert oracle.amax(bits) == xb.to(torch.float32).abs().max().item()


@pytest.mark.parametrize("fmt,maxcode", [(E4M3, 0x7E), (E5M2, 0x7B)])
def test_scale_from_amax(fmt, maxcode):
    fmax = np.float32(oracle.FMT_MAX[fmt])
    rng = np.random.default_rng(2)
    for a in np.concatenate([np.exp2(rng.uniform(-100, 100, size=2000)), [1.0, 448.0, 57344.0, 3.7]]).astype(np.float32):
        s, si = oracle.scale_from_amax(a, fmt)
        assert s == fmax / a                    # numpy float32 division
        assert si == np.float32(1.0) / s
        # the scaled maximum lands exactly on the format's largest code
        assert oracle.encode(a * s, fmt, NOSAT) == maxcode
    for a in (0.0, np.nan, np.inf):
        s, si = oracle.scale_from_amax(np.float32(a), fmt)
        assert s == 1.0 and si == 1.0
    s, si = oracle.scale_from_amax(np.float32(1e-44), fmt)     # quotient overflows -> largest finite
    assert s == np.finfo(np.float32).max and np.isfinite(si)


@pytest.mark.parametrize("fmt,maxcode", [(E4M3, 0x7E), (E5M2, 0x7B)])
def test_power_of_two_scale_from_amax(fmt, maxcode):
    fmax = oracle.FMT_MAX[fmt]
    rng = np.random.default_rng(21)
    for a in np.concatenate([np.exp2(rng.uniform(-100, 100, size=1000)), [1.0, 448.0, 57344.0, 3.7, 7.0, 0.875]]).astype(np.float32):
        s, si = oracle.scale_pow2_from_amax(a, fmt)
        s0 = np.float32(fmax) / a
        m, e = np.frexp(np.float64(s))
        assert m == 0.5                                   # a power of two
        assert s <= s0 < 2 * np.float64(s)                # the largest one not above fmax / amax
        assert np.float64(s) * np.float64(si) == 1.0      # the inverse is exact
        # the scaled maximum lands in the top binade of the format and never overflows
        code = oracle.encode(a * s, fmt, NOSAT)
        assert code <= maxcode and oracle.decode(code, fmt) > fmax / 2 * (1 - 2.0 ** -3)
    for a in (0.0, np.nan, np.inf):
        assert oracle.scale_pow2_from_amax(np.float32(a), fmt) == (1.0, 1.0)


@pytest.mark.parametrize("fmt", [E4M3, E5M2])
def test_fake_quantize_values_are_representable_and_fixed_points(fmt):
    # simulated FP8 (Section 4): the result is the nearest representable value times 1/scale,
    # and applying it twice changes nothing when the scale is a power of two
    rng = np.random.default_rng(22)
    x = (rng.standard_normal(1 << 14) * 3).astype(np.float32)
    s, si = oracle.scale_pow2_from_amax(np.abs(x).max(), fmt)
    y = oracle.fake_quantize(x, s, si, fmt)
    t = oracle.decode_table(fmt)
    finite = t[np.isfinite(t)]
    assert np.isin(y.astype(np.float64) * float(s), finite).all()
    assert np.array_equal(oracle.fake_quantize(y, s, si, fmt), y)
    near = finite[np.abs(finite[None, :] - (x.astype(np.float64) * float(s))[:, None]).argmin(axis=1)]
    assert np.all(np.abs(y.astype(np.float64) * float(s) - x.astype(np.float64) * float(s)) <= np.abs(near - x.astype(np.float64) * float(s)) + 1e-300)


# ------------------------------------------------------------ bf16 rounding --

def test_f64_to_bf16_single_rounding():
    rng = np.random.default_rng(4)
    # exact rational check on random doubles, including bf16 subnormals and overflow
    vals = np.concatenate([rng.standard_normal(300) * np.exp2(rng.uniform(-140, 130, size=300)),
                           [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 3.4e38, 1e-41, 4.6e-41]])
    for v in vals:
        got = oracle.f64_to_bf16(v)
        gv = float(np.array([got << 16], dtype=np.uint32).view(np.float32)[0])
        if np.isinf(gv):
            # only at or above the halfway point to 2^128
            assert abs(v) >= (2.0 ** 128) * (1 - 2.0 ** -9)
            continue
        # neighbours of the returned bf16: the returned one must be nearest (ties: even mantissa)
        mag = got & 0x7FFF
        cands = [m for m in (mag - 1, mag, mag + 1) if 0 <= m <= 0x7F80]
        fv = Fraction(abs(v))
        def val(m):
            f = np.array([m << 16], dtype=np.uint32).view(np.float32)[0]
            return Fraction(2) ** 128 if np.isinf(f) else Fraction(float(f))
        dist = {m: abs(val(m) - fv) for m in cands}
        best = min(dist.values())
        winners = [m for m in cands if dist[m] == best]
        assert mag in winners
        if len(winners) == 2:
            assert mag % 2 == 0
        assert (got >> 15) == int(np.signbit(v))
    # values that are exactly float32: same answer as the float32 -> bf16 routine and as torch
    f = (rng.standard_normal(5000) * np.exp2(rng.uniform(-20, 20, size=5000))).astype(np.float32)
    a = oracle.round_bf16_from_f64(f.astype(np.float64))
    b = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(a, b)
    assert all(oracle.f32_to_bf16(v) == int(w) for v, w in zip(f[:500], b[:500]))
    # a case where rounding through float32 first would give a different (wrong) answer
    v = 1.0 + 2.0 ** -8 + 2.0 ** -40          # just above the bf16 midpoint between 1 and 1+2^-7
    assert oracle.f64_to_bf16(v) == 0x3F81
