/*
 * CPU oracle for the FP8 hot path of "FP8 Formats for Deep Learning"
 * (arXiv 2209.05433).  TEST INFRASTRUCTURE ONLY: nothing on the product path
 * may call this file; it exists so that the CUDA library has something slow
 * and obviously right to be compared with.  It shares no code, table or
 * constant generator with the CUDA sources.
 *
 * Plain C, scalar, one element at a time, no intrinsics, no threads.  Built
 * with -O2 -ffp-contract=off so that no multiply-add is fused.
 *
 * What each function follows:
 *   fp8o_decode            Table 1 and Section 3 (S.E.M fields, bias 7 / 15,
 *                          subnormals, E4M3 keeps exponent 1111 for normals
 *                          256..448 and has one NaN mantissa, E5M2 is IEEE-like).
 *   fp8o_encode            Section 2: conversion from a wider type; special
 *                          values go to special values (E4M3: Inf and NaN both
 *                          become NaN); overflow saturates to the maximum
 *                          finite value, or, in the non-saturating mode the
 *                          section allows, becomes NaN (E4M3) / Inf (E5M2).
 *                          The rounding mode is left open by the paper; round
 *                          to nearest, ties to even, is used.
 *   fp8o_quantize_*        Section 2: multiply by the per-tensor scale factor
 *                          (one single-precision multiply), then convert.
 *   fp8o_dequantize_*      Section 2: convert back and multiply by the inverse
 *                          of the scale factor.
 *   fp8o_amax_*            Section 2: the tensor's maximum magnitude, the input
 *                          of the scale choice.  NaN propagates.
 *   fp8o_scale_from_amax   Section 2: the scale that moves the maximum
 *                          magnitude onto the format's maximum (Table 1).
 *   fp8o_gemm_*            Sections 2 and 4.1: dot products of FP8 inputs with
 *                          a higher precision result, unscaled once per dot
 *                          product.  Accumulated in double.
 *
 * Readings taken where the paper is silent (each is a convention, "parity
 * unpinned" by the paper itself beyond the cited sentences):
 *   - scale multiply and conversion are two roundings (fp32 product, then FP8);
 *   - the special-value rule is applied to the scaled fp32 value, in both
 *     overflow modes (a scaled value of +-Inf is never saturated);
 *   - the NaN emitted is sign | 0x7F in both formats, the sign being that of the
 *     input element (the sign of a NaN product is not defined by IEEE 754);
 *   - the sign of zero, and of anything that rounds to zero, is kept.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

enum { FP8O_E4M3 = 0, FP8O_E5M2 = 1 };
enum { FP8O_SATURATE = 0, FP8O_NOSAT = 1 };

static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* bfloat16 is the upper half of a binary32 pattern: widening is exact. */
static float bf16_to_f32(uint16_t h) { return bits_f32((uint32_t)h << 16); }

/* binary32 -> bfloat16, round to nearest even; NaN stays NaN (quiet, sign kept). */
uint16_t fp8o_f32_to_bf16(float f)
{
    uint32_t u = f32_bits(f);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u)
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* double -> bfloat16 with ONE rounding (nearest even), not via binary32.
 * bf16 has 8 significand bits, minimum normal exponent -126, subnormal
 * quantum 2^-133, and overflows to Inf from 2^128 * (1 - 2^-9) upward. */
uint16_t fp8o_f64_to_bf16(double v)
{
    uint16_t sign = signbit(v) ? 0x8000u : 0u;
    if (isnan(v)) return (uint16_t)(sign | 0x7FC0u);
    double a = fabs(v);
    if (isinf(a)) return (uint16_t)(sign | 0x7F80u);
    if (a == 0.0) return sign;
    int e;
    (void)frexp(a, &e);          /* a = m * 2^e, m in [0.5,1) */
    int q = e - 1;               /* floor(log2 a) */
    if (q < -126) q = -126;
    /* quantum 2^(q-7); a / quantum is exact in double (power-of-two scaling) */
    double t = ldexp(a, -(q - 7));
    double k = floor(t);
    double rem = t - k;          /* exact: t has at most 53 bits */
    if (rem > 0.5 || (rem == 0.5 && fmod(k, 2.0) == 1.0)) k += 1.0;
    /* k in [0, 256]; k == 256 carries into the next exponent */
    uint32_t ki = (uint32_t)k;
    uint32_t mag;
    if (q == -126 && ki < 128u) mag = ki;                       /* subnormal (or zero) */
    else mag = ((uint32_t)(q + 127) << 7) + (ki - 128u);         /* carry propagates */
    if (mag >= 0x7F80u) mag = 0x7F80u;                           /* overflow -> Inf */
    return (uint16_t)(sign | mag);
}

void fp8o_f64_to_bf16_array(const double* v, size_t n, uint16_t* out)
{
    for (size_t i = 0; i < n; ++i) out[i] = fp8o_f64_to_bf16(v[i]);
}

/* ---------------------------------------------------------------- decode -- */

/* Table 1 / Section 3.  Returns the exact real value as a double; NaN and
 * (E5M2 only) infinities as the IEEE specials. */
double fp8o_decode(uint8_t c, int fmt)
{
    int s = c >> 7;
    int e, m, mbits, bias, emax_field;
    if (fmt == FP8O_E4M3) { e = (c >> 3) & 15; m = c & 7; mbits = 3; bias = 7;  emax_field = 15; }
    else                  { e = (c >> 2) & 31; m = c & 3; mbits = 2; bias = 15; emax_field = 31; }
    double sign = s ? -1.0 : 1.0;
    if (fmt == FP8O_E4M3) {
        if (e == emax_field && m == 7) return s ? -NAN : NAN;    /* S.1111.111 only */
    } else {
        if (e == emax_field) {
            if (m == 0) return sign * INFINITY;                  /* S.11111.00 */
            return s ? -NAN : NAN;                               /* S.11111.{01,10,11} */
        }
    }
    if (e == 0)                                                  /* zero and subnormals */
        return sign * ldexp((double)m, 1 - bias - mbits);
    return sign * ldexp(1.0 + (double)m / (double)(1 << mbits), e - bias);
}

void fp8o_decode_table(int fmt, double* table256)
{
    for (int c = 0; c < 256; ++c) table256[c] = fp8o_decode((uint8_t)c, fmt);
}

/* ---------------------------------------------------------------- encode -- */

/* Section 2 conversion of one binary32 value y (already scaled). */
uint8_t fp8o_encode(float y, int fmt, int overflow)
{
    const int emin  = (fmt == FP8O_E4M3) ? -6 : -14;   /* exponent of min normal (Table 1) */
    const int mbits = (fmt == FP8O_E4M3) ? 3 : 2;
    const int bias  = (fmt == FP8O_E4M3) ? 7 : 15;
    const uint32_t maxmag = (fmt == FP8O_E4M3) ? 0x7Eu : 0x7Bu;  /* max normal (Table 1) */
    const uint32_t nanmag = 0x7Fu;
    const uint32_t infmag = 0x7Cu;                               /* E5M2 only */

    uint32_t u = f32_bits(y);
    uint32_t s = u >> 31;
    uint32_t a = u & 0x7FFFFFFFu;

    if (a > 0x7F800000u) return (uint8_t)((s << 7) | nanmag);                 /* NaN -> NaN */
    if (a == 0x7F800000u)                                                      /* Inf */
        return (uint8_t)((s << 7) | (fmt == FP8O_E4M3 ? nanmag : infmag));
    if (a == 0) return (uint8_t)(s << 7);                                      /* signed zero */

    /* |y| = sig * 2^(ex-23) with sig < 2^24 */
    uint64_t sig;
    int ex;
    if ((a >> 23) == 0) { sig = a; ex = -126; }                                /* fp32 subnormal */
    else { sig = (a & 0x7FFFFFu) | 0x800000u; ex = (int)(a >> 23) - 127; }

    int q = ex;                       /* floor(log2 |y|) for normals; subnormals are far below emin */
    if (q < emin) q = emin;
    int shift = (q - mbits) - (ex - 23);     /* |y| / 2^(q-mbits) = sig / 2^shift; shift >= 20 */

    uint64_t k;
    if (shift >= 25) {
        k = 0;                               /* sig < 2^24 <= half quantum, strictly below the tie */
    } else {
        uint64_t half = (uint64_t)1 << (shift - 1);
        uint64_t rem  = sig & (((uint64_t)1 << shift) - 1);
        k = sig >> shift;
        if (rem > half || (rem == half && (k & 1u))) k += 1;   /* nearest, ties to even */
    }

    uint64_t mag;
    if (q == emin) mag = k;                                      /* subnormal range; k == 2^mbits is min normal */
    else mag = ((uint64_t)(q + bias) << mbits) + (k - ((uint64_t)1 << mbits));  /* carry moves the exponent */

    if (mag > maxmag) {
        if (overflow == FP8O_SATURATE) mag = maxmag;
        else mag = (fmt == FP8O_E4M3) ? nanmag : infmag;
    }
    return (uint8_t)((s << 7) | (uint32_t)mag);
}

/* Diagnostic for the reading "two roundings" of the scale multiply: the code a
 * SINGLE rounding of the exact product x*scale would give.  The product of two
 * binary32 values is exact in double, so this is the conversion of that double:
 * same steps as fp8o_encode on a 53-bit significand. */
uint8_t fp8o_encode_exact_product(float x, float scale, int fmt, int overflow)
{
    const int emin  = (fmt == FP8O_E4M3) ? -6 : -14;
    const int mbits = (fmt == FP8O_E4M3) ? 3 : 2;
    const int bias  = (fmt == FP8O_E4M3) ? 7 : 15;
    const uint32_t maxmag = (fmt == FP8O_E4M3) ? 0x7Eu : 0x7Bu;
    double y = (double)x * (double)scale;
    uint32_t s = signbit(y) ? 1u : 0u;
    if (isnan(y)) return (uint8_t)(((signbit(x) ? 1u : 0u) << 7) | 0x7Fu);
    double a = fabs(y);
    if (isinf(a) || a >= ldexp(1.0, 128) * (1.0 - ldexp(1.0, -25)))       /* rounds to binary32 infinity */
        return (uint8_t)((s << 7) | (fmt == FP8O_E4M3 ? 0x7Fu : 0x7Cu));
    if (a == 0.0) return (uint8_t)(s << 7);
    int e;
    (void)frexp(a, &e);
    int q = e - 1;
    if (q < emin) q = emin;
    double t = ldexp(a, -(q - mbits));                 /* |y| in units of the rounding quantum, exact */
    double k = floor(t), rem = t - k;
    if (rem > 0.5 || (rem == 0.5 && fmod(k, 2.0) == 1.0)) k += 1.0;
    uint64_t ki = (uint64_t)k, mag;
    if (q == emin) mag = ki;
    else mag = ((uint64_t)(q + bias) << mbits) + (ki - ((uint64_t)1 << mbits));
    if (mag > maxmag) mag = (overflow == FP8O_SATURATE) ? maxmag : (fmt == FP8O_E4M3 ? 0x7Fu : 0x7Cu);
    return (uint8_t)((s << 7) | (uint32_t)mag);
}

/* how many elements would get a different code under the single-rounding reading */
size_t fp8o_count_double_rounding_f32(const float* x, size_t n, float scale, int fmt, int overflow)
{
    size_t c = 0;
    for (size_t i = 0; i < n; ++i)
        c += fp8o_encode_exact_product(x[i], scale, fmt, overflow) != fp8o_encode((float)((double)x[i] * (double)scale), fmt, overflow)
             && !isnan(x[i]);
    return c;
}

/* ------------------------------------------------------ quantize / dequantize */

/* one IEEE binary32 multiply: the double product of two floats is exact
 * (48 significant bits), so the cast performs the single rounding. */
static float mul_f32(float a, float b) { return (float)((double)a * (double)b); }

/* One element: scale, then convert.  IEEE 754 leaves the sign of a NaN result of
 * a multiplication unspecified (processors differ), so the NaN code takes the
 * sign of the input element x: "the sign of the input is kept". */
static uint8_t quantize_one(float x, float scale, int fmt, int overflow)
{
    float y = mul_f32(x, scale);
    if (isnan(y)) return (uint8_t)((signbit(x) ? 0x80u : 0u) | 0x7Fu);
    return fp8o_encode(y, fmt, overflow);
}

void fp8o_quantize_f32(const float* x, size_t n, float scale, int fmt, int overflow, uint8_t* out)
{
    for (size_t i = 0; i < n; ++i) out[i] = quantize_one(x[i], scale, fmt, overflow);
}

void fp8o_quantize_bf16(const uint16_t* x, size_t n, float scale, int fmt, int overflow, uint8_t* out)
{
    for (size_t i = 0; i < n; ++i) out[i] = quantize_one(bf16_to_f32(x[i]), scale, fmt, overflow);
}

void fp8o_dequantize_f32(const uint8_t* c, size_t n, int fmt, float scale_inv, float* out)
{
    for (size_t i = 0; i < n; ++i) {
        float v = (float)fp8o_decode(c[i], fmt);          /* exact: every FP8 value is a binary32 value */
        out[i] = mul_f32(v, scale_inv);
    }
}

void fp8o_dequantize_bf16(const uint8_t* c, size_t n, int fmt, float scale_inv, uint16_t* out)
{
    for (size_t i = 0; i < n; ++i) {
        float v = (float)fp8o_decode(c[i], fmt);
        out[i] = fp8o_f32_to_bf16(mul_f32(v, scale_inv));
    }
}

/* --------------------------------------------------------------------- amax */

/* Returns the binary32 bit pattern of max |x_i|; 0x7FC00000 if any NaN; +0 when empty. */
uint32_t fp8o_amax_f32(const float* x, size_t n)
{
    int saw_nan = 0;
    float best = 0.0f;
    for (size_t i = 0; i < n; ++i) {
        float v = x[i];
        if (isnan(v)) { saw_nan = 1; continue; }
        float a = fabsf(v);
        if (a > best) best = a;
    }
    return saw_nan ? 0x7FC00000u : f32_bits(best);
}

uint32_t fp8o_amax_bf16(const uint16_t* x, size_t n)
{
    int saw_nan = 0;
    float best = 0.0f;
    for (size_t i = 0; i < n; ++i) {
        float v = bf16_to_f32(x[i]);
        if (isnan(v)) { saw_nan = 1; continue; }
        float a = fabsf(v);
        if (a > best) best = a;
    }
    return saw_nan ? 0x7FC00000u : f32_bits(best);
}

/* Section 2: scale so that the maximum magnitude lands on the format maximum.
 * amax of 0, NaN or Inf gives scale 1; a quotient that overflows is clamped
 * to the largest finite binary32. */
void fp8o_scale_from_amax(float amax, int fmt, float* scale, float* scale_inv)
{
    const float fmax = (fmt == FP8O_E4M3) ? 448.0f : 57344.0f;
    float s;
    if (isnan(amax) || isinf(amax) || amax == 0.0f) s = 1.0f;
    else {
        double qd = (double)fmax / (double)amax;
        /* division of two floats rounded once to float == IEEE binary32 division:
         * double has more than 2*24+2 bits, so no double rounding can occur. */
        s = (float)qd;
        if (isinf(s)) s = 3.40282346638528859812e+38f;
    }
    *scale = s;
    *scale_inv = (float)(1.0 / (double)s);
}

/* Section 3.2: a programmable exponent bias is the same as a power-of-two scale
 * factor.  The scale is the largest power of two not above fmax / amax (the
 * quotient with the guards of fp8o_scale_from_amax); its inverse is exact. */
void fp8o_scale_pow2_from_amax(float amax, int fmt, float* scale, float* scale_inv)
{
    float s0, unused;
    fp8o_scale_from_amax(amax, fmt, &s0, &unused);
    int e;
    (void)frexp((double)s0, &e);                 /* s0 = m * 2^e, m in [0.5, 1)  ->  2^(e-1) <= s0 < 2^e */
    float s = (float)ldexp(1.0, e - 1);          /* exact, also for subnormal s0 */
    *scale = s;
    *scale_inv = (float)(1.0 / (double)s);
}

/* ------------------------------------------------------ per-channel scales */

/* Section 4.2: "per-channel scaling factors for weights, per-tensor scaling
 * factors for activations".  x is rows x cols, row-major with pitch ld (in
 * elements).  axis 0: one channel per column (the maximum runs over rows);
 * axis 1: one channel per row.  Same definition as the per-tensor amax. */
void fp8o_amax_channels_f32(const float* x, int64_t rows, int64_t cols, int64_t ld, int axis, uint32_t* amax_bits)
{
    int64_t channels = axis == 0 ? cols : rows, len = axis == 0 ? rows : cols;
    for (int64_t c = 0; c < channels; ++c) {
        int saw_nan = 0;
        float best = 0.0f;
        for (int64_t i = 0; i < len; ++i) {
            float v = axis == 0 ? x[i * ld + c] : x[c * ld + i];
            if (isnan(v)) { saw_nan = 1; continue; }
            float a = fabsf(v);
            if (a > best) best = a;
        }
        amax_bits[c] = saw_nan ? 0x7FC00000u : f32_bits(best);
    }
}

void fp8o_amax_channels_bf16(const uint16_t* x, int64_t rows, int64_t cols, int64_t ld, int axis, uint32_t* amax_bits)
{
    int64_t channels = axis == 0 ? cols : rows, len = axis == 0 ? rows : cols;
    for (int64_t c = 0; c < channels; ++c) {
        int saw_nan = 0;
        float best = 0.0f;
        for (int64_t i = 0; i < len; ++i) {
            float v = bf16_to_f32(axis == 0 ? x[i * ld + c] : x[c * ld + i]);
            if (isnan(v)) { saw_nan = 1; continue; }
            float a = fabsf(v);
            if (a > best) best = a;
        }
        amax_bits[c] = saw_nan ? 0x7FC00000u : f32_bits(best);
    }
}

/* out[r*ld_out + c] = encode( x[r*ld + c] * scale[channel of (r,c)] ) */
void fp8o_quantize_channels_f32(const float* x, int64_t rows, int64_t cols, int64_t ld, int axis, const float* scale,
                                int fmt, int overflow, uint8_t* out, int64_t ld_out)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c)
            out[r * ld_out + c] = quantize_one(x[r * ld + c], scale[axis == 0 ? c : r], fmt, overflow);
}

void fp8o_quantize_channels_bf16(const uint16_t* x, int64_t rows, int64_t cols, int64_t ld, int axis, const float* scale,
                                 int fmt, int overflow, uint8_t* out, int64_t ld_out)
{
    for (int64_t r = 0; r < rows; ++r)
        for (int64_t c = 0; c < cols; ++c)
            out[r * ld_out + c] = quantize_one(bf16_to_f32(x[r * ld + c]), scale[axis == 0 ? c : r], fmt, overflow);
}

/* --------------------------------------------------------------------- GEMM */

/* One output element of D = (A.B) * sa_inv * sb_inv.
 * A(i,k) is at A[i*a_si + k*a_sk], B(k,j) at B[k*b_sk + j*b_sj] (strides in
 * elements), so both operand layouts of every pass (forward, dgrad, wgrad)
 * are expressible.  ref = sum_k dec(A_ik) dec(B_kj) * sa_inv * sb_inv,
 * sabs = sum_k |dec(A_ik) dec(B_kj)| * sa_inv * sb_inv, both in double, k ascending. */
void fp8o_gemm_element(const uint8_t* A, int fmt_a, int64_t a_si, int64_t a_sk,
                       const uint8_t* B, int fmt_b, int64_t b_sk, int64_t b_sj,
                       int64_t K, int64_t i, int64_t j,
                       float sa_inv, float sb_inv, double* ref, double* sabs)
{
    double acc = 0.0, accabs = 0.0;
    for (int64_t k = 0; k < K; ++k) {
        double a = fp8o_decode(A[i * a_si + k * a_sk], fmt_a);
        double b = fp8o_decode(B[k * b_sk + j * b_sj], fmt_b);
        double p = a * b;
        acc += p;
        accabs += fabs(p);
    }
    double alpha = (double)sa_inv * (double)sb_inv;
    *ref = acc * alpha;
    *sabs = accabs * alpha;
}

/* Rows [i0, i1) of D, all N columns: ref and sabs are (i1-i0) x N row-major. */
void fp8o_gemm_rows(const uint8_t* A, int fmt_a, int64_t a_si, int64_t a_sk,
                    const uint8_t* B, int fmt_b, int64_t b_sk, int64_t b_sj,
                    int64_t N, int64_t K, int64_t i0, int64_t i1,
                    float sa_inv, float sb_inv, double* ref, double* sabs)
{
    for (int64_t i = i0; i < i1; ++i)
        for (int64_t j = 0; j < N; ++j)
            fp8o_gemm_element(A, fmt_a, a_si, a_sk, B, fmt_b, b_sk, b_sj, K, i, j,
                              sa_inv, sb_inv, &ref[(i - i0) * N + j], &sabs[(i - i0) * N + j]);
}

/* Per-channel weight scales: column j of B (one output channel) carries its own
 * inverse scale sb_inv_vec[j]; A keeps one per-tensor inverse scale. */
void fp8o_gemm_rows_colscale(const uint8_t* A, int fmt_a, int64_t a_si, int64_t a_sk,
                             const uint8_t* B, int fmt_b, int64_t b_sk, int64_t b_sj,
                             int64_t N, int64_t K, int64_t i0, int64_t i1,
                             float sa_inv, const float* sb_inv_vec, double* ref, double* sabs)
{
    for (int64_t i = i0; i < i1; ++i)
        for (int64_t j = 0; j < N; ++j)
            fp8o_gemm_element(A, fmt_a, a_si, a_sk, B, fmt_b, b_sk, b_sj, K, i, j,
                              sa_inv, sb_inv_vec[j], &ref[(i - i0) * N + j], &sabs[(i - i0) * N + j]);
}

/* A list of (i,j) samples. */
void fp8o_gemm_samples(const uint8_t* A, int fmt_a, int64_t a_si, int64_t a_sk,
                       const uint8_t* B, int fmt_b, int64_t b_sk, int64_t b_sj,
                       int64_t K, const int64_t* ii, const int64_t* jj, int64_t count,
                       float sa_inv, float sb_inv, double* ref, double* sabs)
{
    for (int64_t s = 0; s < count; ++s)
        fp8o_gemm_element(A, fmt_a, a_si, a_sk, B, fmt_b, b_sk, b_sj, K, ii[s], jj[s],
                          sa_inv, sb_inv, &ref[s], &sabs[s]);
}

/* Exact dot product of decoded codes in fixed point: every finite E4M3 value
 * is a multiple of 2^-9 and every finite E5M2 value a multiple of 2^-16, so
 * each product is an integer number of 2^-(fa+fb) units and the sum fits in
 * 128 bits.  Returns 0 and writes the sum split as hi*2^64+lo (two's
 * complement) plus the unit exponent; returns 1 if a code is NaN or Inf. */
int fp8o_dot_exact(const uint8_t* A, int fmt_a, int64_t a_sk,
                   const uint8_t* B, int fmt_b, int64_t b_sk, int64_t K,
                   int64_t* hi, uint64_t* lo, int* unit_exp)
{
    const int fa = (fmt_a == FP8O_E4M3) ? 9 : 16;
    const int fb = (fmt_b == FP8O_E4M3) ? 9 : 16;
    __int128 acc = 0;
    for (int64_t k = 0; k < K; ++k) {
        double a = fp8o_decode(A[k * a_sk], fmt_a);
        double b = fp8o_decode(B[k * b_sk], fmt_b);
        if (isnan(a) || isnan(b) || isinf(a) || isinf(b)) return 1;
        int64_t ia = (int64_t)ldexp(a, fa);      /* exact integers */
        int64_t ib = (int64_t)ldexp(b, fb);
        acc += (__int128)ia * (__int128)ib;
    }
    *hi = (int64_t)(acc >> 64);
    *lo = (uint64_t)acc;
    *unit_exp = -(fa + fb);
    return 0;
}
