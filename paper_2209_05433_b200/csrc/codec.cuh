// Device-side FP8 codec (Table 1 encodings; Section 2 conversion rules).
//
// Two paths produce identical codes:
//   - the packed hardware converts (cvt.rn.satfinite.{e4m3x2,e5m2x2}.f32), used
//     for every vector whose scaled values are all finite (and, in the
//     non-saturating mode, all in range);
//   - encode_scalar(), an arithmetic encoder used for vectors that contain a
//     special value or (non-saturating mode) an overflow, for ragged tails and
//     for the unaligned element-wise kernels.  It rounds with the float adder
//     (subnormal targets) or with an integer add on the binary32 pattern
//     (normal targets), so a mantissa carry moves the exponent by itself.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace fp8b200 {

constexpr int kE4M3 = 0;
constexpr int kE5M2 = 1;

template <int FMT> struct Fmt;
template <> struct Fmt<kE4M3> {
    static constexpr int mbits = 3, bias = 7;
    static constexpr uint32_t max_mag = 0x7E;       // S.1111.110 = 448
    static constexpr uint32_t overflow_mag = 0x7F;  // no infinity: NaN
    static constexpr uint32_t inf_in_mag = 0x7F;    // wide Inf -> NaN
    static constexpr float nosat_limit = 464.0f;    // |y| >  464 rounds past 448
    static constexpr bool nosat_limit_inclusive = false;
};
template <> struct Fmt<kE5M2> {
    static constexpr int mbits = 2, bias = 15;
    static constexpr uint32_t max_mag = 0x7B;       // S.11110.11 = 57344
    static constexpr uint32_t overflow_mag = 0x7C;  // infinity
    static constexpr uint32_t inf_in_mag = 0x7C;    // wide Inf -> Inf
    static constexpr float nosat_limit = 61440.0f;  // |y| >= 61440 rounds to 2^16
    static constexpr bool nosat_limit_inclusive = true;
};

// One binary32 value (already multiplied by the scale) -> FP8 code, RNE.
template <int FMT, bool NOSAT>
__device__ __forceinline__ uint32_t encode_scalar(float y) {
    using F = Fmt<FMT>;
    const uint32_t u = __float_as_uint(y);
    const uint32_t sign = (u >> 24) & 0x80u;
    const uint32_t a = u & 0x7FFFFFFFu;
    if (a >= 0x7F800000u)                                   // special -> special
        return sign | (a > 0x7F800000u ? 0x7Fu : F::inf_in_mag);
    constexpr int emin = 1 - F::bias;                       // exponent of the minimum normal
    uint32_t mag;
    if (a < (uint32_t)(emin + 127) << 23) {
        // target is subnormal (or zero): adding 2^(emin-mbits+23) makes the float adder
        // round |y| to a multiple of the subnormal quantum 2^(emin-mbits)
        const float magic = __uint_as_float((uint32_t)(emin - F::mbits + 23 + 127) << 23);
        mag = __float_as_uint(__fadd_rn(__uint_as_float(a), magic)) - __float_as_uint(magic);
    } else {
        // normal target: round the 23-bit fraction to mbits, carry runs into the exponent
        const uint32_t r = a + ((1u << (22 - F::mbits)) - 1u) + ((a >> (23 - F::mbits)) & 1u);
        mag = (r >> (23 - F::mbits)) - ((uint32_t)(127 - F::bias) << F::mbits);
    }
    if (mag > F::max_mag) mag = NOSAT ? F::overflow_mag : F::max_mag;
    return sign | mag;
}

// Scaled value y of input element x -> code.  The multiply does not keep the sign
// of a NaN operand on this hardware, so a NaN code takes its sign from x.
template <int FMT, bool NOSAT>
__device__ __forceinline__ uint32_t encode_scaled(float y, uint32_t x_sign_bit31) {
    if (y != y) return ((x_sign_bit31 >> 24) & 0x80u) | 0x7Fu;
    return encode_scalar<FMT, NOSAT>(y);
}

// Two binary32 values -> two codes (lo in bits 0..7, hi in bits 8..15), hardware RNE,
// finite overflow saturated.  Only valid for finite inputs (callers check).
template <int FMT>
__device__ __forceinline__ uint32_t cvt_pair(float lo, float hi) {
    uint16_t r;
    if (FMT == kE4M3) asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    else              asm("cvt.rn.satfinite.e5m2x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}

template <int FMT>
__device__ __forceinline__ uint32_t cvt_quad(float v0, float v1, float v2, float v3) {
    return cvt_pair<FMT>(v0, v1) | (cvt_pair<FMT>(v2, v3) << 16);
}

// Two codes (bits 0..15) -> two binary32 values.  Every FP8 value is a binary16
// value, so the hardware e4m3x2/e5m2x2 -> f16x2 convert is exact.
template <int FMT>
__device__ __forceinline__ float2 decode_pair(uint32_t two_codes) {
    uint32_t h2;
    const uint16_t c = (uint16_t)two_codes;
    if (FMT == kE4M3) asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(c));
    else              asm("cvt.rn.f16x2.e5m2x2 %0, %1;" : "=r"(h2) : "h"(c));
    return __half22float2(*reinterpret_cast<__half2*>(&h2));
}

// binary32 pair -> packed bf16 pair (lo in the low half), RNE.
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

}  // namespace fp8b200
