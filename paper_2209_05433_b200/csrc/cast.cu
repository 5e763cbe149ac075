// amax, scale selection, quantize (wide -> FP8) and dequantize (FP8 -> wide):
// the memory-bound half of the FP8 hot path (Section 2 of the paper).
//
// The flat tensor kernels (amax, quantize, dequantize, the simulated round trip) work on chunks of 16-byte
// items with several independent 128-bit loads in flight per thread, one or two chunks per block, the blocks
// handed out in order by the hardware scheduler; the one-launch current scaling is a co-resident (cooperative)
// grid-stride loop with a grid barrier between its passes.  Every warp-level load and store instruction
// covers one contiguous span.  Consecutive kernels of a stream overlap their launch with the predecessor's
// tail (programmatic dependent launch).  HBM traffic is the algorithmic minimum (each input byte read once per pass, each
// output byte written once).  The 2-D kernels (per-row / per-column scales, quantize with a transposed
// copy) follow the same rules with shapes of their own, described at each kernel.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>
#include <mutex>

#include "codec.cuh"
#include "common.cuh"

namespace fp8b200 {

static std::atomic<uint64_t> g_launches{0};
void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

fp8_status launch_quantize_current(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o, uint8_t* out,
                                   float* amax, float* scale, float* scale_inv, unsigned int* ws, cudaStream_t st);
fp8_status launch_grid_barrier_self_test(long long limit_cycles, cudaStream_t st);

int sm_count() {
    static std::mutex mu;
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
        cached[dev] = v;
    }
    return cached[dev];
}

constexpr int kWideF32 = 0;
constexpr int kWideBF16 = 1;
constexpr int kThreads = 256;

// Input loads of the streaming kernels take the read-only path without L1 allocation (plain loads are a few
// per cent faster on tensors far larger than L2 but slower whenever part of the tensor sits in L2).
__device__ __forceinline__ uint4 ld_in_v4(const void* p) { return ld_nc_v4(p); }
__device__ __forceinline__ uint2 ld_in_v2(const void* p) { return ld_nc_v2(p); }

// Output stores: written once, never re-read by the same kernel; default write-back policy.
template <typename T>
__device__ __forceinline__ void st_out(T* p, T v) { *p = v; }

// ---------------------------------------------------------------------------
// per-item arithmetic
// ---------------------------------------------------------------------------

// Magnitude bits of one 16-byte item folded into a running maximum.
// bf16: packed 16-bit maxima (two lanes per word); f32: 32-bit maxima.
template <int WIDE>
__device__ __forceinline__ uint32_t fold_abs_max(uint32_t m, const uint4& v) {
    if (WIDE == kWideBF16) {
        m = __vmaxu2(m, v.x & 0x7FFF7FFFu);
        m = __vmaxu2(m, v.y & 0x7FFF7FFFu);
        m = __vmaxu2(m, v.z & 0x7FFF7FFFu);
        m = __vmaxu2(m, v.w & 0x7FFF7FFFu);
    } else {
        m = max(m, v.x & 0x7FFFFFFFu);
        m = max(m, v.y & 0x7FFFFFFFu);
        m = max(m, v.z & 0x7FFFFFFFu);
        m = max(m, v.w & 0x7FFFFFFFu);
    }
    return m;
}

// Running maximum -> binary32 magnitude pattern with NaN made canonical.
template <int WIDE>
__device__ __forceinline__ uint32_t finish_abs_max(uint32_t m) {
    if (WIDE == kWideBF16) m = max(m & 0xFFFFu, m >> 16) << 16;
    return canonical_nan_bits(m);
}

template <int WIDE>
__device__ __forceinline__ uint32_t scalar_abs_bits(const void* x, size_t i) {
    if (WIDE == kWideBF16) return ((uint32_t)(reinterpret_cast<const uint16_t*>(x)[i]) & 0x7FFFu) << 16;
    return reinterpret_cast<const uint32_t*>(x)[i] & 0x7FFFFFFFu;
}

template <int WIDE>
__device__ __forceinline__ float scalar_load(const void* x, size_t i) {
    if (WIDE == kWideBF16) return __uint_as_float((uint32_t)(reinterpret_cast<const uint16_t*>(x)[i]) << 16);
    return reinterpret_cast<const float*>(x)[i];
}

// True when the hardware convert cannot be used for this group of scaled values:
// a NaN or infinity is present (y * 0 is NaN exactly then), or, in the
// non-saturating mode, a magnitude reaches the overflow threshold.
template <int FMT, bool NOSAT, int N>
__device__ __forceinline__ bool needs_scalar_path(const float (&y)[N]) {
    float poison = 0.0f;
#pragma unroll
    for (int i = 0; i < N; ++i) poison = fmaf(y[i], 0.0f, poison);
    bool slow = poison != poison;
    if (NOSAT) {
        float top = 0.0f;
#pragma unroll
        for (int i = 0; i < N; ++i) top = fmaxf(top, fabsf(y[i]));
        slow = slow || (Fmt<FMT>::nosat_limit_inclusive ? top >= Fmt<FMT>::nosat_limit : top > Fmt<FMT>::nosat_limit);
    }
    return slow;
}

// 8 bf16 values (one 16-byte item) -> 8 codes.
template <int FMT, bool NOSAT>
__device__ __forceinline__ uint2 quantize_item_bf16(const uint4& v, float scale) {
    float y[8];
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        y[2 * i] = __uint_as_float(w[i] << 16) * scale;
        y[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u) * scale;
    }
    uint2 c;
    if (!needs_scalar_path<FMT, NOSAT>(y)) {
        c.x = cvt_quad<FMT>(y[0], y[1], y[2], y[3]);
        c.y = cvt_quad<FMT>(y[4], y[5], y[6], y[7]);
    } else {
        uint32_t code[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {                       // sign of x: bit 15 (low half) / bit 31 (high half)
            code[2 * i] = encode_scaled<FMT, NOSAT>(y[2 * i], w[i] << 16);
            code[2 * i + 1] = encode_scaled<FMT, NOSAT>(y[2 * i + 1], w[i]);
        }
        c.x = code[0] | (code[1] << 8) | (code[2] << 16) | (code[3] << 24);
        c.y = code[4] | (code[5] << 8) | (code[6] << 16) | (code[7] << 24);
    }
    return c;
}

// 4 binary32 values (one 16-byte item) -> 4 codes.
template <int FMT, bool NOSAT>
__device__ __forceinline__ uint32_t quantize_item_f32(const uint4& v, float scale) {
    float y[4] = {__uint_as_float(v.x) * scale, __uint_as_float(v.y) * scale,
                  __uint_as_float(v.z) * scale, __uint_as_float(v.w) * scale};
    if (!needs_scalar_path<FMT, NOSAT>(y)) return cvt_quad<FMT>(y[0], y[1], y[2], y[3]);
    return encode_scaled<FMT, NOSAT>(y[0], v.x) | (encode_scaled<FMT, NOSAT>(y[1], v.y) << 8) |
           (encode_scaled<FMT, NOSAT>(y[2], v.z) << 16) | (encode_scaled<FMT, NOSAT>(y[3], v.w) << 24);
}

// ---------------------------------------------------------------------------
// kernels: 16-byte aligned fast path
// ---------------------------------------------------------------------------

// One word set to zero: the start value of an amax accumulated with atomicMax by the kernel launched next.
// It lets that kernel be scheduled at once (so its launch overlaps this kernel's wait for everything earlier in the
// stream), then waits, then writes; the kernel behind it waits for this one before it touches memory.
__global__ void k_zero_word(uint32_t* p) {
    grid_launch_dependents();
    grid_dependency_wait();
    *p = 0u;
}

// amax over n elements.  Launched behind k_zero_word(amax_bits), which has zeroed the accumulator.
template <int WIDE, int UNROLL>
__global__ void __launch_bounds__(kThreads) k_amax(const void* __restrict__ x, size_t n, uint32_t* amax_bits) {
    __shared__ uint32_t red[32];
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;              // elements per 16-byte item
    grid_dependency_wait();
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    const size_t n_items = n / EPI;
    const size_t per_chunk = (size_t)kThreads * UNROLL;
    const size_t n_chunks = (n_items + per_chunk - 1) / per_chunk;
    uint32_t m = 0;
    for (size_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const size_t base = chunk * per_chunk + threadIdx.x;
        uint4 v[UNROLL];
        if (base + (size_t)(UNROLL - 1) * kThreads < n_items) {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) v[u] = ld_in_v4(xv + base + (size_t)u * kThreads);
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) m = fold_abs_max<WIDE>(m, v[u]);
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (i < n_items) m = fold_abs_max<WIDE>(m, ld_in_v4(xv + i));
            }
        }
    }
    m = finish_abs_max<WIDE>(m);
    if (blockIdx.x == 0 && threadIdx.x < n - n_items * EPI)      // ragged tail, fewer than EPI elements
        m = max(m, canonical_nan_bits(scalar_abs_bits<WIDE>(x, n_items * EPI + threadIdx.x)));
    grid_launch_dependents();
    block_atomic_max_bits(m, red, amax_bits);
}

// quantize n elements (+ optional amax of the input in the same pass; the kernel is then launched behind k_zero_word).
template <int WIDE, int FMT, bool NOSAT, bool WITH_AMAX, int UNROLL>
__global__ void __launch_bounds__(kThreads)
k_quantize(const void* __restrict__ x, size_t n, const float* __restrict__ scale_dev,
           uint8_t* __restrict__ out, uint32_t* amax_bits, int reverse) {
    __shared__ uint32_t red[32];
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    grid_dependency_wait();
    const float scale = *scale_dev;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    const size_t n_items = n / EPI;
    const size_t per_chunk = (size_t)kThreads * UNROLL;
    const size_t n_chunks = (n_items + per_chunk - 1) / per_chunk;
    uint32_t m = 0;

    auto emit = [&](size_t i, const uint4& v) {
        if (WITH_AMAX) m = fold_abs_max<WIDE>(m, v);
        if (WIDE == kWideBF16) st_out(reinterpret_cast<uint2*>(out) + i, quantize_item_bf16<FMT, NOSAT>(v, scale));
        else                   st_out(reinterpret_cast<uint32_t*>(out) + i, quantize_item_f32<FMT, NOSAT>(v, scale));
    };

    // `reverse`: the first blocks take the last chunks (the part of x a preceding amax pass read last is still in L2)
    for (size_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const size_t base = (reverse ? n_chunks - 1 - chunk : chunk) * per_chunk + threadIdx.x;
        if (base + (size_t)(UNROLL - 1) * kThreads < n_items) {
            uint4 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) v[u] = ld_in_v4(xv + base + (size_t)u * kThreads);
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) emit(base + (size_t)u * kThreads, v[u]);
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (i < n_items) emit(i, ld_in_v4(xv + i));
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < n - n_items * EPI) {    // ragged tail
        const size_t i = n_items * EPI + threadIdx.x;
        if (WITH_AMAX) {
            const uint32_t b = scalar_abs_bits<WIDE>(x, i);
            m = WIDE == kWideBF16 ? __vmaxu2(m, b >> 16) : max(m, b);    // bf16 keeps two packed 16-bit lanes
        }
        const float xf = scalar_load<WIDE>(x, i);
        out[i] = (uint8_t)encode_scaled<FMT, NOSAT>(xf * scale, __float_as_uint(xf));
    }
    grid_launch_dependents();
    if (WITH_AMAX) block_atomic_max_bits(finish_abs_max<WIDE>(m), red, amax_bits);
}

// dequantize: 8 codes (bf16 out) or 4 codes (f32 out) per item, one 16-byte store each.
template <int FMT, int WIDE, int UNROLL>
__global__ void __launch_bounds__(kThreads)
k_dequantize(const uint8_t* __restrict__ c, size_t n, const float* __restrict__ scale_inv_dev, void* __restrict__ out) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    grid_dependency_wait();
    const float si = *scale_inv_dev;
    const size_t n_items = n / EPI;
    const size_t per_chunk = (size_t)kThreads * UNROLL;
    const size_t n_chunks = (n_items + per_chunk - 1) / per_chunk;

    auto emit_bf16 = [&](size_t i, uint2 w) {
        const float2 a = decode_pair<FMT>(w.x), b = decode_pair<FMT>(w.x >> 16);
        const float2 d = decode_pair<FMT>(w.y), e = decode_pair<FMT>(w.y >> 16);
        uint4 o;
        o.x = pack_bf16(a.x * si, a.y * si);
        o.y = pack_bf16(b.x * si, b.y * si);
        o.z = pack_bf16(d.x * si, d.y * si);
        o.w = pack_bf16(e.x * si, e.y * si);
        st_out(reinterpret_cast<uint4*>(out) + i, o);
    };
    auto emit_f32 = [&](size_t i, uint32_t w) {
        const float2 a = decode_pair<FMT>(w), b = decode_pair<FMT>(w >> 16);
        st_out(reinterpret_cast<float4*>(out) + i, make_float4(a.x * si, a.y * si, b.x * si, b.y * si));
    };

    for (size_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const size_t base = chunk * per_chunk + threadIdx.x;
        const bool full = base + (size_t)(UNROLL - 1) * kThreads < n_items;
        if (WIDE == kWideBF16) {
            uint2 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (full || i < n_items) v[u] = ld_in_v2(c + i * 8);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (full || i < n_items) emit_bf16(i, v[u]);
            }
        } else {
            uint32_t v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (full || i < n_items) v[u] = ld_nc_u32(c + i * 4);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (full || i < n_items) emit_f32(i, v[u]);
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < n - n_items * EPI) {    // ragged tail
        const size_t i = n_items * EPI + threadIdx.x;
        const float v = decode_pair<FMT>(c[i]).x * si;
        if (WIDE == kWideBF16) reinterpret_cast<uint16_t*>(out)[i] = (uint16_t)pack_bf16(v, 0.0f);
        else                   reinterpret_cast<float*>(out)[i] = v;
    }
    grid_launch_dependents();
}

// ---------------------------------------------------------------------------
// kernels: element-wise path for pointers that are not 16-byte aligned
// ---------------------------------------------------------------------------

template <int WIDE>
__global__ void __launch_bounds__(kThreads) k_amax_elementwise(const void* __restrict__ x, size_t n, uint32_t* amax_bits) {
    __shared__ uint32_t red[32];
    uint32_t m = 0;
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (size_t)gridDim.x * kThreads)
        m = max(m, scalar_abs_bits<WIDE>(x, i));
    block_atomic_max_bits(canonical_nan_bits(m), red, amax_bits);
}

template <int WIDE, int FMT, bool NOSAT, bool WITH_AMAX>
__global__ void __launch_bounds__(kThreads)
k_quantize_elementwise(const void* __restrict__ x, size_t n, const float* __restrict__ scale_dev,
                       uint8_t* __restrict__ out, uint32_t* amax_bits) {
    __shared__ uint32_t red[32];
    const float scale = *scale_dev;
    uint32_t m = 0;
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (size_t)gridDim.x * kThreads) {
        if (WITH_AMAX) m = max(m, scalar_abs_bits<WIDE>(x, i));
        const float xf = scalar_load<WIDE>(x, i);
        out[i] = (uint8_t)encode_scaled<FMT, NOSAT>(xf * scale, __float_as_uint(xf));
    }
    if (WITH_AMAX) block_atomic_max_bits(canonical_nan_bits(m), red, amax_bits);
}

template <int FMT, int WIDE>
__global__ void __launch_bounds__(kThreads)
k_dequantize_elementwise(const uint8_t* __restrict__ c, size_t n, const float* __restrict__ scale_inv_dev, void* __restrict__ out) {
    const float si = *scale_inv_dev;
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (size_t)gridDim.x * kThreads) {
        const float v = decode_pair<FMT>(c[i]).x * si;
        if (WIDE == kWideBF16) reinterpret_cast<uint16_t*>(out)[i] = (uint16_t)pack_bf16(v, 0.0f);
        else                   reinterpret_cast<float*>(out)[i] = v;
    }
}

// SM clock probe: one thread reads the SM cycle counter and the nanosecond timer, waits `duration_ns` (bounded
// by an iteration count as well), reads both again.  out[0] = SM clocks, out[1] = nanoseconds.
__global__ void k_sm_clock_probe(unsigned long long* out, unsigned long long duration_ns) {
    if (threadIdx.x != 0) return;
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t0));
    const long long c0 = clock64();
    t = t0;
    for (unsigned int i = 0; i < 50000000u && t - t0 < duration_ns; ++i) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    const long long c1 = clock64();
    out[0] = (unsigned long long)(c1 - c0);
    out[1] = t - t0;
}

// scale = fmax / amax with the guards of the interface; one thread.
__global__ void k_scale_from_amax(const float* amax_dev, float fmax, float* scale_dev, float* scale_inv_dev) {
    grid_dependency_wait();
    const float a = *amax_dev;
    float s = 1.0f;
    if (a == a && a != 0.0f && fabsf(a) != __int_as_float(0x7F800000)) {
        s = __fdiv_rn(fmax, a);
        if (fabsf(s) == __int_as_float(0x7F800000)) s = __int_as_float(0x7F7FFFFF);
    }
    *scale_dev = s;
    *scale_inv_dev = __fdiv_rn(1.0f, s);
}

// scale and inverse scale from an amax value: the arithmetic of k_scale_from_amax, callable from other kernels
__device__ __forceinline__ void scale_pair_from_amax(float a, float fmax, float& s, float& si) {
    s = 1.0f;
    if (a == a && a != 0.0f && fabsf(a) != __int_as_float(0x7F800000)) {
        s = __fdiv_rn(fmax, a);
        if (fabsf(s) == __int_as_float(0x7F800000)) s = __int_as_float(0x7F7FFFFF);
    }
    si = __fdiv_rn(1.0f, s);
}

// Error latch of the cast kernels' bounded waits: [0] = code, [1] = block.
__device__ unsigned int g_cast_latch[2] = {0u, 0u};
constexpr unsigned int kWaitGridBarrier = 16u;
constexpr long long kGridWaitLimitCycles = 4000000000ll;       // about 2 s of SM clocks

// One-launch current scaling of a tensor larger than kCurrentKeepFromMB: the last kCurrentKeepMB megabytes read by
// the first pass are asked to stay in L2 (the second pass starts there), the rest to leave first.  Smaller tensors
// are left to the default replacement: they mostly fit.
constexpr size_t kCurrentKeepMB = 96, kCurrentKeepFromMB = 160;
// From this input size on, fp8_quantize_current runs the three streaming kernels instead of the one cooperative
// launch: their scheduler-balanced blocks beat the co-resident grid on long streams (2^28 bf16 elements: +2 %,
// 2^30: +8 %), where a few launch gaps do not show; below it the two are within noise of each other.
constexpr size_t kCurrentChainFromBytes = (size_t)256 << 20;
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint4 ld_v4_policy(const void* ptr, uint64_t policy) {
    uint4 v;
    asm volatile("ld.global.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(ptr), "l"(policy));
    return v;
}


// Grid-wide barrier of the one-launch kernels (all CTAs co-resident), bounded: thread 0 of every CTA announces its
// arrival in ws[1] and polls until `arrivals` CTAs have, or gives up after `wait_limit` SM clocks (latching the time-out).
// bcast[0] receives the running amax bits of ws[0], bcast[1] whether the barrier held.  Ends with __syncthreads.
__device__ __forceinline__ void grid_barrier_read_amax(unsigned int* ws, unsigned int arrivals, long long wait_limit, uint32_t* bcast) {
    if (threadIdx.x == 0) {
        __threadfence();
        atomicAdd(&ws[1], 1u);
        uint32_t okflag = 1u;
        long long t0 = 0;
        for (uint32_t spins = 1;; ++spins) {
            unsigned int arrived;
            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(arrived) : "l"(&ws[1]) : "memory");
            if (arrived >= arrivals) break;
            if ((spins & 255u) == 0u) {
                const long long now = clock64();
                if (t0 == 0) t0 = now;
                else if (now - t0 > wait_limit) {
                    if (atomicCAS(&g_cast_latch[0], 0u, kWaitGridBarrier) == 0u) g_cast_latch[1] = blockIdx.x;
                    okflag = 0u;
                    break;
                }
            }
        }
        unsigned int bits;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(bits) : "l"(&ws[0]) : "memory");
        bcast[0] = bits;
        bcast[1] = okflag;
    }
    __syncthreads();
}

// Leaves the control words as they were found: the last CTA out zeroes them (also after a time-out).
__device__ __forceinline__ void leave_and_reset(unsigned int* ws) {
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int gone = atomicAdd(&ws[2], 1u);
        if (gone == gridDim.x - 1) {
            ws[0] = 0u;
            ws[2] = 0u;
            __threadfence();
            ws[1] = 0u;
        }
    }
}

// Current scaling in ONE launch: amax of x, scale = fmax / amax, quantize with that scale.
// All CTAs are co-resident (cooperative launch).  ws[0] = running amax bits, ws[1] = arrivals at the
// grid barrier, ws[2] = departures; the three words are zero on entry and the last CTA to leave puts
// them back to zero.  The second pass walks each CTA's chunks in reverse so that the part of x read
// last in the first pass is re-read from L2.
// `arrivals` is the number of CTAs the barrier waits for (the grid size; the wait self-test passes one more, which
// can never arrive) and `wait_limit` the SM clocks a CTA waits before it gives up.
template <int WIDE, int FMT, bool NOSAT, int UNROLL>
__global__ void __launch_bounds__(kThreads)
k_quantize_current(const void* __restrict__ x, size_t n, float fmax, uint8_t* __restrict__ out,
                   float* amax_out, float* scale_out, float* scale_inv_out, unsigned int* ws,
                   unsigned int arrivals, long long wait_limit) {
    __shared__ uint32_t red[32];
    __shared__ uint32_t bcast[2];
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    const size_t n_items = n / EPI;
    const size_t per_chunk = (size_t)kThreads * UNROLL;
    const size_t n_chunks = (n_items + per_chunk - 1) / per_chunk;
    const size_t tail = n - n_items * EPI;

    // ---- pass 1: amax
    const bool large = n_chunks * per_chunk * 16 > (kCurrentKeepFromMB << 20);
    const uint64_t pol_keep = l2_policy_evict_last(), pol_stream = l2_policy_evict_first();
    const size_t keep_chunks = (kCurrentKeepMB << 20) / (per_chunk * 16);
    const size_t keep_from = n_chunks > keep_chunks ? n_chunks - keep_chunks : 0;
    uint32_t m = 0;
    for (size_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const size_t base = chunk * per_chunk + threadIdx.x;
        if (base + (size_t)(UNROLL - 1) * kThreads < n_items) {
            uint4 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                if (large) v[u] = ld_v4_policy(xv + base + (size_t)u * kThreads, chunk >= keep_from ? pol_keep : pol_stream);
                else       v[u] = *(xv + base + (size_t)u * kThreads);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) m = fold_abs_max<WIDE>(m, v[u]);
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (i < n_items) m = fold_abs_max<WIDE>(m, *(xv + i));
            }
        }
    }
    m = finish_abs_max<WIDE>(m);
    if (blockIdx.x == 0 && threadIdx.x < tail)
        m = max(m, canonical_nan_bits(scalar_abs_bits<WIDE>(x, n_items * EPI + threadIdx.x)));
    block_atomic_max_bits(m, red, ws);

    // ---- grid barrier (bounded), then every CTA reads the same amax
    grid_barrier_read_amax(ws, arrivals, wait_limit, bcast);
    const float amax = __uint_as_float(bcast[0]);
    const bool ok = bcast[1] != 0u;
    float scale, scale_inv;
    scale_pair_from_amax(amax, fmax, scale, scale_inv);
    if (blockIdx.x == 0 && threadIdx.x == 0 && ok) {
        *amax_out = amax;
        *scale_out = scale;
        *scale_inv_out = scale_inv;
    }

    // ---- pass 2: quantize, this CTA's chunks in reverse order
    if (ok && n_chunks > blockIdx.x) {
        const size_t my_chunks = (n_chunks - blockIdx.x + gridDim.x - 1) / gridDim.x;
        for (size_t c = my_chunks; c-- > 0;) {
            const size_t chunk = blockIdx.x + c * gridDim.x;
            const size_t base = chunk * per_chunk + threadIdx.x;
            if (base + (size_t)(UNROLL - 1) * kThreads < n_items) {
                uint4 v[UNROLL];
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) v[u] = *(xv + base + (size_t)u * kThreads);      // plain loads: the re-read hits L2
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const size_t i = base + (size_t)u * kThreads;
                    if (WIDE == kWideBF16) st_out(reinterpret_cast<uint2*>(out) + i, quantize_item_bf16<FMT, NOSAT>(v[u], scale));
                    else                   st_out(reinterpret_cast<uint32_t*>(out) + i, quantize_item_f32<FMT, NOSAT>(v[u], scale));
                }
            } else {
#pragma unroll
                for (int u = 0; u < UNROLL; ++u) {
                    const size_t i = base + (size_t)u * kThreads;
                    if (i < n_items) {
                        const uint4 v = ld_in_v4(xv + i);
                        if (WIDE == kWideBF16) st_out(reinterpret_cast<uint2*>(out) + i, quantize_item_bf16<FMT, NOSAT>(v, scale));
                        else                   st_out(reinterpret_cast<uint32_t*>(out) + i, quantize_item_f32<FMT, NOSAT>(v, scale));
                    }
                }
            }
        }
    }
    if (ok && blockIdx.x == 0 && threadIdx.x < tail) {
        const size_t i = n_items * EPI + threadIdx.x;
        const float xf = scalar_load<WIDE>(x, i);
        out[i] = (uint8_t)encode_scaled<FMT, NOSAT>(xf * scale, __float_as_uint(xf));
    }

    leave_and_reset(ws);
}

// The same conversion for a tensor that fits the shared memory of the whole GPU (one CTA per SM, each keeping its
// contiguous slice of x in shared memory between the passes): x is read from global memory ONCE (3 B of traffic per
// bf16 element instead of 5).  Pass 1 copies the slice into shared memory and folds the amax, the bounded grid barrier
// follows, pass 2 converts from shared memory.  n is a multiple of the elements per 16-byte item here (the launcher
// sends ragged sizes elsewhere); ws as in k_quantize_current.
constexpr int kResidentThreads = 1024;
template <int WIDE, int FMT, bool NOSAT>
__global__ void __launch_bounds__(kResidentThreads, 1)
k_quantize_current_resident(const void* __restrict__ x, size_t n_items, size_t items_per_cta, float fmax, uint8_t* __restrict__ out,
                            float* amax_out, float* scale_out, float* scale_inv_out, unsigned int* ws,
                            unsigned int arrivals, long long wait_limit) {
    extern __shared__ uint4 slice[];
    __shared__ uint32_t red[32];
    __shared__ uint32_t bcast[2];
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    const size_t first = (size_t)blockIdx.x * items_per_cta;
    const size_t mine = first < n_items ? min(items_per_cta, n_items - first) : 0;

    // ---- pass 1: global -> shared, amax on the way (four loads in flight per thread)
    uint32_t m = 0;
    size_t i = threadIdx.x;
    for (; i + 3 * (size_t)kResidentThreads < mine; i += 4 * (size_t)kResidentThreads) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_in_v4(xv + first + i + (size_t)u * kResidentThreads);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            slice[i + (size_t)u * kResidentThreads] = v[u];
            m = fold_abs_max<WIDE>(m, v[u]);
        }
    }
    for (; i < mine; i += kResidentThreads) {
        const uint4 v = ld_in_v4(xv + first + i);
        slice[i] = v;
        m = fold_abs_max<WIDE>(m, v);
    }
    block_atomic_max_bits(finish_abs_max<WIDE>(m), red, ws);

    grid_barrier_read_amax(ws, arrivals, wait_limit, bcast);
    const float amax = __uint_as_float(bcast[0]);
    const bool ok = bcast[1] != 0u;
    float scale, scale_inv;
    scale_pair_from_amax(amax, fmax, scale, scale_inv);
    if (blockIdx.x == 0 && threadIdx.x == 0 && ok) {
        *amax_out = amax;
        *scale_out = scale;
        *scale_inv_out = scale_inv;
    }

    // ---- pass 2: shared -> codes (every thread re-reads the items it wrote itself)
    if (ok) {
        for (size_t j = threadIdx.x; j < mine; j += kResidentThreads) {
            const uint4 v = slice[j];
            if (WIDE == kWideBF16) st_out(reinterpret_cast<uint2*>(out) + first + j, quantize_item_bf16<FMT, NOSAT>(v, scale));
            else                   st_out(reinterpret_cast<uint32_t*>(out) + first + j, quantize_item_f32<FMT, NOSAT>(v, scale));
        }
    }
    leave_and_reset(ws);
}

// ---------------------------------------------------------------------------
// fake quantization: wide -> FP8 -> wide in one pass (what the simulated-FP8 experiments of Section 4 run)
// ---------------------------------------------------------------------------

// one scaled value -> its FP8 code -> back to binary32 times scale_inv (scalar path, any input)
template <int FMT, bool NOSAT>
__device__ __forceinline__ float fake_one(float xf, float scale, float scale_inv) {
    const uint32_t code = encode_scaled<FMT, NOSAT>(xf * scale, __float_as_uint(xf));
    return decode_pair<FMT>(code).x * scale_inv;
}

template <int WIDE, int FMT, bool NOSAT, int UNROLL>
__global__ void __launch_bounds__(kThreads)
k_fake_quantize(const void* __restrict__ x, size_t n, const float* __restrict__ scale_dev,
                const float* __restrict__ scale_inv_dev, void* __restrict__ out) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    grid_dependency_wait();
    const float scale = *scale_dev, si = *scale_inv_dev;
    const uint4* xv = reinterpret_cast<const uint4*>(x);
    const size_t n_items = n / EPI;
    const size_t per_chunk = (size_t)kThreads * UNROLL;
    const size_t n_chunks = (n_items + per_chunk - 1) / per_chunk;

    auto emit = [&](size_t i, const uint4& v) {
        if (WIDE == kWideBF16) {
            const uint2 c = quantize_item_bf16<FMT, NOSAT>(v, scale);
            const float2 a = decode_pair<FMT>(c.x), b = decode_pair<FMT>(c.x >> 16);
            const float2 d = decode_pair<FMT>(c.y), e = decode_pair<FMT>(c.y >> 16);
            uint4 o;
            o.x = pack_bf16(a.x * si, a.y * si);
            o.y = pack_bf16(b.x * si, b.y * si);
            o.z = pack_bf16(d.x * si, d.y * si);
            o.w = pack_bf16(e.x * si, e.y * si);
            st_out(reinterpret_cast<uint4*>(out) + i, o);
        } else {
            const uint32_t c = quantize_item_f32<FMT, NOSAT>(v, scale);
            const float2 a = decode_pair<FMT>(c), b = decode_pair<FMT>(c >> 16);
            st_out(reinterpret_cast<float4*>(out) + i, make_float4(a.x * si, a.y * si, b.x * si, b.y * si));
        }
    };

    for (size_t chunk = blockIdx.x; chunk < n_chunks; chunk += gridDim.x) {
        const size_t base = chunk * per_chunk + threadIdx.x;
        if (base + (size_t)(UNROLL - 1) * kThreads < n_items) {
            uint4 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) v[u] = ld_nc_v4(xv + base + (size_t)u * kThreads);
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) emit(base + (size_t)u * kThreads, v[u]);
        } else {
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const size_t i = base + (size_t)u * kThreads;
                if (i < n_items) emit(i, ld_nc_v4(xv + i));
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < n - n_items * EPI) {    // ragged tail
        const size_t i = n_items * EPI + threadIdx.x;
        const float v = fake_one<FMT, NOSAT>(scalar_load<WIDE>(x, i), scale, si);
        if (WIDE == kWideBF16) reinterpret_cast<uint16_t*>(out)[i] = (uint16_t)pack_bf16(v, 0.0f);
        else                   reinterpret_cast<float*>(out)[i] = v;
    }
    grid_launch_dependents();
}

template <int WIDE, int FMT, bool NOSAT>
__global__ void __launch_bounds__(kThreads)
k_fake_quantize_elementwise(const void* __restrict__ x, size_t n, const float* __restrict__ scale_dev,
                            const float* __restrict__ scale_inv_dev, void* __restrict__ out) {
    const float scale = *scale_dev, si = *scale_inv_dev;
    for (size_t i = (size_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (size_t)gridDim.x * kThreads) {
        const float v = fake_one<FMT, NOSAT>(scalar_load<WIDE>(x, i), scale, si);
        if (WIDE == kWideBF16) reinterpret_cast<uint16_t*>(out)[i] = (uint16_t)pack_bf16(v, 0.0f);
        else                   reinterpret_cast<float*>(out)[i] = v;
    }
}

// power-of-two scale: the largest power of two not above fmax / amax (same guards as k_scale_from_amax).
// With such a scale the conversion is the paper's variant with a programmable exponent bias (Section 3.2).
__global__ void k_scale_pow2_from_amax(const float* amax_dev, float fmax, float* scale_dev, float* scale_inv_dev) {
    float s, si;
    grid_dependency_wait();
    scale_pair_from_amax(*amax_dev, fmax, s, si);
    uint32_t b = __float_as_uint(s);
    if ((b >> 23) != 0u) b &= 0x7F800000u;                       // normal: drop the fraction
    else if (b != 0u) b = 1u << (31 - __clz(b));                  // subnormal: keep the leading bit
    s = __uint_as_float(b);
    *scale_dev = s;
    *scale_inv_dev = __fdiv_rn(1.0f, s);
}

// ---------------------------------------------------------------------------
// per-channel scales (Section 4.2: per-channel for weights, per-tensor for activations)
// x is rows x cols, row-major, pitch ld elements.  AXIS 0: one channel per column; AXIS 1: one per row.
// ---------------------------------------------------------------------------

// AXIS 0, vector path.  Block = 64 items wide x 4 row lanes: a thread owns one 16-byte item of columns
// (8 bf16 / 4 f32) and every fourth row of the block's slab; per-column maxima stay separate inside the
// packed words.  The four row lanes meet in shared memory, then one atomicMax per column per block.
// amax_bits[cols] must be zero before.
constexpr int kColsMinRows = 256;
constexpr int kColsTx = 64, kColsTy = 4, kColsUnroll = 8;       // 64 x 4 threads, eight row loads in flight per thread
template <int WIDE>
__global__ void __launch_bounds__(kColsTx * kColsTy)
k_amax_cols(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, int64_t rows_per_slab, uint32_t* amax_bits) {
    __shared__ uint4 part[kColsTy][kColsTx];
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    const int tx = threadIdx.x, ty = threadIdx.y;
    const int64_t c0 = ((int64_t)blockIdx.x * kColsTx + tx) * EPI;
    const bool live = c0 < cols;
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_slab;
    const int64_t r1 = min(rows, r0 + rows_per_slab);
    const char* base = reinterpret_cast<const char*>(x) + c0 * ESZ;
    uint4 m = make_uint4(0u, 0u, 0u, 0u);
    auto fold = [&](const uint4& v) {
        if (WIDE == kWideBF16) {
            m.x = __vmaxu2(m.x, v.x & 0x7FFF7FFFu); m.y = __vmaxu2(m.y, v.y & 0x7FFF7FFFu);
            m.z = __vmaxu2(m.z, v.z & 0x7FFF7FFFu); m.w = __vmaxu2(m.w, v.w & 0x7FFF7FFFu);
        } else {
            m.x = max(m.x, v.x & 0x7FFFFFFFu); m.y = max(m.y, v.y & 0x7FFFFFFFu);
            m.z = max(m.z, v.z & 0x7FFFFFFFu); m.w = max(m.w, v.w & 0x7FFFFFFFu);
        }
    };
    if (live) {
        int64_t r = r0 + ty;
        for (; r + (kColsUnroll - 1) * kColsTy < r1; r += kColsUnroll * kColsTy) {
            uint4 v[kColsUnroll];
#pragma unroll
            for (int u = 0; u < kColsUnroll; ++u) v[u] = ld_in_v4(base + (r + u * kColsTy) * ld * ESZ);
#pragma unroll
            for (int u = 0; u < kColsUnroll; ++u) fold(v[u]);
        }
        for (; r < r1; r += kColsTy) fold(ld_in_v4(base + r * ld * ESZ));
    }
    part[ty][tx] = m;
    __syncthreads();
    if (ty == 0 && live) {
#pragma unroll
        for (int k = 1; k < kColsTy; ++k) {
            const uint4 o = part[k][tx];
            if (WIDE == kWideBF16) { m.x = __vmaxu2(m.x, o.x); m.y = __vmaxu2(m.y, o.y); m.z = __vmaxu2(m.z, o.z); m.w = __vmaxu2(m.w, o.w); }
            else                   { m.x = max(m.x, o.x); m.y = max(m.y, o.y); m.z = max(m.z, o.z); m.w = max(m.w, o.w); }
        }
        const uint32_t w[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
        for (int i = 0; i < EPI; ++i) {
            if (c0 + i < cols) {
                const uint32_t bits = WIDE == kWideBF16 ? (((i & 1) ? (w[i >> 1] >> 16) : (w[i >> 1] & 0xFFFFu)) << 16) : w[i];
                if (bits) atomicMax(&amax_bits[c0 + i], canonical_nan_bits(bits));
            }
        }
    }
}

// AXIS 1, vector path.  A row is cut into segments of 32 lanes x kRowsUnroll 16-byte items; a warp takes one
// (row, segment) unit at a time with all its loads in flight, so short-and-wide and tall-and-narrow tensors both
// fill the GPU.  One unit per row: the warp stores the row's amax; several: atomicMax onto a zeroed vector.
constexpr int kRowsUnroll = 4;
constexpr int kRowsAmaxUnroll = 8;
// amax: a unit is a row's span of `span` items (a multiple of 32 x kRowsAmaxUnroll), `segs` spans per row
template <int WIDE>
__global__ void __launch_bounds__(kThreads)
k_amax_rows(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, int64_t segs, int64_t span, uint32_t* amax_bits) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * kThreads) >> 5;
    const int64_t n_items = cols / EPI;
    for (int64_t u = warp; u < rows * segs; u += n_warps) {
        const int64_t r = u / segs, seg = u - r * segs;
        const char* row = reinterpret_cast<const char*>(x) + r * ld * ESZ;
        const int64_t end = min(n_items, (seg + 1) * span);
        int64_t i = seg * span + lane;
        uint32_t m = 0;
        for (; i + 32 * (kRowsAmaxUnroll - 1) < end; i += 32 * kRowsAmaxUnroll) {
            uint4 v[kRowsAmaxUnroll];
#pragma unroll
            for (int k = 0; k < kRowsAmaxUnroll; ++k) v[k] = ld_in_v4(row + (i + 32 * k) * 16);
#pragma unroll
            for (int k = 0; k < kRowsAmaxUnroll; ++k) m = fold_abs_max<WIDE>(m, v[k]);
        }
        for (; i < end; i += 32) m = fold_abs_max<WIDE>(m, ld_in_v4(row + i * 16));
        m = finish_abs_max<WIDE>(m);
        if (seg == segs - 1)                                          // ragged tail of the row
            for (int64_t c = n_items * EPI + lane; c < cols; c += 32) m = max(m, canonical_nan_bits(scalar_abs_bits<WIDE>(row, c)));
        m = warp_max_u32(m);
        if (lane == 0) {
            if (segs == 1) amax_bits[r] = m;
            else if (m) atomicMax(&amax_bits[r], m);
        }
    }
}

// any alignment: one thread per element, channel maxima by atomicMax (amax_bits zero before)
template <int WIDE, int AXIS>
__global__ void __launch_bounds__(kThreads)
k_amax_channels_elementwise(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, uint32_t* amax_bits) {
    const int64_t total = rows * cols;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kThreads) {
        const int64_t r = i / cols, c = i - r * cols;
        const uint32_t bits = canonical_nan_bits(scalar_abs_bits<WIDE>(x, r * ld + c));
        if (bits) atomicMax(&amax_bits[AXIS == 0 ? c : r], bits);
    }
}

// N scaled values with their source sign words -> packed codes (N = 4 or 8)
template <int FMT, bool NOSAT, int N>
__device__ __forceinline__ void encode_group(const float (&y)[N], const uint32_t (&xsign)[N], uint32_t (&codes)[N / 4]) {
    if (!needs_scalar_path<FMT, NOSAT>(y)) {
#pragma unroll
        for (int q = 0; q < N / 4; ++q) codes[q] = cvt_quad<FMT>(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
    } else {
#pragma unroll
        for (int q = 0; q < N / 4; ++q)
            codes[q] = encode_scaled<FMT, NOSAT>(y[4 * q], xsign[4 * q]) | (encode_scaled<FMT, NOSAT>(y[4 * q + 1], xsign[4 * q + 1]) << 8) |
                       (encode_scaled<FMT, NOSAT>(y[4 * q + 2], xsign[4 * q + 2]) << 16) | (encode_scaled<FMT, NOSAT>(y[4 * q + 3], xsign[4 * q + 3]) << 24);
    }
}

// one 16-byte item with one scale per element (AXIS 0) -> packed codes
template <int WIDE, int FMT, bool NOSAT>
__device__ __forceinline__ void quantize_item_scales(const uint4& v, const float* sc, uint32_t* codes) {
    if (WIDE == kWideBF16) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        float y[8];
        uint32_t xs[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            y[2 * i] = __uint_as_float(w[i] << 16) * sc[2 * i];
            y[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u) * sc[2 * i + 1];
            xs[2 * i] = w[i] << 16;
            xs[2 * i + 1] = w[i];
        }
        uint32_t c[2];
        encode_group<FMT, NOSAT, 8>(y, xs, c);
        codes[0] = c[0]; codes[1] = c[1];
    } else {
        float y[4] = {__uint_as_float(v.x) * sc[0], __uint_as_float(v.y) * sc[1], __uint_as_float(v.z) * sc[2], __uint_as_float(v.w) * sc[3]};
        uint32_t xs[4] = {v.x, v.y, v.z, v.w};
        uint32_t c[1];
        encode_group<FMT, NOSAT, 4>(y, xs, c);
        codes[0] = c[0];
    }
}

// AXIS 0, vector path.  Same 64 x 4 block shape as k_amax_cols: a thread keeps the scales of its item of
// columns in registers and converts every fourth row of the slab, four loads in flight.
template <int WIDE, int FMT, bool NOSAT>
__global__ void __launch_bounds__(kColsTx * kColsTy)
k_quantize_cols(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, int64_t rows_per_slab,
                const float* __restrict__ scale, uint8_t* __restrict__ out, int64_t ld_out) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    const int64_t c0 = ((int64_t)blockIdx.x * kColsTx + threadIdx.x) * EPI;
    if (c0 + EPI > cols) return;                                   // ragged right edge: handled by the tail kernel
    float sc[EPI];
#pragma unroll
    for (int i = 0; i < EPI; ++i) sc[i] = __ldg(scale + c0 + i);
    const int64_t r0 = (int64_t)blockIdx.y * rows_per_slab;
    const int64_t r1 = min(rows, r0 + rows_per_slab);
    const char* base = reinterpret_cast<const char*>(x) + c0 * ESZ;
    auto emit = [&](int64_t r, const uint4& v) {
        uint32_t c[2];
        quantize_item_scales<WIDE, FMT, NOSAT>(v, sc, c);
        if (WIDE == kWideBF16) st_out(reinterpret_cast<uint2*>(out + r * ld_out + c0), make_uint2(c[0], c[1]));
        else                   st_out(reinterpret_cast<uint32_t*>(out + r * ld_out + c0), c[0]);
    };
    int64_t r = r0 + threadIdx.y;
    for (; r + 3 * kColsTy < r1; r += 4 * kColsTy) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = ld_in_v4(base + (r + u * kColsTy) * ld * ESZ);
#pragma unroll
        for (int u = 0; u < 4; ++u) emit(r + u * kColsTy, v[u]);
    }
    for (; r < r1; r += kColsTy) emit(r, ld_in_v4(base + r * ld * ESZ));
}

// AXIS 1, vector path: a warp per (row, segment) unit as in k_amax_rows, the row's scale in a register.
template <int WIDE, int FMT, bool NOSAT>
__global__ void __launch_bounds__(kThreads)
k_quantize_rows(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, int64_t segs, const float* __restrict__ scale,
                uint8_t* __restrict__ out, int64_t ld_out) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * kThreads) >> 5;
    const int64_t n_items = cols / EPI;
    auto emit = [&](uint8_t* orow, int64_t i, const uint4& v, float s) {
        if (WIDE == kWideBF16) st_out(reinterpret_cast<uint2*>(orow) + i, quantize_item_bf16<FMT, NOSAT>(v, s));
        else                   st_out(reinterpret_cast<uint32_t*>(orow) + i, quantize_item_f32<FMT, NOSAT>(v, s));
    };
    for (int64_t u = warp; u < rows * segs; u += n_warps) {
        const int64_t r = u / segs, seg = u - r * segs;
        const float s = __ldg(scale + r);
        const char* row = reinterpret_cast<const char*>(x) + r * ld * ESZ;
        uint8_t* orow = out + r * ld_out;
        const int64_t i0 = seg * (32 * kRowsUnroll) + lane;
        if (i0 + 32 * (kRowsUnroll - 1) < n_items) {
            uint4 v[kRowsUnroll];
#pragma unroll
            for (int k = 0; k < kRowsUnroll; ++k) v[k] = ld_in_v4(row + (i0 + 32 * k) * 16);
#pragma unroll
            for (int k = 0; k < kRowsUnroll; ++k) emit(orow, i0 + 32 * k, v[k], s);
        } else {
            for (int64_t i = i0; i < n_items; i += 32) emit(orow, i, ld_in_v4(row + i * 16), s);
        }
        if (seg == segs - 1) {
            for (int64_t c = n_items * EPI + lane; c < cols; c += 32) {
                const float xf = scalar_load<WIDE>(row, c);
                orow[c] = (uint8_t)encode_scaled<FMT, NOSAT>(xf * s, __float_as_uint(xf));
            }
        }
    }
}

// any alignment / ragged columns [c_begin, cols): one thread per element
template <int WIDE, int FMT, bool NOSAT, int AXIS>
__global__ void __launch_bounds__(kThreads)
k_quantize_channels_elementwise(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ld, int64_t c_begin,
                                const float* __restrict__ scale, uint8_t* __restrict__ out, int64_t ld_out) {
    const int64_t width = cols - c_begin;
    const int64_t total = rows * width;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < total; i += (int64_t)gridDim.x * kThreads) {
        const int64_t r = i / width, c = c_begin + (i - r * width);
        const float xf = scalar_load<WIDE>(x, r * ld + c);
        out[r * ld_out + c] = (uint8_t)encode_scaled<FMT, NOSAT>(xf * __ldg(scale + (AXIS == 0 ? c : r)), __float_as_uint(xf));
    }
}

// `count` scales at once (per-channel); pow2 != 0 rounds each down to a power of two
__global__ void __launch_bounds__(kThreads)
k_scales_from_amax(const float* amax, int64_t count, float fmax, int pow2, float* scale, float* scale_inv) {
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < count; i += (int64_t)gridDim.x * kThreads) {
        float s, si;
        scale_pair_from_amax(amax[i], fmax, s, si);
        if (pow2) {
            uint32_t b = __float_as_uint(s);
            if ((b >> 23) != 0u) b &= 0x7F800000u;
            else if (b != 0u) b = 1u << (31 - __clz(b));
            s = __uint_as_float(b);
            si = __fdiv_rn(1.0f, s);
        }
        scale[i] = s;
        scale_inv[i] = si;
    }
}

// ---------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------

// ---------------------------------------------------------------------------
// quantize + transposed copy: codes of x[rows, cols] written row-major (optional) and as [cols, rows]
// ---------------------------------------------------------------------------

constexpr int kTrTile = 128;         // tile edge in elements: a transposed output row of one tile is one 128-byte line

// bytes (a0..a3 are four rows of four codes) -> four words holding the columns
__device__ __forceinline__ void transpose_4x4_bytes(uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t (&t)[4]) {
    const uint32_t lo01 = __byte_perm(a0, a1, 0x5140), hi01 = __byte_perm(a0, a1, 0x7362);
    const uint32_t lo23 = __byte_perm(a2, a3, 0x5140), hi23 = __byte_perm(a2, a3, 0x7362);
    t[0] = __byte_perm(lo01, lo23, 0x5410);
    t[1] = __byte_perm(lo01, lo23, 0x7632);
    t[2] = __byte_perm(hi01, hi23, 0x5410);
    t[3] = __byte_perm(hi01, hi23, 0x7632);
}

// threads per CTA and CTAs per SM: 4 x 256 threads for bf16 input, 3 x 256 for binary32
template <int WIDE> struct TrGeo {
    static constexpr int THREADS = kThreads;
    static constexpr int MIN_CTAS = WIDE == kWideBF16 ? 4 : 3;
};

// One 128 x 128 tile per CTA, 8 or 16 warps, several CTAs resident per SM (the loads in flight live in registers, so
// residency is what hides the memory latency).  A thread converts 4-row x 16-byte blocks (4 x 8 bf16 or 4 x 4
// binary32, all its sixteen or eight 16-byte row loads issued up front), stores the row-major codes from
// registers (whole 128-byte lines per warp store), transposes 4 x 4 code blocks with byte permutes and parks
// the columns in shared memory (word index XOR-swizzled: conflict-free both ways); after the barrier each
// warp writes its share of the transposed rows, 128 contiguous bytes per store.
// rows is a multiple of 4 and cols of the elements per 16 bytes here, and every pointer / pitch allows the
// 16-byte loads and the 4- or 8-byte stores (the launcher checks).
template <int WIDE, int FMT, bool NOSAT>
__global__ void __launch_bounds__(TrGeo<WIDE>::THREADS, TrGeo<WIDE>::MIN_CTAS)
k_quantize_transpose(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ldx, const float* __restrict__ scale_dev,
                     uint8_t* __restrict__ out, int64_t ldo, uint8_t* __restrict__ out_t, int64_t ldt, int tiles_c,
                     uint32_t* amax_bits) {
    __shared__ uint32_t tile_t[kTrTile * 32];                     // [column][row / 4], swizzled
    __shared__ uint32_t red[32];
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    constexpr int EPT = 16 / ESZ;                                 // elements (columns) per thread and row
    constexpr int NB = EPT / 4;                                   // 4 x 4 code blocks per thread and row group
    constexpr int LPR = kTrTile / EPT;                            // lanes per tile row
    constexpr int RG = 32 / LPR;                                  // 4-row groups per warp instruction
    constexpr int WARPS = TrGeo<WIDE>::THREADS / 32;
    constexpr int STEPS = kTrTile / 4 / (WARPS * RG);
    const float scale = *scale_dev;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int h = lane / LPR, q = lane % LPR;
    const int64_t tr = blockIdx.x / tiles_c, tc = blockIdx.x - tr * tiles_c;
    const int64_t r0 = tr * kTrTile, c0 = tc * kTrTile;
    const int64_t c = c0 + EPT * q;
    const bool col_ok = c < cols;
    const uint8_t* xb = reinterpret_cast<const uint8_t*>(x);
    uint32_t m = 0;

    uint4 v[STEPS][4];
#pragma unroll
    for (int s = 0; s < STEPS; ++s) {
        const int64_t r = r0 + 4 * ((s * WARPS + warp) * RG + h);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[s][i] = make_uint4(0u, 0u, 0u, 0u);
            if (col_ok && r + i < rows) v[s][i] = ld_in_v4(xb + ((r + i) * ldx + c) * ESZ);
        }
    }
#pragma unroll
    for (int s = 0; s < STEPS; ++s) {
        const int g = (s * WARPS + warp) * RG + h;                // 4-row group of the tile
        const int64_t r = r0 + 4 * g;
        uint32_t code[NB][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            m = fold_abs_max<WIDE>(m, v[s][i]);                  // always folded (free next to the memory traffic)
            uint32_t cw[NB];
            if (WIDE == kWideBF16) {
                const uint2 c2 = quantize_item_bf16<FMT, NOSAT>(v[s][i], scale);
                cw[0] = c2.x; cw[NB - 1] = c2.y;
            } else {
                cw[0] = quantize_item_f32<FMT, NOSAT>(v[s][i], scale);
            }
#pragma unroll
            for (int b = 0; b < NB; ++b) code[b][i] = cw[b];
            if (out && col_ok && r + i < rows) {
                uint8_t* p = out + (r + i) * ldo + c;
                if (NB == 2) st_out(reinterpret_cast<uint2*>(p), make_uint2(cw[0], cw[NB - 1]));
                else         st_out(reinterpret_cast<uint32_t*>(p), cw[0]);
            }
        }
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            uint32_t t[4];
            transpose_4x4_bytes(code[b][0], code[b][1], code[b][2], code[b][3], t);
#pragma unroll
            for (int j = 0; j < 4; ++j) tile_t[(EPT * q + 4 * b + j) * 32 + (g ^ (RG * q))] = t[j];
        }
    }
    __syncthreads();
    const int64_t rt = r0 + 4 * lane;                             // first of the four source rows this lane stores
#pragma unroll
    for (int k = 0; k < kTrTile / WARPS; ++k) {
        const int ct = warp * (kTrTile / WARPS) + k;              // column of the tile = row of the transposed output
        const uint32_t w = tile_t[ct * 32 + (lane ^ (RG * (ct / EPT)))];
        if (c0 + ct < cols && rt < rows) st_out(reinterpret_cast<uint32_t*>(out_t + (c0 + ct) * ldt + rt), w);
    }
    if (amax_bits) block_atomic_max_bits(finish_abs_max<WIDE>(m), red, amax_bits);
}

// Any shape, pitch and alignment: one element per thread (the transposed stores are not coalesced).
template <int WIDE, int FMT, bool NOSAT>
__global__ void __launch_bounds__(kThreads)
k_quantize_transpose_elementwise(const void* __restrict__ x, int64_t rows, int64_t cols, int64_t ldx, const float* __restrict__ scale_dev,
                                 uint8_t* __restrict__ out, int64_t ldo, uint8_t* __restrict__ out_t, int64_t ldt, uint32_t* amax_bits) {
    __shared__ uint32_t red[32];
    const float scale = *scale_dev;
    uint32_t m = 0;
    const int64_t n = rows * cols;
    for (int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x; i < n; i += (int64_t)gridDim.x * kThreads) {
        const int64_t r = i / cols, c = i - r * cols;
        const size_t at = (size_t)(r * ldx + c);
        m = max(m, scalar_abs_bits<WIDE>(x, at));
        const float xf = scalar_load<WIDE>(x, at);
        const uint8_t code = (uint8_t)encode_scaled<FMT, NOSAT>(xf * scale, __float_as_uint(xf));
        if (out) out[r * ldo + c] = code;
        out_t[c * ldt + r] = code;
    }
    if (amax_bits) block_atomic_max_bits(canonical_nan_bits(m), red, amax_bits);
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Grid of a streaming kernel: one block per `chunks_per_block` chunks, handed out by the hardware scheduler in
// order as blocks retire.  Short-lived blocks balance the load between SMs that see different memory bandwidth: a
// persistent grid with an equal share per block ends with a tail and measured 4 % (amax) to 12-16 % (dequantize, the
// simulated round trip) slower on 2^28 bf16 elements.  Kernels without a reduction take one chunk per block
// (8-16 KB of input); kernels that end in a block reduction and an atomic take 32 KB of input per block.
static int stream_grid(size_t work_chunks, int chunks_per_block) {
    size_t g = (work_chunks + (size_t)chunks_per_block - 1) / (size_t)chunks_per_block;
    if (g > ((size_t)1 << 30)) g = (size_t)1 << 30;
    if (g < 1) g = 1;
    return (int)g;
}

// Co-resident grid of the cooperative one-launch kernel: SMs x occupancy at most, no more than there is work.
template <typename Kernel>
static int resident_grid(Kernel kernel, size_t work_chunks) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm < 1) per_sm = 1;
    size_t g = (size_t)sm_count() * (size_t)per_sm;
    if (g > work_chunks) g = work_chunks;
    if (g < 1) g = 1;
    return (int)g;
}

static size_t chunks_of(size_t n, int epi, int unroll) {
    const size_t items = n / (size_t)epi;
    const size_t per_chunk = (size_t)kThreads * (size_t)unroll;
    return (items + per_chunk - 1) / per_chunk;
}

// chunks per block of the kernels that end in a reduction: 32 KB of input per block in both cases
constexpr int kAmaxChunksPerBlock = 1, kQuantAmaxChunksPerBlock = 2;
// independent 16-byte loads in flight per thread
constexpr int kAmaxUnroll = 8;
constexpr int kQuantUnrollBF16 = 4;
constexpr int kQuantUnrollF32 = 8;
constexpr int kDequantUnroll = 4;
constexpr int kFakeUnroll = 2;

template <int WIDE>
static fp8_status launch_amax(const void* x, size_t n, uint32_t* bits, cudaStream_t st) {
    if (aligned16(x)) {
        constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
        const bool small = n * (WIDE == kWideBF16 ? 2 : 4) <= ((size_t)64 << 20);     // half-size chunks, as in launch_quantize
        const cudaError_t e = small
            ? launch_programmatic(k_amax<WIDE, kAmaxUnroll / 2>, dim3(stream_grid(chunks_of(n, EPI, kAmaxUnroll / 2), kAmaxChunksPerBlock)), dim3(kThreads), st, x, n, bits)
            : launch_programmatic(k_amax<WIDE, kAmaxUnroll>, dim3(stream_grid(chunks_of(n, EPI, kAmaxUnroll), kAmaxChunksPerBlock)), dim3(kThreads), st, x, n, bits);
        if (e != cudaSuccess) return FP8_ERR_CUDA;
    } else {
        auto k = k_amax_elementwise<WIDE>;
        const int grid = stream_grid((n + kThreads - 1) / kThreads, 16);
        k<<<grid, kThreads, 0, st>>>(x, n, bits);
    }
    count_launches(1);
    return launch_status();
}

template <int WIDE, int FMT, bool NOSAT, bool WITH_AMAX, int UNROLL>
static cudaError_t launch_quantize_vector(const void* x, size_t n, const float* scale, uint8_t* out, uint32_t* bits, cudaStream_t st, int reverse) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    auto k = k_quantize<WIDE, FMT, NOSAT, WITH_AMAX, UNROLL>;
    int grid = stream_grid(chunks_of(n, EPI, UNROLL), WITH_AMAX ? kQuantAmaxChunksPerBlock : 1);
    if (WITH_AMAX) {                                              // a small tensor still wants about fourteen blocks per SM
        const size_t chunks = chunks_of(n, EPI, UNROLL), floor_blocks = (size_t)14 * (size_t)sm_count();
        const size_t low = chunks < floor_blocks ? chunks : floor_blocks;
        if ((size_t)grid < low) grid = (int)low;
    }
    return launch_programmatic(k, dim3(grid), dim3(kThreads), st, x, n, scale, out, bits, reverse);
}

template <int WIDE, int FMT, bool NOSAT, bool WITH_AMAX>
static fp8_status launch_quantize(const void* x, size_t n, const float* scale, uint8_t* out, uint32_t* bits, cudaStream_t st,
                                  int reverse = 0) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    constexpr int UNROLL = WIDE == kWideBF16 ? kQuantUnrollBF16 : kQuantUnrollF32;
    // the vector path stores EPI codes per item: out must be EPI-byte aligned, x 16-byte aligned
    if (aligned16(x) && (reinterpret_cast<uintptr_t>(out) & (EPI - 1)) == 0) {
        // With the input amax folded in, a tensor of at most 64 MB runs half-size chunks (a launch of a few microseconds
        // is mostly ramp and tail: 2^24 bf16 elements 10.6 -> 10.1 us, 2^20 2.8 -> 2.4 us on a ring of distinct tensors;
        // the same chunks cost 3.5 % at 2^28)
        const bool small = WITH_AMAX && n * ESZ <= ((size_t)64 << 20);
        const cudaError_t e = small ? launch_quantize_vector<WIDE, FMT, NOSAT, WITH_AMAX, UNROLL / 2>(x, n, scale, out, bits, st, reverse)
                                    : launch_quantize_vector<WIDE, FMT, NOSAT, WITH_AMAX, UNROLL>(x, n, scale, out, bits, st, reverse);
        if (e != cudaSuccess) return FP8_ERR_CUDA;
    } else {
        auto k = k_quantize_elementwise<WIDE, FMT, NOSAT, WITH_AMAX>;
        const int grid = stream_grid((n + kThreads - 1) / kThreads, 16);
        k<<<grid, kThreads, 0, st>>>(x, n, scale, out, bits);
    }
    count_launches(1);
    return launch_status();
}

template <int WIDE, int FMT>
static fp8_status dispatch_quantize(const void* x, size_t n, bool nosat, const float* scale, uint8_t* out, uint32_t* bits, cudaStream_t st,
                                    int reverse = 0) {
    if (nosat) return bits ? launch_quantize<WIDE, FMT, true, true>(x, n, scale, out, bits, st, reverse)
                           : launch_quantize<WIDE, FMT, true, false>(x, n, scale, out, bits, st, reverse);
    return bits ? launch_quantize<WIDE, FMT, false, true>(x, n, scale, out, bits, st, reverse)
                : launch_quantize<WIDE, FMT, false, false>(x, n, scale, out, bits, st, reverse);
}

// amax -> scale -> quantize of one tensor as the three streaming kernels back to back (identical results to the
// one-launch kernel); the quantize pass walks the tensor from its end, where the amax pass has just been.
static fp8_status quantize_current_chain(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o, uint8_t* out,
                                         float* amax, float* scale, float* scale_inv, cudaStream_t st) {
    fp8_status s = fp8_amax(x, t, n, amax, st);
    if (s == FP8_OK) s = fp8_scale_from_amax(amax, f, scale, scale_inv, st);
    if (s != FP8_OK || n == 0) return s;
    const bool nosat = o == FP8_NOSAT;
    if (t == FP8_F32)
        return f == FP8_E4M3 ? dispatch_quantize<kWideF32, kE4M3>(x, n, nosat, scale, out, nullptr, st, 1)
                             : dispatch_quantize<kWideF32, kE5M2>(x, n, nosat, scale, out, nullptr, st, 1);
    return f == FP8_E4M3 ? dispatch_quantize<kWideBF16, kE4M3>(x, n, nosat, scale, out, nullptr, st, 1)
                         : dispatch_quantize<kWideBF16, kE5M2>(x, n, nosat, scale, out, nullptr, st, 1);
}

template <int FMT, int WIDE>
static fp8_status launch_dequantize(const uint8_t* c, size_t n, const float* si, void* out, cudaStream_t st) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    if (aligned16(out) && (reinterpret_cast<uintptr_t>(c) & (EPI - 1)) == 0) {
        auto k = k_dequantize<FMT, WIDE, kDequantUnroll>;
        const int grid = stream_grid(chunks_of(n, EPI, kDequantUnroll), 1);
        if (launch_programmatic(k, dim3(grid), dim3(kThreads), st, c, n, si, out) != cudaSuccess) return FP8_ERR_CUDA;
    } else {
        auto k = k_dequantize_elementwise<FMT, WIDE>;
        const int grid = stream_grid((n + kThreads - 1) / kThreads, 16);
        k<<<grid, kThreads, 0, st>>>(c, n, si, out);
    }
    count_launches(1);
    return launch_status();
}

// The start value of an amax: a one-thread kernel rather than a memset node, so that the kernel behind it can be
// scheduled while this one still waits for the stream's earlier work.
static fp8_status zero_word(void* p, cudaStream_t st) {
    if (launch_programmatic(k_zero_word, dim3(1), dim3(1), st, reinterpret_cast<uint32_t*>(p)) != cudaSuccess) return FP8_ERR_CUDA;
    count_launches(1);
    return FP8_OK;
}

template <int WIDE, int FMT, bool NOSAT>
static fp8_status launch_current(const void* x, size_t n, float fmax, uint8_t* out, float* amax, float* scale, float* scale_inv,
                                 unsigned int* ws, cudaStream_t st) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int UNROLL = 4;
    auto k = k_quantize_current<WIDE, FMT, NOSAT, UNROLL>;
    size_t chunks = chunks_of(n, EPI, UNROLL);
    if (chunks < 1) chunks = 1;
    const int grid = resident_grid(k, chunks);
    unsigned int arrivals = (unsigned int)grid;
    long long wait_limit = kGridWaitLimitCycles;
    void* args[] = {(void*)&x, (void*)&n, (void*)&fmax, (void*)&out, (void*)&amax, (void*)&scale, (void*)&scale_inv, (void*)&ws,
                    (void*)&arrivals, (void*)&wait_limit};
    if (cudaLaunchCooperativeKernel((const void*)k, dim3(grid), dim3(kThreads), args, 0, st) != cudaSuccess) {
        (void)cudaGetLastError();                                  // e.g. the device cannot hold the whole grid right now
        return FP8_ERR_UNSUPPORTED;                                // the caller falls back to the three separate kernels
    }
    count_launches(1);
    return launch_status();
}

// Shared memory one CTA may use for its slice (the rest of the 227 KB is the kernel's static arrays and slack).
constexpr size_t kResidentSliceBytes = 224 * 1024;

template <int WIDE, int FMT, bool NOSAT>
static fp8_status launch_current_resident(const void* x, size_t n, float fmax, uint8_t* out, float* amax, float* scale, float* scale_inv,
                                          unsigned int* ws, cudaStream_t st) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    auto k = k_quantize_current_resident<WIDE, FMT, NOSAT>;
    static std::mutex mu;
    static bool ready[64] = {false};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FP8_ERR_CUDA;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!ready[dev]) {
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kResidentSliceBytes) != cudaSuccess) return FP8_ERR_CUDA;
            ready[dev] = true;
        }
    }
    size_t n_items = n / EPI;
    const int sms = sm_count();
    // whole items per CTA, a multiple of the block size so that pass 1 runs its unrolled loop; no more CTAs than needed
    size_t items_per_cta = (n_items + (size_t)sms - 1) / (size_t)sms;
    items_per_cta = (items_per_cta + kResidentThreads - 1) / kResidentThreads * kResidentThreads;
    int grid = (int)((n_items + items_per_cta - 1) / items_per_cta);
    if (grid < 1) grid = 1;
    size_t smem = items_per_cta * 16;
    unsigned int arrivals = (unsigned int)grid;
    long long wait_limit = kGridWaitLimitCycles;
    void* args[] = {(void*)&x, (void*)&n_items, (void*)&items_per_cta, (void*)&fmax, (void*)&out, (void*)&amax, (void*)&scale, (void*)&scale_inv,
                    (void*)&ws, (void*)&arrivals, (void*)&wait_limit};
    if (cudaLaunchCooperativeKernel((const void*)k, dim3(grid), dim3(kResidentThreads), args, smem, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return FP8_ERR_UNSUPPORTED;
    }
    count_launches(1);
    return launch_status();
}

// The vector path needs x 16-byte aligned and out aligned to the codes one item produces; other
// alignments take the three separate calls (identical results).
fp8_status launch_quantize_current(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o, uint8_t* out,
                                   float* amax, float* scale, float* scale_inv, unsigned int* ws, cudaStream_t st) {
    const int epi = t == FP8_BF16 ? 8 : 4;
    const size_t bytes = n * (t == FP8_BF16 ? 2 : 4);
    if (n == 0 || !aligned16(x) || (reinterpret_cast<uintptr_t>(out) & (epi - 1)) != 0 || bytes >= kCurrentChainFromBytes)
        return quantize_current_chain(x, t, n, f, o, out, amax, scale, scale_inv, st);
    const float fmax = f == FP8_E4M3 ? 448.0f : 57344.0f;
    const bool nosat = o == FP8_NOSAT;
    fp8_status s;
    // a tensor of whole 16-byte items that fits the shared memory of all SMs: read it from global memory once
    const size_t per_cta = ((n / epi + (size_t)sm_count() - 1) / (size_t)sm_count() + kResidentThreads - 1) / kResidentThreads * kResidentThreads;
    if (n % epi == 0 && per_cta * 16 <= kResidentSliceBytes) {
        if (t == FP8_F32) {
            if (f == FP8_E4M3) s = nosat ? launch_current_resident<kWideF32, kE4M3, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                         : launch_current_resident<kWideF32, kE4M3, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
            else               s = nosat ? launch_current_resident<kWideF32, kE5M2, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                         : launch_current_resident<kWideF32, kE5M2, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
        } else {
            if (f == FP8_E4M3) s = nosat ? launch_current_resident<kWideBF16, kE4M3, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                         : launch_current_resident<kWideBF16, kE4M3, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
            else               s = nosat ? launch_current_resident<kWideBF16, kE5M2, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                         : launch_current_resident<kWideBF16, kE5M2, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
        }
        if (s != FP8_ERR_UNSUPPORTED) return s;                   // refused (e.g. not all CTAs can be resident): the general kernel below
    }
    if (t == FP8_F32) {
        if (f == FP8_E4M3) s = nosat ? launch_current<kWideF32, kE4M3, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                     : launch_current<kWideF32, kE4M3, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
        else               s = nosat ? launch_current<kWideF32, kE5M2, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                     : launch_current<kWideF32, kE5M2, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
    } else {
        if (f == FP8_E4M3) s = nosat ? launch_current<kWideBF16, kE4M3, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                     : launch_current<kWideBF16, kE4M3, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
        else               s = nosat ? launch_current<kWideBF16, kE5M2, true>(x, n, fmax, out, amax, scale, scale_inv, ws, st)
                                     : launch_current<kWideBF16, kE5M2, false>(x, n, fmax, out, amax, scale, scale_inv, ws, st);
    }
    if (s == FP8_ERR_UNSUPPORTED)                                  // cooperative launch refused: same results, three kernels
        s = quantize_current_chain(x, t, n, f, o, out, amax, scale, scale_inv, st);
    return s;
}

template <int WIDE, int FMT, bool NOSAT>
static fp8_status launch_fake(const void* x, size_t n, const float* scale, const float* si, void* out, cudaStream_t st) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int UNROLL = kFakeUnroll;
    if (aligned16(x) && aligned16(out)) {
        auto k = k_fake_quantize<WIDE, FMT, NOSAT, UNROLL>;
        const int grid = stream_grid(chunks_of(n, EPI, UNROLL), 1);
        if (launch_programmatic(k, dim3(grid), dim3(kThreads), st, x, n, scale, si, out) != cudaSuccess) return FP8_ERR_CUDA;
    } else {
        auto k = k_fake_quantize_elementwise<WIDE, FMT, NOSAT>;
        const int grid = stream_grid((n + kThreads - 1) / kThreads, 16);
        k<<<grid, kThreads, 0, st>>>(x, n, scale, si, out);
    }
    count_launches(1);
    return launch_status();
}

static int grid_for(int64_t work_items) {
    int64_t g = (work_items + kThreads - 1) / kThreads;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (g > cap) g = cap;
    if (g < 1) g = 1;
    return (int)g;
}

// One warp per unit of work, every unit its own short-lived warp: the hardware scheduler hands the blocks out in index order
// and evens out what an equal static share per resident block cannot (see the flat kernels).
static int grid_one_warp_per_unit(int64_t units) {
    int64_t g = (units * 32 + kThreads - 1) / kThreads;
    if (g > 0x7FFFFFFF) g = 0x7FFFFFFF;                  // the kernels stride over what is left
    if (g < 1) g = 1;
    return (int)g;
}

// segments per row of the row kernels: 32 lanes x kRowsUnroll items each, at least one
static int64_t row_segments(int64_t n_items) {
    const int64_t per = 32 * kRowsUnroll;
    const int64_t segs = (n_items + per - 1) / per;
    return segs < 1 ? 1 : segs;
}

// rows per slab of the column kernels: about `blocks_per_sm` blocks per SM in all, but at least `min_rows` rows
static int64_t slab_rows(int64_t rows, int64_t col_blocks, int64_t min_rows = kColsMinRows, int64_t blocks_per_sm = 16) {
    const int64_t want_blocks = (int64_t)sm_count() * blocks_per_sm;
    int64_t slabs = (want_blocks + col_blocks - 1) / col_blocks;
    if (slabs < 1) slabs = 1;
    int64_t per = (rows + slabs - 1) / slabs;
    per = (per + 15) / 16 * 16;
    if (per < min_rows) per = min_rows;                  // short slabs are all launch, tail and (amax) atomics
    while ((rows + per - 1) / per > 65535) per *= 2;
    return per;
}

template <int WIDE>
static fp8_status launch_amax_channels(const void* x, int64_t rows, int64_t cols, int64_t ld, int axis, uint32_t* bits, cudaStream_t st) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    const int64_t channels = axis == 0 ? cols : rows;
    const bool vec = aligned16(x) && ((ld * ESZ) & 15) == 0;
    if (axis == 1 && vec) {
        // spans per row: enough units for about four warps' worth per resident warp, no span shorter than one unrolled pass
        const int64_t n_items = cols / EPI, pass = 32 * kRowsAmaxUnroll;
        const int64_t want_units = (int64_t)sm_count() * 8 * (kThreads / 32) * 4;
        int64_t segs = (want_units + rows - 1) / rows;
        const int64_t max_segs = (n_items + pass - 1) / pass;
        if (segs > max_segs) segs = max_segs;
        if (segs < 1) segs = 1;
        const int64_t span = ((n_items + segs - 1) / segs + pass - 1) / pass * pass;
        segs = span > 0 ? (n_items + span - 1) / span : 1;
        if (segs < 1) segs = 1;
        if (segs > 1) {                                             // several warps share a row: atomicMax onto zeros
            if (cudaMemsetAsync(bits, 0, (size_t)channels * 4, st) != cudaSuccess) return FP8_ERR_CUDA;
            count_launches(1);
        }
        k_amax_rows<WIDE><<<grid_one_warp_per_unit(rows * segs), kThreads, 0, st>>>(x, rows, cols, ld, segs, span, bits);
        count_launches(1);
        return launch_status();
    }
    if (cudaMemsetAsync(bits, 0, (size_t)channels * 4, st) != cudaSuccess) return FP8_ERR_CUDA;
    count_launches(1);
    if (axis == 0 && vec && cols % EPI == 0) {
        const int64_t col_blocks = (cols / EPI + kColsTx - 1) / kColsTx;
        const int64_t per = slab_rows(rows, col_blocks);
        dim3 grid((unsigned)col_blocks, (unsigned)((rows + per - 1) / per));
        k_amax_cols<WIDE><<<grid, dim3(kColsTx, kColsTy), 0, st>>>(x, rows, cols, ld, per, bits);
    } else if (axis == 0) {
        k_amax_channels_elementwise<WIDE, 0><<<grid_for(rows * cols), kThreads, 0, st>>>(x, rows, cols, ld, bits);
    } else {
        k_amax_channels_elementwise<WIDE, 1><<<grid_for(rows * cols), kThreads, 0, st>>>(x, rows, cols, ld, bits);
    }
    count_launches(1);
    return launch_status();
}

template <int WIDE, int FMT, bool NOSAT>
static fp8_status launch_quantize_channels(const void* x, int64_t rows, int64_t cols, int64_t ld, int axis, const float* scale,
                                           uint8_t* out, int64_t ld_out, cudaStream_t st) {
    constexpr int EPI = WIDE == kWideBF16 ? 8 : 4;
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    const bool vec = aligned16(x) && ((ld * ESZ) & 15) == 0 && (reinterpret_cast<uintptr_t>(out) & (EPI - 1)) == 0 && (ld_out % EPI) == 0;
    if (vec && axis == 1) {
        const int64_t segs = row_segments(cols / EPI);
        k_quantize_rows<WIDE, FMT, NOSAT><<<grid_one_warp_per_unit(rows * segs), kThreads, 0, st>>>(x, rows, cols, ld, segs, scale, out, ld_out);
        count_launches(1);
        return launch_status();
    }
    if (vec && axis == 0 && cols >= EPI) {
        const int64_t full_cols = cols / EPI * EPI;
        const int64_t col_blocks = (full_cols / EPI + kColsTx - 1) / kColsTx;
        // From 256 MB on the conversion runs as many short blocks (64-row slabs, several waves handed out by the hardware
        // scheduler: +3.5 % at 268 MB, +7 % at 1.2 GB); smaller tensors keep 256-row slabs (64-row slabs: -5 % at 134 MB).
        const bool big = (uint64_t)rows * (uint64_t)cols * ESZ >= ((uint64_t)256 << 20);
        const int64_t per = big ? slab_rows(rows, col_blocks, 64, 64) : slab_rows(rows, col_blocks);
        dim3 grid((unsigned)col_blocks, (unsigned)((rows + per - 1) / per));
        k_quantize_cols<WIDE, FMT, NOSAT><<<grid, dim3(kColsTx, kColsTy), 0, st>>>(x, rows, full_cols, ld, per, scale, out, ld_out);
        count_launches(1);
        if (full_cols < cols) {
            k_quantize_channels_elementwise<WIDE, FMT, NOSAT, 0><<<grid_for(rows * (cols - full_cols)), kThreads, 0, st>>>(
                x, rows, cols, ld, full_cols, scale, out, ld_out);
            count_launches(1);
        }
        return launch_status();
    }
    if (axis == 0) k_quantize_channels_elementwise<WIDE, FMT, NOSAT, 0><<<grid_for(rows * cols), kThreads, 0, st>>>(x, rows, cols, ld, 0, scale, out, ld_out);
    else           k_quantize_channels_elementwise<WIDE, FMT, NOSAT, 1><<<grid_for(rows * cols), kThreads, 0, st>>>(x, rows, cols, ld, 0, scale, out, ld_out);
    count_launches(1);
    return launch_status();
}

template <int WIDE, int FMT, bool NOSAT>
static fp8_status launch_quantize_transpose(const void* x, int64_t rows, int64_t cols, int64_t ldx, const float* scale,
                                            uint8_t* out, int64_t ldo, uint8_t* out_t, int64_t ldt, uint32_t* bits, cudaStream_t st) {
    constexpr int ESZ = WIDE == kWideBF16 ? 2 : 4;
    const int64_t tiles_r = (rows + kTrTile - 1) / kTrTile, tiles_c = (cols + kTrTile - 1) / kTrTile;
    constexpr int EPT = 16 / ESZ;                                 // elements per 16-byte load
    const bool fast = (rows & 3) == 0 && (cols % EPT) == 0 && aligned16(x) && (ldx % EPT) == 0 &&
                      (!out || ((reinterpret_cast<uintptr_t>(out) % (EPT)) == 0 && (ldo % EPT) == 0)) &&
                      (reinterpret_cast<uintptr_t>(out_t) & 3) == 0 && (ldt & 3) == 0 && tiles_r * tiles_c <= 0x7FFFFFFF;
    if (fast)
        k_quantize_transpose<WIDE, FMT, NOSAT><<<(unsigned)(tiles_r * tiles_c), TrGeo<WIDE>::THREADS, 0, st>>>(
            x, rows, cols, ldx, scale, out, ldo, out_t, ldt, (int)tiles_c, bits);
    else
        k_quantize_transpose_elementwise<WIDE, FMT, NOSAT><<<grid_for(rows * cols), kThreads, 0, st>>>(
            x, rows, cols, ldx, scale, out, ldo, out_t, ldt, bits);
    count_launches(1);
    return launch_status();
}

template <int WIDE, int FMT>
static fp8_status dispatch_quantize_transpose(const void* x, int64_t rows, int64_t cols, int64_t ldx, bool nosat, const float* scale,
                                              uint8_t* out, int64_t ldo, uint8_t* out_t, int64_t ldt, uint32_t* bits, cudaStream_t st) {
    return nosat ? launch_quantize_transpose<WIDE, FMT, true>(x, rows, cols, ldx, scale, out, ldo, out_t, ldt, bits, st)
                 : launch_quantize_transpose<WIDE, FMT, false>(x, rows, cols, ldx, scale, out, ldo, out_t, ldt, bits, st);
}

}  // namespace fp8b200

using namespace fp8b200;

extern "C" {

fp8_status fp8_amax(const void* x, fp8_wide t, size_t n, float* amax_dev, void* stream) {
    if (!amax_dev || (!x && n)) return FP8_ERR_NULL;
    if (t != FP8_F32 && t != FP8_BF16) return FP8_ERR_ENUM;
    cudaStream_t st = (cudaStream_t)stream;
    fp8_status s = zero_word(amax_dev, st);
    if (s != FP8_OK || n == 0) return s;
    uint32_t* bits = reinterpret_cast<uint32_t*>(amax_dev);
    return t == FP8_F32 ? launch_amax<kWideF32>(x, n, bits, st) : launch_amax<kWideBF16>(x, n, bits, st);
}

fp8_status fp8_scale_from_amax(const float* amax_dev, fp8_format f, float* scale_dev, float* scale_inv_dev, void* stream) {
    if (!amax_dev || !scale_dev || !scale_inv_dev) return FP8_ERR_NULL;
    if (f != FP8_E4M3 && f != FP8_E5M2) return FP8_ERR_ENUM;
    if (launch_programmatic(k_scale_from_amax, dim3(1), dim3(1), (cudaStream_t)stream, amax_dev, f == FP8_E4M3 ? 448.0f : 57344.0f,
                            scale_dev, scale_inv_dev) != cudaSuccess)
        return FP8_ERR_CUDA;
    count_launches(1);
    return launch_status();
}

fp8_status fp8_quantize(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o,
                        const float* scale_dev, uint8_t* out, float* amax_dev, void* stream) {
    if (!scale_dev || ((!x || !out) && n)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (f != FP8_E4M3 && f != FP8_E5M2) || (o != FP8_SATURATE && o != FP8_NOSAT))
        return FP8_ERR_ENUM;
    cudaStream_t st = (cudaStream_t)stream;
    if (amax_dev) {
        fp8_status s = zero_word(amax_dev, st);
        if (s != FP8_OK) return s;
    }
    if (n == 0) return FP8_OK;
    uint32_t* bits = reinterpret_cast<uint32_t*>(amax_dev);
    const bool nosat = o == FP8_NOSAT;
    if (t == FP8_F32)
        return f == FP8_E4M3 ? dispatch_quantize<kWideF32, kE4M3>(x, n, nosat, scale_dev, out, bits, st)
                             : dispatch_quantize<kWideF32, kE5M2>(x, n, nosat, scale_dev, out, bits, st);
    return f == FP8_E4M3 ? dispatch_quantize<kWideBF16, kE4M3>(x, n, nosat, scale_dev, out, bits, st)
                         : dispatch_quantize<kWideBF16, kE5M2>(x, n, nosat, scale_dev, out, bits, st);
}

fp8_status fp8_quantize_current(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o, uint8_t* out,
                                float* amax_dev, float* scale_dev, float* scale_inv_dev, void* workspace, void* stream) {
    if (!amax_dev || !scale_dev || !scale_inv_dev || !workspace || ((!x || !out) && n)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (f != FP8_E4M3 && f != FP8_E5M2) || (o != FP8_SATURATE && o != FP8_NOSAT))
        return FP8_ERR_ENUM;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return FP8_ERR_ALIGN;
    return fp8b200::launch_quantize_current(x, t, n, f, o, out, amax_dev, scale_dev, scale_inv_dev,
                                            reinterpret_cast<unsigned int*>(workspace), (cudaStream_t)stream);
}

size_t fp8_quantize_current_workspace_bytes(void) { return 16; }

// ---- fp8_quantize_current_static: the same kernel, its scratch words in library-owned static memory ----
//
// g_static_scratch is what the kernel uses as its three control words.  In host code this name is only
// a stand-in for the device object: its device address is obtained once per device with
// cudaGetSymbolAddress (that device being current) and that address is what the kernel receives.
constexpr size_t kStaticScratchBytes = 256;
static __device__ __align__(256) unsigned int g_static_scratch[kStaticScratchBytes / sizeof(unsigned int)];

static fp8_status static_scratch_address(unsigned int** out) {
    static std::mutex mu;
    static unsigned int* addr[64] = {nullptr};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return FP8_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (addr[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return FP8_ERR_CUDA;
        addr[dev] = reinterpret_cast<unsigned int*>(p);
    }
    *out = addr[dev];
    return FP8_OK;
}

fp8_status fp8_quantize_current_static(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o, uint8_t* out,
                                       float* amax_dev, float* scale_dev, float* scale_inv_dev, void* stream) {
    if (!amax_dev || !scale_dev || !scale_inv_dev || ((!x || !out) && n)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (f != FP8_E4M3 && f != FP8_E5M2) || (o != FP8_SATURATE && o != FP8_NOSAT))
        return FP8_ERR_ENUM;
    if (n > FP8_STATIC_MAX_ELEMENTS) return FP8_ERR_UNSUPPORTED;
    unsigned int* scratch = nullptr;
    fp8_status s = static_scratch_address(&scratch);
    if (s != FP8_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the last call left (zeros, unless that call gave up on its barrier): start clean
    if (cudaMemsetAsync(scratch, 0, 16, st) != cudaSuccess) return FP8_ERR_CUDA;
    count_launches(1);
    return fp8b200::launch_quantize_current(x, t, n, f, o, out, amax_dev, scale_dev, scale_inv_dev, scratch, st);
}


void fp8_cast_read_clear_latch(unsigned int out2[2]) {
    out2[0] = out2[1] = 0u;
    if (cudaMemcpyFromSymbol(out2, fp8b200::g_cast_latch, 2 * sizeof(unsigned int)) != cudaSuccess) return;
    if (out2[0] != 0u) {
        const unsigned int zero[2] = {0u, 0u};
        cudaMemcpyToSymbol(fp8b200::g_cast_latch, zero, sizeof(zero));
    }
}

fp8_status fp8_amax_channels(const void* x, fp8_wide t, int64_t rows, int64_t cols, int64_t ld, int axis,
                             float* amax_vec_dev, void* stream) {
    if (!amax_vec_dev || (!x && rows > 0 && cols > 0)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (axis != 0 && axis != 1)) return FP8_ERR_ENUM;
    if (rows < 0 || cols < 0 || ld < cols) return FP8_ERR_SHAPE;
    const int64_t channels = axis == 0 ? cols : rows;
    if (channels == 0) return FP8_OK;
    cudaStream_t st = (cudaStream_t)stream;
    uint32_t* bits = reinterpret_cast<uint32_t*>(amax_vec_dev);
    if (rows == 0 || cols == 0) {                                   // empty channels: amax 0
        if (cudaMemsetAsync(bits, 0, (size_t)channels * 4, st) != cudaSuccess) return FP8_ERR_CUDA;
        count_launches(1);
        return FP8_OK;
    }
    return t == FP8_F32 ? launch_amax_channels<kWideF32>(x, rows, cols, ld, axis, bits, st)
                        : launch_amax_channels<kWideBF16>(x, rows, cols, ld, axis, bits, st);
}

fp8_status fp8_scales_from_amax(const float* amax_vec_dev, int64_t count, fp8_format f, int pow2,
                                float* scale_vec_dev, float* scale_inv_vec_dev, void* stream) {
    if (count < 0) return FP8_ERR_SHAPE;
    if (count == 0) return FP8_OK;
    if (!amax_vec_dev || !scale_vec_dev || !scale_inv_vec_dev) return FP8_ERR_NULL;
    if (f != FP8_E4M3 && f != FP8_E5M2) return FP8_ERR_ENUM;
    k_scales_from_amax<<<grid_for(count), kThreads, 0, (cudaStream_t)stream>>>(amax_vec_dev, count, f == FP8_E4M3 ? 448.0f : 57344.0f,
                                                                               pow2 ? 1 : 0, scale_vec_dev, scale_inv_vec_dev);
    count_launches(1);
    return launch_status();
}

fp8_status fp8_quantize_channels(const void* x, fp8_wide t, int64_t rows, int64_t cols, int64_t ld, int axis, fp8_format f,
                                 fp8_overflow o, const float* scale_vec_dev, uint8_t* out, int64_t ld_out, void* stream) {
    if (!scale_vec_dev || ((!x || !out) && rows > 0 && cols > 0)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (f != FP8_E4M3 && f != FP8_E5M2) || (o != FP8_SATURATE && o != FP8_NOSAT) ||
        (axis != 0 && axis != 1))
        return FP8_ERR_ENUM;
    if (rows < 0 || cols < 0 || ld < cols || ld_out < cols) return FP8_ERR_SHAPE;
    if (rows == 0 || cols == 0) return FP8_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const bool nosat = o == FP8_NOSAT;
    if (t == FP8_F32) {
        if (f == FP8_E4M3) return nosat ? launch_quantize_channels<kWideF32, kE4M3, true>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st)
                                        : launch_quantize_channels<kWideF32, kE4M3, false>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st);
        return nosat ? launch_quantize_channels<kWideF32, kE5M2, true>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st)
                     : launch_quantize_channels<kWideF32, kE5M2, false>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st);
    }
    if (f == FP8_E4M3) return nosat ? launch_quantize_channels<kWideBF16, kE4M3, true>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st)
                                    : launch_quantize_channels<kWideBF16, kE4M3, false>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st);
    return nosat ? launch_quantize_channels<kWideBF16, kE5M2, true>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st)
                 : launch_quantize_channels<kWideBF16, kE5M2, false>(x, rows, cols, ld, axis, scale_vec_dev, out, ld_out, st);
}

fp8_status fp8_quantize_transpose(const void* x, fp8_wide t, int64_t rows, int64_t cols, int64_t ldx, fp8_format f, fp8_overflow o,
                                  const float* scale_dev, uint8_t* out, int64_t ldo, uint8_t* out_t, int64_t ldt,
                                  float* amax_dev, void* stream) {
    if (!scale_dev || ((!x || !out_t) && rows > 0 && cols > 0)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (f != FP8_E4M3 && f != FP8_E5M2) || (o != FP8_SATURATE && o != FP8_NOSAT))
        return FP8_ERR_ENUM;
    if (rows < 0 || cols < 0 || ldx < cols || (out && ldo < cols) || ldt < rows) return FP8_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (amax_dev) {
        fp8_status s = zero_word(amax_dev, st);
        if (s != FP8_OK) return s;
    }
    if (rows == 0 || cols == 0) return FP8_OK;
    uint32_t* bits = reinterpret_cast<uint32_t*>(amax_dev);
    const bool nosat = o == FP8_NOSAT;
    if (t == FP8_F32)
        return f == FP8_E4M3 ? dispatch_quantize_transpose<kWideF32, kE4M3>(x, rows, cols, ldx, nosat, scale_dev, out, ldo, out_t, ldt, bits, st)
                             : dispatch_quantize_transpose<kWideF32, kE5M2>(x, rows, cols, ldx, nosat, scale_dev, out, ldo, out_t, ldt, bits, st);
    return f == FP8_E4M3 ? dispatch_quantize_transpose<kWideBF16, kE4M3>(x, rows, cols, ldx, nosat, scale_dev, out, ldo, out_t, ldt, bits, st)
                         : dispatch_quantize_transpose<kWideBF16, kE5M2>(x, rows, cols, ldx, nosat, scale_dev, out, ldo, out_t, ldt, bits, st);
}

fp8_status fp8_fake_quantize(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o,
                             const float* scale_dev, const float* scale_inv_dev, void* out, void* stream) {
    if (!scale_dev || !scale_inv_dev || ((!x || !out) && n)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (f != FP8_E4M3 && f != FP8_E5M2) || (o != FP8_SATURATE && o != FP8_NOSAT))
        return FP8_ERR_ENUM;
    if (n == 0) return FP8_OK;
    cudaStream_t st = (cudaStream_t)stream;
    const bool nosat = o == FP8_NOSAT;
    if (t == FP8_F32) {
        if (f == FP8_E4M3) return nosat ? launch_fake<kWideF32, kE4M3, true>(x, n, scale_dev, scale_inv_dev, out, st)
                                        : launch_fake<kWideF32, kE4M3, false>(x, n, scale_dev, scale_inv_dev, out, st);
        return nosat ? launch_fake<kWideF32, kE5M2, true>(x, n, scale_dev, scale_inv_dev, out, st)
                     : launch_fake<kWideF32, kE5M2, false>(x, n, scale_dev, scale_inv_dev, out, st);
    }
    if (f == FP8_E4M3) return nosat ? launch_fake<kWideBF16, kE4M3, true>(x, n, scale_dev, scale_inv_dev, out, st)
                                    : launch_fake<kWideBF16, kE4M3, false>(x, n, scale_dev, scale_inv_dev, out, st);
    return nosat ? launch_fake<kWideBF16, kE5M2, true>(x, n, scale_dev, scale_inv_dev, out, st)
                 : launch_fake<kWideBF16, kE5M2, false>(x, n, scale_dev, scale_inv_dev, out, st);
}

fp8_status fp8_scale_pow2_from_amax(const float* amax_dev, fp8_format f, float* scale_dev, float* scale_inv_dev, void* stream) {
    if (!amax_dev || !scale_dev || !scale_inv_dev) return FP8_ERR_NULL;
    if (f != FP8_E4M3 && f != FP8_E5M2) return FP8_ERR_ENUM;
    k_scale_pow2_from_amax<<<1, 1, 0, (cudaStream_t)stream>>>(amax_dev, f == FP8_E4M3 ? 448.0f : 57344.0f, scale_dev, scale_inv_dev);
    count_launches(1);
    return launch_status();
}

fp8_status fp8_dequantize(const uint8_t* c, size_t n, fp8_format f, const float* scale_inv_dev, void* out, fp8_wide t, void* stream) {
    if (!scale_inv_dev || ((!c || !out) && n)) return FP8_ERR_NULL;
    if ((t != FP8_F32 && t != FP8_BF16) || (f != FP8_E4M3 && f != FP8_E5M2)) return FP8_ERR_ENUM;
    if (n == 0) return FP8_OK;
    cudaStream_t st = (cudaStream_t)stream;
    if (t == FP8_F32)
        return f == FP8_E4M3 ? launch_dequantize<kE4M3, kWideF32>(c, n, scale_inv_dev, out, st)
                             : launch_dequantize<kE5M2, kWideF32>(c, n, scale_inv_dev, out, st);
    return f == FP8_E4M3 ? launch_dequantize<kE4M3, kWideBF16>(c, n, scale_inv_dev, out, st)
                         : launch_dequantize<kE5M2, kWideBF16>(c, n, scale_inv_dev, out, st);
}

fp8_status fp8_sm_clock_probe(uint64_t* out_dev, uint32_t duration_us, void* stream) {
    if (!out_dev) return FP8_ERR_NULL;
    if (duration_us == 0 || duration_us > 100000u) return FP8_ERR_UNSUPPORTED;      // at most a tenth of a second
    k_sm_clock_probe<<<1, 32, 0, (cudaStream_t)stream>>>(reinterpret_cast<unsigned long long*>(out_dev), (unsigned long long)duration_us * 1000ull);
    count_launches(1);
    return launch_status();
}

const char* fp8_status_string(fp8_status s) {
    switch (s) {
        case FP8_OK: return "ok";
        case FP8_ERR_NULL: return "null pointer";
        case FP8_ERR_ENUM: return "enum out of range";
        case FP8_ERR_SHAPE: return "bad shape or leading dimension";
        case FP8_ERR_ALIGN: return "operand not 16-byte aligned";
        case FP8_ERR_UNSUPPORTED: return "unsupported size";
        case FP8_ERR_CUDA: return "CUDA error";
        case FP8_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

uint64_t fp8_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"

// Self-test of the bounded grid barrier: the one-launch kernel on an empty tensor, its barrier told to wait for one
// CTA more than the grid has.  Every CTA gives up after `limit_cycles`, latches the time-out and returns without
// writing anything; the last one out leaves the control words zeroed, as always.  Uses the static control words.
fp8_status fp8b200::launch_grid_barrier_self_test(long long limit_cycles, cudaStream_t st) {
    unsigned int* scratch = nullptr;
    fp8_status s = static_scratch_address(&scratch);
    if (s != FP8_OK) return s;
    if (cudaMemsetAsync(scratch, 0, 16, st) != cudaSuccess) return FP8_ERR_CUDA;
    count_launches(1);
    auto k = k_quantize_current<kWideBF16, kE4M3, false, 4>;
    const void* x = nullptr;
    size_t n = 0;
    float fmax = 448.0f;
    uint8_t* out = nullptr;
    float* none = nullptr;
    const int grid = 8;
    unsigned int arrivals = (unsigned int)grid + 1u;
    void* args[] = {(void*)&x, (void*)&n, (void*)&fmax, (void*)&out, (void*)&none, (void*)&none, (void*)&none, (void*)&scratch,
                    (void*)&arrivals, (void*)&limit_cycles};
    if (cudaLaunchCooperativeKernel((const void*)k, dim3(grid), dim3(kThreads), args, 0, st) != cudaSuccess) {
        (void)cudaGetLastError();
        return FP8_ERR_CUDA;
    }
    count_launches(1);
    return launch_status();
}
