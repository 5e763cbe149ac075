// FP8 GEMM on the 5th-generation tensor cores (sm_100a): Sections 2 and 4.1 of
// the paper: dot products of FP8 inputs accumulated in binary32, unscaled once
// per dot product, written in a wider type.
//
// One persistent CTA per SM.  CG (CTA group) = 2: the two CTAs of a cluster
// work on one 256 x 256 output tile, each holding 128 rows of A, half of the B
// tile and its own 128 x 256 accumulator; the leader CTA issues
// tcgen05.mma.cta_group::2 (M256 N256 K32) for both.  That halves the B bytes
// each SM stages and reads per flop.  CG = 1 (128 x 256 tiles, one CTA) serves
// problems with at most 128 rows.
//   warp 0       TMA producer: cp.async.bulk.tensor loads of this CTA's A rows
//                and B rows into a 128B-swizzled smem ring; completion is
//                signalled on the leader CTA's "full" barrier
//   warp 1       TMEM allocation (both CTAs) and, in the leader, one lane issuing
//                the MMAs into one of two 256-column TMEM accumulators;
//                tcgen05.commit releases the smem stage in both CTAs / publishes
//                the finished accumulator to both CTAs' epilogues
//   warps 2..5   (2..9 for short K, 4..11 for split accumulation)
//                epilogue: tcgen05.ld of the accumulator (each warp owns its 32
//                TMEM lanes), multiply by sa_inv*sb_inv, round to bf16 / keep
//                fp32, amax of the stored values, swizzled staging in shared
//                memory and TMA tensor stores (edges clipped by the TMA unit).
//                The epilogue of tile i overlaps the main loop of tile i+1.
// Operands may be K-major or MN-major (forward / dgrad / wgrad layouts); the
// two formats of a mixed E5M2 x E4M3 product are set in the instruction
// descriptor.  Every TMA load has one destination: the shared memory of the CTA that issues it.
// Every mbarrier wait is bounded (about 2 s): on expiry the kernel latches an error code,
// all roles drain, TMEM is freed and the kernel returns.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "codec.cuh"
#include "common.cuh"

namespace fp8b200 {

__device__ unsigned int g_async_latch[2] = {0u, 0u};

namespace gemm {


constexpr int BM = 128;             // tile rows  (= UMMA M, one TMEM lane per row)
constexpr int BN = 256;             // tile cols  (= UMMA N, one TMEM column per col)
constexpr int BK = 128;             // K-block in elements = bytes = one 128B swizzle row
constexpr int UMMA_K = 32;          // K of one tcgen05.mma for 8-bit operands
constexpr int MAX_STAGES = 6;
constexpr int ACC_STAGES = 2;       // 2 x 256 columns = all 512 TMEM columns
constexpr int GROUP_M = 16;         // tile raster: GROUP_M row-tiles share each sweep over N
// Epilogue width: 4 warps with two staging buffers each (long K: the epilogue has slack, fewer resident warps
// leave the MMA-issuing thread undisturbed) or 8 warps (short K: the kernel is bound by its output stream; two
// warps per TMEM lane quarter split the tile's columns and each warp has three buffers, two ring stages' worth).
// Split accumulation also runs 8 warps (one buffer each): its partial sums need 128 registers per thread.
constexpr int SHORT_K_BLOCKS = 8;   // K <= 1024: eight epilogue warps
constexpr int SPLIT_BLOCKS = 16;    // split accumulation: the TMEM accumulator is drained into registers every 2048 of K
constexpr uint32_t A_BYTES = BM * BK;          // 16 KiB: this CTA's 128 rows of A
// per CTA group size: B bytes staged by one CTA, stage size, ring depth (192 KiB of tiles either way)
template <int CG> struct Geo {
    static constexpr uint32_t B_BYTES = (BN / CG) * BK;             // 32 KiB alone, 16 KiB when paired
    static constexpr uint32_t STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = CG == 1 ? 4 : 6;
    static constexpr int TILE_M = BM * CG;
    static constexpr int FG = 2;                                    // K-blocks (stages) consumed per full-barrier wait
};
constexpr uint32_t SMEM_TILES = 4 * (A_BYTES + BN * BK);            // = 6 * (A_BYTES + BN/2 * BK)
constexpr uint32_t EPI_BUF_BYTES = 4096;                            // 32 rows x 128 B, one TMA store box
constexpr uint32_t SMEM_EPI = 8 * EPI_BUF_BYTES;                    // staging buffers of the epilogue warps (4 x 2 or 8 x 1; short K adds two ring stages)
constexpr uint32_t SMEM_BARRIERS = 256;
constexpr uint32_t SMEM_BYTES = SMEM_TILES + SMEM_EPI + SMEM_BARRIERS + 1024;   // + slack to align the ring to 1024 B
constexpr uint32_t TMEM_COLS = 512;

constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;   // about 2 s of SM clocks per wait

// codes written to the error latch
enum : uint32_t { WAIT_EMPTY = 1, WAIT_FULL = 2, WAIT_ACC_EMPTY = 3, WAIT_ACC_FULL = 4, WAIT_SELF_TEST = 9 };

// ---- PTX wrappers ----------------------------------------------------------

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false after about `limit` SM clocks (checked every 1024 failed polls, so that
// the common short wait never reads a timer), or as soon as another role of this CTA has given up
// (abort flag), having latched `code`.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t code,
                                          long long limit = WAIT_LIMIT_CYCLES) {
    long long t0 = 0;
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spins & 1023u) == 0u) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) {
                *abort_flag = 1u;
                if (atomicCAS(&g_async_latch[0], 0u, code) == 0u) g_async_latch[1] = blockIdx.x;
                return false;
            }
        }
    }
}

// cluster (CTA pair) helpers
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {     // same variable in CTA `rank`
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_cluster(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// TMA load whose completion is counted on a barrier that may live in the peer CTA of the pair
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t cluster_bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(cluster_bar), "l"(policy) : "memory");
}
// commit of a CTA-pair MMA: arrives on the barrier at this offset in both CTAs
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void tc_mma_f8_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy) : "memory");
}
// L2 eviction policies: operand panels are re-read by many CTAs (keep), the output is written once (stream)
__device__ __forceinline__ uint64_t policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// TMA tensor store of one staged box, tracked by the issuing thread's bulk async-group
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3, %4}], [%1], %5;"
                 ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "l"(policy) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void tc_mma_f8(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}

__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor (sm_100 format): start address, leading and
// stride byte offsets in 16-byte units, version 1, 128-byte swizzle.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;          // descriptor version of this architecture
    d |= (uint64_t)2 << 61;          // SWIZZLE_128B
    return d;
}

struct Params {
    int64_t M, N, K;
    int64_t ldd;                    // elements
    void* D;
    const float* sa_inv;
    const float* sb_inv;
    uint32_t* amax_bits;            // may be null
    uint32_t idesc;                 // M field set for the CTA group the kernel was built for
    int tiles_m, tiles_n;           // tiles of (128*CG) x 256
    int a_mn, b_mn;                 // operand stored with its M (resp. N) index contiguous
    int batch;                      // independent problems sharing the scales (strided batch); tiles_m*tiles_n tiles each
    int64_t stride_d;               // elements between consecutive batch members of D
    const float* sb_inv_vec;        // optional: one inverse scale per column of B (per output channel), N entries
    const float* scale_d;           // FP8 output only: scale applied before the conversion
    int nosat;                      // FP8 output only: non-saturating conversion
};

// what the epilogue writes
constexpr int OUT_F32 = 0, OUT_BF16 = 1, OUT_E4M3 = 2, OUT_E5M2 = 3;

// 32 accumulator values (already multiplied by alpha) -> 32 FP8 codes of y = v * scale_d, packed in 8 words.
// Same rules as the cast kernels: hardware convert unless a special value (or, non-saturating, an overflow)
// is present; a NaN code takes the sign of v.
__device__ __forceinline__ float fmax_nan(float a, float b) {      // NaN if either operand is NaN
    float d;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(d) : "f"(a), "f"(b));
    return d;
}

template <int FMT>
__device__ __forceinline__ void encode32(const float (&v)[32], float scale_d, bool nosat, uint32_t (&w)[8]) {
    float y[32];
    float top = 0.0f;                                             // max |y|, NaN if any y is NaN
#pragma unroll
    for (int i = 0; i < 32; ++i) {
        y[i] = v[i] * scale_d;
        top = fmax_nan(top, fabsf(y[i]));
    }
    const bool over = Fmt<FMT>::nosat_limit_inclusive ? top >= Fmt<FMT>::nosat_limit : top > Fmt<FMT>::nosat_limit;
    const bool finite = top <= 3.402823466e38f;                   // false for NaN and for Inf
    if (finite && !(nosat && over)) {
#pragma unroll
        for (int q = 0; q < 8; ++q) w[q] = cvt_quad<FMT>(y[4 * q], y[4 * q + 1], y[4 * q + 2], y[4 * q + 3]);
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint32_t word = 0;
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                const float yy = y[4 * q + b];
                uint32_t code;
                if (yy != yy) code = ((__float_as_uint(v[4 * q + b]) >> 24) & 0x80u) | 0x7Fu;
                else code = nosat ? encode_scalar<FMT, true>(yy) : encode_scalar<FMT, false>(yy);
                word |= code << (8 * b);
            }
            w[q] = word;
        }
    }
}

struct alignas(8) Barriers {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t acc_full[ACC_STAGES];
    uint64_t acc_empty[ACC_STAGES];
    uint32_t tmem_base;
    uint32_t abort_flag;
};
static_assert(sizeof(Barriers) <= SMEM_BARRIERS, "barrier block too large");

// tile index -> (row-tile, col-tile): GROUP_M row-tiles advance together over N,
// so that the CTAs running at one time share their A and B panels in L2.
__device__ __forceinline__ void tile_coords(int t, int tiles_m, int tiles_n, int& tm, int& tn) {
    const int per_group = GROUP_M * tiles_n;
    const int g = t / per_group;
    const int first_m = g * GROUP_M;
    const int rows = min(GROUP_M, tiles_m - first_m);
    const int r = t - g * per_group;
    tm = first_m + r % rows;
    tn = r / rows;
}

// CG: CTAs per tile (1 or 2).  OUT: what the epilogue writes (fp32, bf16, E4M3 or E5M2 codes).
// Operand layouts (K-major or MN-major) are run-time properties: they only change TMA coordinates and
// shared-memory descriptor constants.
// SPLIT: split accumulation (needs 8 epilogue warps): the tensor core adds each K=32 block into the binary32
// accumulator with truncation, so over a long K same-sign products lose up to (K/32) 2^-23 of their sum; here
// the accumulator is closed every SPLIT_BLOCKS K-blocks and the partial sums are added in registers with
// round-to-nearest, which keeps the error below 1e-5 of sum|a.b| for any data.
// Warp layout.  Warp 0 loads, warp 1 issues the MMAs, the epilogue warps start at EPI_BASE.  Split accumulation keeps 128
// partial sums per epilogue thread and wants two TMEM loads in flight beside them, more registers than a thread of a
// 320-thread block can have (168): its instances run 12 warps in three aligned groups of four, the first group (loader,
// MMA issuer, two idle warps) gives registers up with setmaxnreg and the two epilogue groups take them.
template <bool SPLIT> struct Roles {
    static constexpr int EPI_BASE = SPLIT ? 4 : 2;
    static constexpr int REGS_FRONT = 56, REGS_EPILOGUE = 224;   // 4 x 32 x 56 + 8 x 32 x 224 = 64512 <= 65536
};
template <int CG, int OUT, int EPI_WARPS, bool SPLIT>
__global__ void __launch_bounds__(32 * (Roles<SPLIT>::EPI_BASE + EPI_WARPS), 1)
k_gemm_fp8(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
           const __grid_constant__ CUtensorMap map_d, const Params p) {
    using G = Geo<CG>;
    // Short K (eight epilogue warps, one accumulator per tile): the kernel is bound by its output stream, so
    // two stages of the operand ring are given to the epilogue: three staging buffers per warp, whose TMA
    // stores drain while the warp converts its next boxes.
    constexpr bool SHORT = EPI_WARPS == 8 && !SPLIT;
    constexpr int EPI_BUFS = SHORT ? 3 : 8 / EPI_WARPS;
    constexpr int STAGES = SHORT ? G::STAGES - 2 : G::STAGES;
    constexpr uint32_t STAGE_BYTES = G::STAGE_BYTES;
    constexpr uint32_t RING_BYTES = (uint32_t)STAGES * STAGE_BYTES;
    static_assert(STAGES % G::FG == 0 && STAGES >= G::FG, "ring depth is a multiple of the stages consumed per wait");
    static_assert(RING_BYTES + (uint32_t)(EPI_WARPS * EPI_BUFS) * EPI_BUF_BYTES <= SMEM_TILES + SMEM_EPI, "shared memory budget");
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;                 // 1024-byte aligned tile ring
    Barriers* bars = reinterpret_cast<Barriers*>(smem_raw + (ring - raw) + SMEM_TILES + SMEM_EPI);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = CG == 2 ? cluster_ctarank() : 0u;   // 0 = leader of the pair
    const int worker = blockIdx.x / CG, num_workers = gridDim.x / CG;
    const int tiles_per_batch = p.tiles_m * p.tiles_n;
    const int num_tiles = tiles_per_batch * p.batch;
    const int k_blocks = (int)((p.K + BK - 1) / BK);
    const bool A_MN = p.a_mn != 0, B_MN = p.b_mn != 0;
    static_assert(!SPLIT || EPI_WARPS == 8, "split accumulation uses eight epilogue warps");
    constexpr int FG = G::FG;
    const int k_pad = (k_blocks + FG - 1) / FG * FG;               // K-blocks are consumed FG at a time
    const int chunk_blocks = SPLIT ? SPLIT_BLOCKS : k_pad;         // K-blocks per use of a TMEM accumulator

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(smem_u32(&bars->full[s]), FG * CG); mbar_init(smem_u32(&bars->empty[s]), 1); }
        for (int a = 0; a < ACC_STAGES; ++a) { mbar_init(smem_u32(&bars->acc_full[a]), 1); mbar_init(smem_u32(&bars->acc_empty[a]), EPI_WARPS * CG); }
        bars->abort_flag = 0u;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                                              // whole warp (of each CTA): all 512 TMEM columns
        if (CG == 2) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_base)), "r"(TMEM_COLS) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();                              // the peer's barriers are initialised too
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    constexpr int EPI_BASE = Roles<SPLIT>::EPI_BASE;
    if (warp < EPI_BASE) {
    // every warp of the first group executes the same register release, then takes its role
    if (SPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(Roles<SPLIT>::REGS_FRONT));
    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer (each CTA loads its own rows)
        uint32_t stage = 0, phase = 0;
        bool ok = true;
        const uint64_t keep = policy_evict_last();
        int tile_no = 0;
        for (int t = worker; t < num_tiles && ok; t += num_workers) {
            int tm, tn;
            const int bi = t / tiles_per_batch;                                 // batch member
            tile_coords(t - bi * tiles_per_batch, p.tiles_m, p.tiles_n, tm, tn);
            const int m0 = tm * G::TILE_M + (int)cta_rank * BM;                 // this CTA's 128 rows of A
            const int n0 = tn * BN + (int)cta_rank * (BN / CG);                 // this CTA's rows of B
            // Every second tile of a worker walks K from its end: the workers of a wave finish a tile together at one end
            // of their operand panels and start the next tile there, where L2 still holds what they share (measured
            // 10-28 % fewer DRAM reads on four of the five workload GEMMs, +1.5-2.8 % sustained throughput on three).
            const bool backwards = (tile_no++ & 1) != 0;
            for (int kb = 0; kb < k_pad; ++kb) {
                ok = mbar_wait(smem_u32(&bars->empty[stage]), phase ^ 1u, abort_flag, WAIT_EMPTY);
                if (!ok) break;
                if (lane == 0) {
                    const uint32_t sa = ring + stage * STAGE_BYTES;
                    const uint32_t sb = sa + A_BYTES;
                    const int k0 = (backwards && kb < k_blocks ? k_blocks - 1 - kb : kb) * BK;
                    const uint32_t pair_bar = smem_u32(&bars->full[stage / FG]);          // one barrier per FG stages
                    if (CG == 2) {
                        const uint32_t full = map_to_cta(pair_bar, 0);                    // the leader's barrier
                        if (kb < k_blocks) {
                            mbar_arrive_expect_tx_cluster(full, STAGE_BYTES);
                            if (A_MN) tma_load_3d_pair(sa, &map_a, m0, k0, bi, full, keep);     // box {128 m, 128 k}
                            else      tma_load_3d_pair(sa, &map_a, k0, m0, bi, full, keep);     // box {128 k, 128 m}
                            if (B_MN) tma_load_3d_pair(sb, &map_b, n0, k0, bi, full, keep);     // box {128 n, 128 k}
                            else      tma_load_3d_pair(sb, &map_b, k0, n0, bi, full, keep);     // box {128 k, 128 n}
                        } else {
                            mbar_arrive_cluster(full);                                    // padding block: nothing to load
                        }
                    } else {
                        if (kb < k_blocks) {
                            mbar_arrive_expect_tx(pair_bar, STAGE_BYTES);
                            if (A_MN) tma_load_3d(sa, &map_a, m0, k0, bi, pair_bar, keep);
                            else      tma_load_3d(sa, &map_a, k0, m0, bi, pair_bar, keep);
                            if (B_MN) {                                               // two boxes {128 n, 128 k}
                                tma_load_3d(sb, &map_b, n0, k0, bi, pair_bar, keep);
                                tma_load_3d(sb + G::B_BYTES / 2, &map_b, n0 + 128, k0, bi, pair_bar, keep);
                            } else {
                                tma_load_3d(sb, &map_b, k0, n0, bi, pair_bar, keep);        // box {128 k, 256 n}
                            }
                        } else {
                            mbar_arrive(pair_bar);
                        }
                    }
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1u; }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (leader CTA only)
        uint32_t stage = 0, phase = 0;
        bool ok = cta_rank == 0;
        int it = 0;
        const uint32_t a_kstep = A_MN ? UMMA_K * 128 : UMMA_K, a_lbo = A_MN ? BK * 128 : 16;
        const uint32_t b_kstep = B_MN ? UMMA_K * 128 : UMMA_K, b_lbo = B_MN ? BK * 128 : 16;
        for (int t = worker; t < num_tiles && ok; t += num_workers) {
          for (int kc = 0; kc < k_pad && ok; kc += chunk_blocks, ++it) {          // `it` counts accumulator uses
            const uint32_t acc = (uint32_t)it & 1u, acc_phase = ((uint32_t)it >> 1) & 1u;
            ok = mbar_wait(smem_u32(&bars->acc_empty[acc]), acc_phase ^ 1u, abort_flag, WAIT_ACC_EMPTY);
            if (!ok) break;
            tc_fence_after();
            const uint32_t tmem_d = tmem_base + acc * BN;
            const int kend = min(k_pad, kc + chunk_blocks);
            const int last_real = min(k_blocks, kend) - 1;                        // its MMAs complete the accumulator
            for (int kb = kc; kb < kend; kb += FG) {
                // one wait per TWO K-blocks: every barrier query between MMA issues costs about one MMA time
                ok = mbar_wait(smem_u32(&bars->full[stage / FG]), phase, abort_flag, WAIT_FULL);
                if (!ok) break;
                tc_fence_after();
                if (lane == 0) {
#pragma unroll
                    for (int h = 0; h < FG; ++h) {
                        const uint32_t st = stage + h;
                        if (kb + h < k_blocks) {
                            const uint32_t sa = ring + st * STAGE_BYTES;
                            const uint32_t sb = sa + A_BYTES;
#pragma unroll
                            for (int k = 0; k < BK / UMMA_K; ++k) {
                                // K-major: 8-row groups 1024 B apart, +32 B per K step inside the swizzled row.
                                // MN-major: 8-k groups 1024 B apart, 128-wide MN blocks BK*128 B apart, +32 k-rows per step.
                                const uint64_t da = smem_desc(sa + k * a_kstep, a_lbo, 1024);
                                const uint64_t db = smem_desc(sb + k * b_kstep, b_lbo, 1024);
                                if (CG == 2) tc_mma_f8_pair(tmem_d, da, db, p.idesc, ((kb - kc) | h | k) != 0 ? 1u : 0u);
                                else         tc_mma_f8(tmem_d, da, db, p.idesc, ((kb - kc) | h | k) != 0 ? 1u : 0u);
                            }
                        }
                        // frees the smem stage (in both CTAs) when the MMAs retire (a padding block frees at once);
                        // the last real block of the chunk also publishes the accumulator
                        if (CG == 2) {
                            tc_commit_pair(smem_u32(&bars->empty[st]));
                            if (kb + h == last_real) tc_commit_pair(smem_u32(&bars->acc_full[acc]));
                        } else {
                            tc_commit(smem_u32(&bars->empty[st]));
                            if (kb + h == last_real) tc_commit(smem_u32(&bars->acc_full[acc]));
                        }
                    }
                }
                __syncwarp();
                stage += FG;
                if (stage == STAGES) { stage = 0; phase ^= 1u; }
            }
          }
        }
    }
    } else {
        // ------------------------------------------------------------ epilogue (each CTA drains its own 128 rows)
        if (SPLIT) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(Roles<SPLIT>::REGS_EPILOGUE));
        const int q = warp & 3;                                   // TMEM lane quarter this warp may read
        const float sa_inv = __ldg(p.sa_inv);
        const float alpha = p.sb_inv_vec ? 0.0f : sa_inv * __ldg(p.sb_inv);
        const float scale_d = (OUT == OUT_E4M3 || OUT == OUT_E5M2) ? __ldg(p.scale_d) : 1.0f;
        uint32_t running = 0;                                     // bf16: max of stored 16-bit magnitude patterns, two lanes
        float runf = 0.0f;                                        // fp32 / FP8 output: max |v|, NaN once any v is NaN
        const uint32_t epi_base = ring + RING_BYTES + (uint32_t)(warp - EPI_BASE) * (uint32_t)EPI_BUFS * EPI_BUF_BYTES;
        constexpr int COL_SPLIT = EPI_WARPS / 4;                  // warps sharing a lane quarter split the columns
        const int col_part = (warp - EPI_BASE) >> 2;
        uint32_t buf = 0;
        const uint64_t stream_out = policy_evict_first();
        bool ok = true;
        int it = 0;
        float part[SPLIT ? 128 : 1];                              // split accumulation: this thread's 128 partial sums
        for (int t = worker; t < num_tiles && ok; t += num_workers) {
          int tm, tn;
          const int bi = t / tiles_per_batch;
          tile_coords(t - bi * tiles_per_batch, p.tiles_m, p.tiles_n, tm, tn);
          for (int kc = 0; kc < k_pad && ok; kc += chunk_blocks, ++it) {         // `it` counts accumulator uses
            const uint32_t acc = (uint32_t)it & 1u, acc_phase = ((uint32_t)it >> 1) & 1u;
            ok = mbar_wait(smem_u32(&bars->acc_full[acc]), acc_phase, abort_flag, WAIT_ACC_FULL);
            if (!ok) break;
            tc_fence_after();
            const int row0 = tm * G::TILE_M + (int)cta_rank * BM + q * 32;      // first of this warp's 32 rows
            const bool row_ok = (int64_t)row0 + lane < p.M;
            const int64_t col0 = (int64_t)tn * BN;
            const uint32_t taddr = tmem_base + acc * BN + ((uint32_t)(q * 32) << 16);
            constexpr int ESZ = OUT == OUT_F32 ? 4 : OUT == OUT_BF16 ? 2 : 1;
            constexpr int CHUNK = 128 / ESZ;                      // columns per staged box: 128 bytes per row
            constexpr int SUBS = CHUNK / 32;                      // 32-column TMEM loads per box
            constexpr int WORDS = 32 * ESZ / 4;                   // 32-bit words one load contributes to the row
            constexpr int NBOX = BN / CHUNK / COL_SPLIT;          // boxes per warp and tile
            if (SPLIT) {
                // Split accumulation: every chunk of K, the last one included, is first moved into registers
                // (round-to-nearest adds onto the partial sums) and the accumulator handed back at once, so that
                // the MMA warp never waits for the conversion and the stores of a tile's last chunk.
                const bool have_part = kc != 0;
#pragma unroll
                for (int s2 = 0; s2 < (SPLIT ? 2 : 0); ++s2) {    // two 32-column loads in flight, one wait for both
                    uint32_t r[2][32];
                    tc_ld32(taddr + col_part * (BN / COL_SPLIT) + (2 * s2) * 32, r[0]);
                    tc_ld32(taddr + col_part * (BN / COL_SPLIT) + (2 * s2 + 1) * 32, r[1]);
                    tc_wait_ld();
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            float& acc_part = part[((2 * s2 + h) * 32 + i) % (SPLIT ? 128 : 1)];
                            acc_part = (have_part ? acc_part : 0.0f) + __uint_as_float(r[h][i]);
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    if (CG == 2) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[acc]), 0));
                    else         mbar_arrive(smem_u32(&bars->acc_empty[acc]));
                }
                if (kc + chunk_blocks < k_pad) continue;          // more of K to come
            }
#pragma unroll (SPLIT ? NBOX : 1)
            for (int cc = 0; cc < NBOX; ++cc) {
                const int c = col_part * NBOX + cc;
                const int64_t col = col0 + (int64_t)c * CHUNK;
                // A box that crosses the right edge is clipped by the TMA unit in 16-byte units: when the row
                // length in bytes is not a multiple of 16 that last box is written with plain stores instead.
                const bool direct = col + CHUNK > p.N && ((p.N * ESZ) & 15) != 0;
                const uint32_t sbuf = epi_base + buf * EPI_BUF_BYTES;
                const uint32_t srow = sbuf + lane * 128;
                if (!direct) {
                    if (lane == 0) bulk_wait_read<EPI_BUFS - 1>();  // the box last stored from this buffer has left it
                    __syncwarp();
                }
                // TMEM loads go out two at a time (one wait for both) where a box spans several loads
                constexpr int PRE = SUBS >= 2 ? 2 : 1;
                uint32_t rr[PRE][32];
#pragma unroll
                for (int sub = 0; sub < SUBS; ++sub) {
                    if (!SPLIT && sub % PRE == 0) {
#pragma unroll
                        for (int g = 0; g < PRE; ++g) tc_ld32(taddr + c * CHUNK + (sub + g) * 32, rr[g]);
                        tc_wait_ld();
                    }
                    uint32_t (&r)[32] = rr[sub % PRE];
                    if (SPLIT) {                                  // the sums are in registers already
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(part[((cc * SUBS + sub) * 32 + i) % (SPLIT ? 128 : 1)]);
                    }
                    float v[32];
                    if (p.sb_inv_vec) {                       // per-channel weight scales: one alpha per column
                        const int64_t scol_v = col + sub * 32;
#pragma unroll
                        for (int i = 0; i < 32; ++i) {
                            const float sb = scol_v + i < p.N ? __ldg(p.sb_inv_vec + scol_v + i) : 0.0f;
                            v[i] = __uint_as_float(r[i]) * (sa_inv * sb);
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]) * alpha;
                    }
                    uint32_t w[WORDS];                            // this thread's bytes of its row for these 32 columns
                    if (OUT == OUT_F32) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) w[i] = __float_as_uint(v[i]);
                    } else if (OUT == OUT_BF16) {
#pragma unroll
                        for (int i = 0; i < 16; ++i) w[i] = pack_bf16(v[2 * i], v[2 * i + 1]);
                    } else {
                        uint32_t codes[8];
                        if (OUT == OUT_E4M3) encode32<kE4M3>(v, scale_d, p.nosat != 0, codes);
                        else                 encode32<kE5M2>(v, scale_d, p.nosat != 0, codes);
#pragma unroll
                        for (int i = 0; i < 8; ++i) w[i] = codes[i];
                    }
                    // amax over in-bounds elements: of the stored values (fp32, bf16), of v before the output
                    // scale and conversion (FP8 output)
                    const int64_t scol = col + sub * 32;
                    if (row_ok && scol < p.N) {
                        if (scol + 32 <= p.N) {
                            if (OUT == OUT_BF16) {
#pragma unroll
                                for (int i = 0; i < 16; ++i) running = __vmaxu2(running, w[i] & 0x7FFF7FFFu);
                            } else {
#pragma unroll
                                for (int i = 0; i < 32; ++i) runf = fmax_nan(runf, fabsf(v[i]));
                            }
                        } else {
                            for (int i = 0; i < 32 && scol + i < p.N; ++i) {
                                if (OUT == OUT_BF16) running = __vmaxu2(running, ((i & 1) ? (w[i >> 1] >> 16) : w[i >> 1]) & 0x7FFFu);
                                else                 runf = fmax_nan(runf, fabsf(v[i]));
                            }
                        }
                    }
                    if (direct) {
                        if (row_ok) {
                            uint8_t* drow = reinterpret_cast<uint8_t*>(p.D) + ((int64_t)bi * p.stride_d + ((int64_t)row0 + lane) * p.ldd + scol) * ESZ;
                            for (int i = 0; i < 32 && scol + i < p.N; ++i) {
                                if (OUT == OUT_F32)       reinterpret_cast<uint32_t*>(drow)[i] = w[i];
                                else if (OUT == OUT_BF16) reinterpret_cast<uint16_t*>(drow)[i] = (uint16_t)((i & 1) ? (w[i >> 1] >> 16) : w[i >> 1]);
                                else                      drow[i] = (uint8_t)(w[i >> 2] >> (8 * (i & 3)));
                            }
                        }
                    } else {
                        // the 32 x 128 B box is staged with the 128-byte swizzle the tensor map expects
#pragma unroll
                        for (int j = 0; j < WORDS / 4; ++j) {
                            const int pos = sub * (WORDS / 4) + j;            // 16-byte position inside the 128-byte row
                            st_shared_v4(srow + ((pos ^ (lane & 7)) << 4), w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                        }
                    }
                }
                if (direct) continue;
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (row0 < p.M && col < p.N) tma_store_3d(&map_d, sbuf, (int)(col * ESZ), row0, bi, stream_out);
                    bulk_commit();
                }
                buf = (buf + 1u) % (uint32_t)EPI_BUFS;
            }
            if (!SPLIT) {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {                                  // accumulator may be overwritten: tell the leader's MMA warp
                    if (CG == 2) mbar_arrive_cluster(map_to_cta(smem_u32(&bars->acc_empty[acc]), 0));
                    else         mbar_arrive(smem_u32(&bars->acc_empty[acc]));
                }
            }
          }
        }
        if (lane == 0) bulk_wait_all();                           // every store has reached global memory before exit
        if (p.amax_bits) {
            uint32_t bits = OUT == OUT_BF16 ? (max(running & 0xFFFFu, running >> 16) << 16) : __float_as_uint(runf);
            bits = warp_max_u32(canonical_nan_bits(bits));
            if (lane == 0 && bits != 0u) atomicMax(p.amax_bits, bits);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (CG == 2) cluster_sync_all();        // neither CTA leaves while the other may still touch its smem, barriers or TMEM
    if (warp == 1) {
        tc_fence_after();
        if (CG == 2) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
        else         asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    }
}

// ---- host ------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    });
    return fn;
}

// 3-D byte tensor {inner, outer, batch} with row pitch `pitch` and batch pitch `batch_pitch` (bytes),
// box {box_inner, box_outer, 1}, 128B swizzle, zero fill.
static bool make_map(CUtensorMap* map, const void* base, uint64_t inner, uint64_t outer, uint64_t pitch,
                     uint64_t batch, uint64_t batch_pitch, uint32_t box_inner, uint32_t box_outer) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {inner, outer, batch};
    const cuuint64_t strides[2] = {pitch, batch > 1 ? batch_pitch : pitch * outer};
    const cuuint32_t box[3] = {box_inner, box_outer, 1};
    const cuuint32_t elem[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(base), dims, strides, box, elem,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// CTA-pair kernels launch as clusters of 2; the grid is one CTA per SM that can be paired.
// The dynamic shared-memory attribute and the number of co-resident clusters are properties of
// (kernel instance, device): looked up on the first launch of an instance on a device, then reused.
template <int CG, int OUT, int EPI_WARPS, bool SPLIT = false>
static fp8_status launch(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md, const Params& p, int64_t num_tiles, cudaStream_t st) {
    auto k = k_gemm_fp8<CG, OUT, EPI_WARPS, SPLIT>;
    constexpr int THREADS = 32 * (Roles<SPLIT>::EPI_BASE + EPI_WARPS);
    constexpr int MAX_DEVICES = 64;
    static std::mutex mu;
    static int cached_workers[MAX_DEVICES] = {0};                 // 0 = not looked up yet
    cudaLaunchConfig_t cfg = {};
    cfg.blockDim = dim3(THREADS, 1, 1);
    cfg.dynamicSmemBytes = SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CG;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FP8_ERR_CUDA;
    int workers = 0;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (dev >= 0 && dev < MAX_DEVICES) workers = cached_workers[dev];
        if (workers == 0) {
            if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES) != cudaSuccess) return FP8_ERR_CUDA;
            workers = sm_count() / CG;
            if (CG == 2) {
                cfg.gridDim = dim3(2 * workers, 1, 1);
                int clusters = 0;
                if (cudaOccupancyMaxActiveClusters(&clusters, k, &cfg) == cudaSuccess && clusters > 0 && clusters < workers) workers = clusters;
            }
            if (dev >= 0 && dev < MAX_DEVICES) cached_workers[dev] = workers;
        }
    }
    if ((int64_t)workers > num_tiles) workers = (int)num_tiles;
    cfg.gridDim = dim3(workers * CG, 1, 1);
    if (cudaLaunchKernelEx(&cfg, k, ma, mb, md, p) != cudaSuccess) return FP8_ERR_CUDA;
    count_launches(1);
    return launch_status();
}

template <int CG>
static fp8_status dispatch(int out_kind, bool short_k, bool split, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& md,
                           const Params& p, int64_t num_tiles, cudaStream_t st) {
    if (split && !short_k) {                                      // within one chunk of K there is nothing to split
        switch (out_kind) {
            case OUT_F32:  return launch<CG, OUT_F32, 8, true>(ma, mb, md, p, num_tiles, st);
            case OUT_BF16: return launch<CG, OUT_BF16, 8, true>(ma, mb, md, p, num_tiles, st);
            case OUT_E4M3: return launch<CG, OUT_E4M3, 8, true>(ma, mb, md, p, num_tiles, st);
            default:       return launch<CG, OUT_E5M2, 8, true>(ma, mb, md, p, num_tiles, st);
        }
    }
    if (short_k) {
        switch (out_kind) {
            case OUT_F32:  return launch<CG, OUT_F32, 8>(ma, mb, md, p, num_tiles, st);
            case OUT_BF16: return launch<CG, OUT_BF16, 8>(ma, mb, md, p, num_tiles, st);
            case OUT_E4M3: return launch<CG, OUT_E4M3, 8>(ma, mb, md, p, num_tiles, st);
            default:       return launch<CG, OUT_E5M2, 8>(ma, mb, md, p, num_tiles, st);
        }
    }
    switch (out_kind) {
        case OUT_F32:  return launch<CG, OUT_F32, 4>(ma, mb, md, p, num_tiles, st);
        case OUT_BF16: return launch<CG, OUT_BF16, 4>(ma, mb, md, p, num_tiles, st);
        case OUT_E4M3: return launch<CG, OUT_E4M3, 4>(ma, mb, md, p, num_tiles, st);
        default:       return launch<CG, OUT_E5M2, 4>(ma, mb, md, p, num_tiles, st);
    }
}

// Shared body of fp8_gemm and fp8_gemm_fp8out.
struct Batch { int64_t count, stride_a, stride_b, stride_d; };      // strides in elements

static fp8_status gemm_impl(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, void* D, int out_kind, int nosat,
                            const float* sa_inv, const float* sb_inv, const float* sb_inv_vec, const float* scale_d,
                            float* amax_d_dev, cudaStream_t st, Batch bt = Batch{1, 0, 0, 0}) {
    const int64_t M = d->M, N = d->N, K = d->K;
    if (M < 0 || N < 0 || K < 0 || bt.count < 0) return FP8_ERR_SHAPE;
    const bool a_mn = d->ma == FP8_MAJOR_MN, b_mn = d->mb == FP8_MAJOR_MN;
    const int64_t esz = out_kind == OUT_F32 ? 4 : out_kind == OUT_BF16 ? 2 : 1;
    // CTA pairs (256-row tiles) unless the whole problem has at most 128 rows
    const int cg = M > BM ? 2 : 1;
    const int64_t tile_m = (int64_t)BM * cg;
    const int64_t tiles_m = (M + tile_m - 1) / tile_m, tiles_n = (N + BN - 1) / BN;
    // ---- validation: nothing is enqueued before every check has passed
    if (M > 0 && N > 0) {
        if (!D) return FP8_ERR_NULL;
        if (d->ldd < N) return FP8_ERR_SHAPE;
        if (K > 0) {
            if (!A || !B) return FP8_ERR_NULL;
            if (d->lda < (a_mn ? M : K) || d->ldb < (b_mn ? N : K)) return FP8_ERR_SHAPE;
            if ((reinterpret_cast<uintptr_t>(A) & 15u) || (reinterpret_cast<uintptr_t>(B) & 15u) || (d->lda & 15) || (d->ldb & 15))
                return FP8_ERR_ALIGN;
        }
        if ((reinterpret_cast<uintptr_t>(D) & 15u) || ((d->ldd * esz) & 15)) return FP8_ERR_ALIGN;
        if (bt.count > 1) {
            // written members may not overlap; read-only members may interleave or overlap
            if (bt.stride_a <= 0 || bt.stride_b <= 0 || bt.stride_d < M * d->ldd) return FP8_ERR_SHAPE;
            if ((bt.stride_a & 15) || (bt.stride_b & 15) || ((bt.stride_d * esz) & 15)) return FP8_ERR_ALIGN;
        }
        if (tiles_m * tiles_n * (bt.count > 0 ? bt.count : 1) > (int64_t)1 << 30 || M > ((int64_t)1 << 31) - 256 ||
            N > ((int64_t)1 << 31) - 512 || K > ((int64_t)1 << 31) - 256 || bt.count > 65535)
            return FP8_ERR_UNSUPPORTED;
    }
    // ---- work
    if (amax_d_dev) {
        if (cudaMemsetAsync(amax_d_dev, 0, 4, st) != cudaSuccess) return FP8_ERR_CUDA;
        count_launches(1);
    }
    if (M == 0 || N == 0 || bt.count == 0) return FP8_OK;
    if (K == 0) {                                                 // empty sum: zeros in every output type
        for (int64_t b = 0; b < bt.count; ++b) {
            if (cudaMemset2DAsync(reinterpret_cast<uint8_t*>(D) + b * bt.stride_d * esz, (size_t)(d->ldd * esz), 0, (size_t)(N * esz),
                                  (size_t)M, st) != cudaSuccess)
                return FP8_ERR_CUDA;
            count_launches(1);
        }
        return FP8_OK;
    }

    CUtensorMap map_a, map_b;
    const uint32_t b_rows = (uint32_t)(BN / cg);                  // B rows one CTA loads per K-block
    const uint64_t nb = (uint64_t)bt.count;
    bool ok = a_mn ? make_map(&map_a, A, (uint64_t)M, (uint64_t)K, (uint64_t)d->lda, nb, (uint64_t)bt.stride_a, 128, BK)
                   : make_map(&map_a, A, (uint64_t)K, (uint64_t)M, (uint64_t)d->lda, nb, (uint64_t)bt.stride_a, BK, BM);
    ok = ok && (b_mn ? make_map(&map_b, B, (uint64_t)N, (uint64_t)K, (uint64_t)d->ldb, nb, (uint64_t)bt.stride_b, 128, BK)
                     : make_map(&map_b, B, (uint64_t)K, (uint64_t)N, (uint64_t)d->ldb, nb, (uint64_t)bt.stride_b, BK, b_rows));
    // D as a byte tensor {N*esz, M}: boxes of 128 bytes x 32 rows, the unit each epilogue warp stores
    CUtensorMap map_d;
    ok = ok && make_map(&map_d, D, (uint64_t)(N * esz), (uint64_t)M, (uint64_t)(d->ldd * esz), nb, (uint64_t)(bt.stride_d * esz), 128, 32);
    if (!ok) return FP8_ERR_CUDA;

    Params p;
    p.M = M; p.N = N; p.K = K; p.ldd = d->ldd; p.D = D;
    p.sa_inv = sa_inv; p.sb_inv = sb_inv; p.sb_inv_vec = sb_inv_vec;
    p.amax_bits = reinterpret_cast<uint32_t*>(amax_d_dev);
    p.tiles_m = (int)tiles_m; p.tiles_n = (int)tiles_n;
    p.a_mn = a_mn ? 1 : 0; p.b_mn = b_mn ? 1 : 0;
    p.batch = (int)bt.count; p.stride_d = bt.stride_d;
    p.scale_d = scale_d; p.nosat = nosat;
    // instruction descriptor: fp32 accumulate, operand formats and majors, N/8, M/16 (M = 256 for a CTA pair)
    p.idesc = (1u << 4) | ((uint32_t)d->fa << 7) | ((uint32_t)d->fb << 10) | ((a_mn ? 1u : 0u) << 15) |
              ((b_mn ? 1u : 0u) << 16) | ((uint32_t)(BN >> 3) << 17) | ((uint32_t)(tile_m >> 4) << 24);
    const bool short_k = (K + BK - 1) / BK <= SHORT_K_BLOCKS;
    const bool split = d->acc == FP8_ACC_SPLIT;
    return cg == 2 ? dispatch<2>(out_kind, short_k, split, map_a, map_b, map_d, p, tiles_m * tiles_n * bt.count, st)
                   : dispatch<1>(out_kind, short_k, split, map_a, map_b, map_d, p, tiles_m * tiles_n * bt.count, st);
}

// ---- split-K for problems with few output tiles --------------------------------------------

// Sum of `splits` fp32 partial products (already multiplied by alpha), rounded to the output type, with the
// amax of the stored values.  Four columns per thread; the additions run in slice order, so the result does
// not depend on the launch shape.
template <int OUT>
__global__ void __launch_bounds__(256)
k_splitk_reduce(const float* __restrict__ part, int splits, int64_t M, int64_t N, void* __restrict__ D, int64_t ldd,
                uint32_t* amax_bits) {
    __shared__ uint32_t red[32];
    const int64_t quads_per_row = (N + 3) / 4;
    const int64_t total = M * quads_per_row;
    const int64_t plane = M * N;
    uint32_t running = 0;
    for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < total; q += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = q / quads_per_row, j = (q - i * quads_per_row) * 4;
        const int n = (int)min((int64_t)4, N - j);
        float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        const float* p = part + i * N + j;
        if (n == 4 && (N & 3) == 0) {
            for (int sidx = 0; sidx < splits; ++sidx) {
                const float4 t = *reinterpret_cast<const float4*>(p + (int64_t)sidx * plane);
                v[0] += t.x; v[1] += t.y; v[2] += t.z; v[3] += t.w;
            }
        } else {
            for (int sidx = 0; sidx < splits; ++sidx)
                for (int e = 0; e < n; ++e) v[e] += p[(int64_t)sidx * plane + e];
        }
        if (OUT == OUT_F32) {
            float* d = reinterpret_cast<float*>(D) + i * ldd + j;
            for (int e = 0; e < n; ++e) {
                d[e] = v[e];
                running = max(running, canonical_nan_bits(__float_as_uint(v[e]) & 0x7FFFFFFFu));
            }
        } else {
            uint16_t* d = reinterpret_cast<uint16_t*>(D) + i * ldd + j;
            const uint32_t w0 = pack_bf16(v[0], v[1]), w1 = pack_bf16(v[2], v[3]);
            const uint16_t h[4] = {(uint16_t)w0, (uint16_t)(w0 >> 16), (uint16_t)w1, (uint16_t)(w1 >> 16)};
            for (int e = 0; e < n; ++e) {
                d[e] = h[e];
                running = max(running, canonical_nan_bits(((uint32_t)h[e] & 0x7FFFu) << 16));
            }
        }
    }
    if (amax_bits) block_atomic_max_bits(running, red, amax_bits);
}

// Number of K-slices for a problem.  Measured on B200: one output tile (a CTA, or a CTA pair) streams its operand
// panels at about 90 GB/s (its ring of stages in flight over the memory latency), so a product with T tiles reads
// its operands at min(T x 90 GB/s, HBM); slices multiply T, and cost a second launch plus the fp32 partials
// (about 9 us + 8 B per partial element).  The smallest power of two (at most 16, slices multiples of 256 of K
// and at least 1024 long, tiles x slices within the SMs) whose modelled time is at least 15 % below the
// unsliced one is taken; 1 otherwise.
static int choose_splits(int64_t M, int64_t N, int64_t K) {
    if (M <= 0 || N <= 0 || K < 2048 || (N & 3) != 0) return 1;    // fp32 partial rows are whole 16-byte units
    const int cg = M > BM ? 2 : 1;
    const double tiles = (double)(((M + BM * cg - 1) / (BM * cg)) * ((N + BN - 1) / BN));
    const double workers = (double)(sm_count() / cg);
    const double bytes = (double)K * (double)(M + N);
    const double tile_rate = 90e9, hbm_rate = 6.0e12, split_cost = 9e-6, partial_rate = 5.0e12;
    auto modelled = [&](int sl) {
        double rate = tiles * sl * tile_rate;
        if (rate > hbm_rate) rate = hbm_rate;
        return bytes / rate + (sl > 1 ? split_cost + 8.0 * sl * (double)M * (double)N / partial_rate : 0.0);
    };
    const double base = modelled(1);
    int best = 1;
    double best_t = base;
    for (int sl = 2; sl <= 16; sl *= 2) {
        if (tiles * sl > workers || K % ((int64_t)sl * 256) != 0 || K / sl < 1024) break;
        const double t = modelled(sl);
        if (t < 0.95 * best_t) { best = sl; best_t = t; }
    }
    return best_t <= 0.85 * base ? best : 1;
}

// Self-test of the bounded mbarrier wait: one CTA initialises a barrier that nobody arrives on and waits
// for it with the given limit; the wait gives up, latches WAIT_SELF_TEST and the kernel returns.
__global__ void k_wait_self_test(long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0u;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0) (void)mbar_wait(smem_u32(&bar), 0u, &abort_flag, WAIT_SELF_TEST, limit_cycles);
    __syncthreads();
}

}  // namespace gemm

fp8_status launch_grid_barrier_self_test(long long limit_cycles, cudaStream_t st);      // defined with the cast kernels

}  // namespace fp8b200

using namespace fp8b200;

extern "C" {

static bool desc_enums_ok(const fp8_gemm_desc* d) {
    return (d->fa == FP8_E4M3 || d->fa == FP8_E5M2) && (d->fb == FP8_E4M3 || d->fb == FP8_E5M2) &&
           (d->ma == FP8_MAJOR_K || d->ma == FP8_MAJOR_MN) && (d->mb == FP8_MAJOR_K || d->mb == FP8_MAJOR_MN) &&
           (d->acc == FP8_ACC_FAST || d->acc == FP8_ACC_SPLIT);
}

fp8_status fp8_gemm(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, void* D,
                    const float* scale_inv_a_dev, const float* scale_inv_b_dev, float* amax_d_dev, void* stream) {
    using namespace fp8b200::gemm;
    if (!d || !scale_inv_a_dev || !scale_inv_b_dev) return FP8_ERR_NULL;
    if (!desc_enums_ok(d) || (d->out != FP8_F32 && d->out != FP8_BF16)) return FP8_ERR_ENUM;
    return gemm_impl(d, A, B, D, d->out == FP8_BF16 ? OUT_BF16 : OUT_F32, 0, scale_inv_a_dev, scale_inv_b_dev, nullptr, nullptr,
                     amax_d_dev, (cudaStream_t)stream);
}

fp8_status fp8_gemm_batched(const fp8_gemm_desc* d, int64_t batch, const uint8_t* A, int64_t stride_a, const uint8_t* B, int64_t stride_b,
                            void* D, int64_t stride_d, const float* scale_inv_a_dev, const float* scale_inv_b_dev,
                            float* amax_d_dev, void* stream) {
    using namespace fp8b200::gemm;
    if (!d || !scale_inv_a_dev || !scale_inv_b_dev) return FP8_ERR_NULL;
    if (!desc_enums_ok(d) || (d->out != FP8_F32 && d->out != FP8_BF16)) return FP8_ERR_ENUM;
    return gemm_impl(d, A, B, D, d->out == FP8_BF16 ? OUT_BF16 : OUT_F32, 0, scale_inv_a_dev, scale_inv_b_dev, nullptr, nullptr,
                     amax_d_dev, (cudaStream_t)stream, Batch{batch, stride_a, stride_b, stride_d});
}

fp8_status fp8_gemm_channel_scales(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, void* D,
                                   const float* scale_inv_a_dev, const float* scale_inv_b_vec_dev, float* amax_d_dev, void* stream) {
    using namespace fp8b200::gemm;
    if (!d || !scale_inv_a_dev || !scale_inv_b_vec_dev) return FP8_ERR_NULL;
    if (!desc_enums_ok(d) || (d->out != FP8_F32 && d->out != FP8_BF16)) return FP8_ERR_ENUM;
    return gemm_impl(d, A, B, D, d->out == FP8_BF16 ? OUT_BF16 : OUT_F32, 0, scale_inv_a_dev, nullptr, scale_inv_b_vec_dev, nullptr,
                     amax_d_dev, (cudaStream_t)stream);
}

fp8_status fp8_gemm_fp8out(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, uint8_t* D, fp8_format fd, fp8_overflow od,
                           const float* scale_inv_a_dev, const float* scale_inv_b_dev, const float* scale_d_dev,
                           float* amax_d_dev, void* stream) {
    using namespace fp8b200::gemm;
    if (!d || !scale_inv_a_dev || !scale_inv_b_dev || !scale_d_dev) return FP8_ERR_NULL;
    if (!desc_enums_ok(d) || (fd != FP8_E4M3 && fd != FP8_E5M2) || (od != FP8_SATURATE && od != FP8_NOSAT)) return FP8_ERR_ENUM;
    return gemm_impl(d, A, B, D, fd == FP8_E4M3 ? OUT_E4M3 : OUT_E5M2, od == FP8_NOSAT ? 1 : 0, scale_inv_a_dev, scale_inv_b_dev,
                     nullptr, scale_d_dev, amax_d_dev, (cudaStream_t)stream);
}

fp8_status fp8_gemm_splitk_workspace(const fp8_gemm_desc* d, int* splits_out, size_t* bytes_out) {
    using namespace fp8b200::gemm;
    if (!d || !splits_out || !bytes_out) return FP8_ERR_NULL;
    if (d->M < 0 || d->N < 0 || d->K < 0) return FP8_ERR_SHAPE;
    const int s = choose_splits(d->M, d->N, d->K);
    *splits_out = s;
    *bytes_out = s > 1 ? (size_t)s * (size_t)d->M * (size_t)d->N * sizeof(float) : 0;
    return FP8_OK;
}

fp8_status fp8_gemm_splitk(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, void* D,
                           const float* scale_inv_a_dev, const float* scale_inv_b_dev, float* amax_d_dev,
                           void* workspace_dev, size_t workspace_bytes, void* stream) {
    using namespace fp8b200::gemm;
    if (!d || !scale_inv_a_dev || !scale_inv_b_dev) return FP8_ERR_NULL;
    if (!desc_enums_ok(d) || (d->out != FP8_F32 && d->out != FP8_BF16)) return FP8_ERR_ENUM;
    const int out_kind = d->out == FP8_BF16 ? OUT_BF16 : OUT_F32;
    cudaStream_t st = (cudaStream_t)stream;
    const int splits = (d->M >= 0 && d->N >= 0 && d->K >= 0) ? choose_splits(d->M, d->N, d->K) : 1;
    if (splits == 1)
        return gemm_impl(d, A, B, D, out_kind, 0, scale_inv_a_dev, scale_inv_b_dev, nullptr, nullptr, amax_d_dev, st);
    const size_t need = (size_t)splits * (size_t)d->M * (size_t)d->N * sizeof(float);
    if (!workspace_dev || !D) return FP8_ERR_NULL;
    if (workspace_bytes < need) return FP8_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(workspace_dev) & 15u) return FP8_ERR_ALIGN;
    const int64_t esz = out_kind == OUT_F32 ? 4 : 2;
    if (d->ldd < d->N) return FP8_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(D) & (uintptr_t)(esz - 1)) != 0) return FP8_ERR_ALIGN;
    // the K-slices as members of one batched product with fp32 output (alpha applied per slice)
    const int64_t ks = d->K / splits;
    fp8_gemm_desc slice = *d;
    slice.K = ks;
    slice.ldd = d->N;
    slice.out = FP8_F32;
    const bool a_mn = d->ma == FP8_MAJOR_MN, b_mn = d->mb == FP8_MAJOR_MN;
    Batch bt{splits, a_mn ? ks * d->lda : ks, b_mn ? ks * d->ldb : ks, d->M * d->N};
    fp8_status rc = gemm_impl(&slice, A, B, workspace_dev, OUT_F32, 0, scale_inv_a_dev, scale_inv_b_dev, nullptr, nullptr, nullptr, st, bt);
    if (rc != FP8_OK) return rc;
    if (amax_d_dev) {
        if (cudaMemsetAsync(amax_d_dev, 0, 4, st) != cudaSuccess) return FP8_ERR_CUDA;
        count_launches(1);
    }
    const int64_t quads = d->M * ((d->N + 3) / 4);
    int64_t grid = (quads + 255) / 256;
    const int64_t cap = (int64_t)sm_count() * 8;
    if (grid > cap) grid = cap;
    if (out_kind == OUT_F32)
        k_splitk_reduce<OUT_F32><<<(unsigned)grid, 256, 0, st>>>(reinterpret_cast<const float*>(workspace_dev), splits, d->M, d->N, D, d->ldd,
                                                                  reinterpret_cast<uint32_t*>(amax_d_dev));
    else
        k_splitk_reduce<OUT_BF16><<<(unsigned)grid, 256, 0, st>>>(reinterpret_cast<const float*>(workspace_dev), splits, d->M, d->N, D, d->ldd,
                                                                   reinterpret_cast<uint32_t*>(amax_d_dev));
    count_launches(1);
    return launch_status();
}


fp8_status fp8_self_test_expire_wait(int which, uint64_t limit_cycles, void* stream) {
    if (which != FP8_WAIT_MBARRIER && which != FP8_WAIT_GRID_BARRIER) return FP8_ERR_ENUM;
    if (limit_cycles == 0 || limit_cycles > 2000000000ull) return FP8_ERR_UNSUPPORTED;      // at most about a second
    cudaStream_t st = (cudaStream_t)stream;
    if (which == FP8_WAIT_GRID_BARRIER) return fp8b200::launch_grid_barrier_self_test((long long)limit_cycles, st);
    fp8b200::gemm::k_wait_self_test<<<1, 32, 0, st>>>((long long)limit_cycles);
    count_launches(1);
    return launch_status();
}

void fp8_cast_read_clear_latch(unsigned int out2[2]);      // defined with the cast kernels

fp8_status fp8_async_status(uint32_t* detail) {
    unsigned int latch[2] = {0u, 0u};
    if (cudaDeviceSynchronize() != cudaSuccess) return FP8_ERR_CUDA;
    unsigned int cast_latch[2];
    fp8_cast_read_clear_latch(cast_latch);
    if (cudaMemcpyFromSymbol(latch, g_async_latch, sizeof(latch)) != cudaSuccess) return FP8_ERR_CUDA;
    if (latch[0] == 0u && cast_latch[0] != 0u) {
        if (detail) *detail = cast_latch[0];
        return FP8_ERR_TIMEOUT;
    }
    if (detail) *detail = latch[0];
    if (latch[0] == 0u) return FP8_OK;
    const unsigned int zero[2] = {0u, 0u};
    if (cudaMemcpyToSymbol(g_async_latch, zero, sizeof(zero)) != cudaSuccess) return FP8_ERR_CUDA;
    return FP8_ERR_TIMEOUT;
}

}  // extern "C"
