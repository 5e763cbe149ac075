/*
 * fp8_b200 — C ABI of the B200 (sm_100a) FP8 hot path of
 * "FP8 Formats for Deep Learning" (arXiv 2209.05433).
 *
 * Conventions shared by every call
 *   - Every pointer whose name ends in _dev, and every tensor pointer (x, c,
 *     out, A, B, D), is a DEVICE pointer owned by the caller.  The library
 *     never allocates or frees device memory and keeps no per-call state.
 *   - Scalars that flow between calls (amax, scale, scale_inv) live in device
 *     memory, so amax -> scale -> quantize -> gemm chain on one stream with no
 *     host synchronisation.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls only enqueue work and return; argument errors are found on the
 *     host before anything is launched.
 *   - The return value is a status code; nothing aborts or throws.  A launch
 *     failure is reported as FP8_ERR_CUDA.  A device-side wait that ran out of
 *     patience (never expected) is latched and read by fp8_async_status().
 *   - bf16 tensors are arrays of 16-bit patterns (the upper half of binary32);
 *     FP8 tensors are arrays of 8-bit codes in the paper's S.E.M layout.
 */
#ifndef FP8_B200_H
#define FP8_B200_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FP8_OK = 0,
    FP8_ERR_NULL = 1,        /* a required pointer is NULL */
    FP8_ERR_ENUM = 2,        /* an enum argument is out of range */
    FP8_ERR_SHAPE = 3,       /* negative size, or a leading dimension smaller than the row */
    FP8_ERR_ALIGN = 4,       /* GEMM operand base or leading dimension not 16-byte aligned */
    FP8_ERR_UNSUPPORTED = 5, /* a size beyond what the launch geometry can address */
    FP8_ERR_CUDA = 6,        /* the CUDA runtime / driver reported an error */
    FP8_ERR_TIMEOUT = 7      /* a bounded device-side wait expired (see fp8_async_status) */
} fp8_status;

/* The two encodings of Section 3 / Table 1. */
typedef enum { FP8_E4M3 = 0, FP8_E5M2 = 1 } fp8_format;
/* The wider type a tensor is converted from / to (Section 2). */
typedef enum { FP8_F32 = 0, FP8_BF16 = 1 } fp8_wide;
/* Section 2: overflow saturates to the maximum finite value (default), or, in the
 * non-saturating mode, becomes NaN (E4M3, which has no infinity) / Inf (E5M2). */
typedef enum { FP8_SATURATE = 0, FP8_NOSAT = 1 } fp8_overflow;
/* Which index of a GEMM operand is contiguous in memory. */
typedef enum { FP8_MAJOR_K = 0, FP8_MAJOR_MN = 1 } fp8_major;
/* how a GEMM accumulates over K (see fp8_gemm) */
typedef enum { FP8_ACC_SPLIT = 0, FP8_ACC_FAST = 1 } fp8_accumulate;

/*
 * fp8_amax — maximum magnitude of a tensor (Section 2: the quantity the scale
 * factor is chosen from).
 *   x         device, n elements of type t, any element-aligned address.
 *   amax_dev  device, one float, OVERWRITTEN with max_i |x_i| (+0 when n == 0).
 *             If any element is NaN the result is NaN (pattern 0x7FC00000);
 *             otherwise an infinity gives +Inf.  The result is exact and does
 *             not depend on reduction order.
 */
fp8_status fp8_amax(const void* x, fp8_wide t, size_t n, float* amax_dev, void* stream);

/*
 * fp8_scale_from_amax — Section 2: the scale factor that moves the tensor's
 * maximum magnitude onto the format's maximum (Table 1: 448 / 57344).
 *   scale = fmax / amax (binary32 division); amax of 0, NaN or Inf gives 1; a
 *   quotient that overflows is clamped to the largest finite binary32.
 *   scale_inv = 1 / scale.  All three pointers are device floats.
 */
fp8_status fp8_scale_from_amax(const float* amax_dev, fp8_format f,
                               float* scale_dev, float* scale_inv_dev, void* stream);

/*
 * fp8_quantize — Section 2: multiply by the per-tensor scale factor, convert to
 * FP8 (Table 1 encodings) with round-to-nearest-even.
 *   out_i = encode_f( binary32(x_i) * scale ), the product rounded to binary32
 *   first.  Special values convert to special values in both overflow modes:
 *   NaN -> sign|0x7F; +-Inf -> E4M3 sign|0x7F (NaN), E5M2 sign|0x7C (Inf); this
 *   rule is applied to the scaled value.  Finite overflow follows `o`.  The sign
 *   of zero and of values that round to zero is kept.
 *   x          device, n elements of type t.
 *   scale_dev  device float, read by the kernel.
 *   out        device, n bytes.
 *   amax_dev   NULL, or a device float OVERWRITTEN with amax(x) of the same pass
 *              (same definition as fp8_amax), for callers that scale with the
 *              previous step's amax.
 *   Fast path: x and out both 16-byte aligned; other alignments take a slower
 *   element-wise path with identical results.
 */
fp8_status fp8_quantize(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o,
                        const float* scale_dev, uint8_t* out, float* amax_dev, void* stream);

/*
 * fp8_quantize_current — Section 2, the whole current-scaling conversion of one tensor in ONE call:
 * the scale is chosen from the tensor's own maximum magnitude, then the tensor is converted with it.
 * Results are identical, bit for bit, to fp8_amax + fp8_scale_from_amax + fp8_quantize:
 *   *amax_dev = amax(x); *scale_dev = fmax/amax (same guards); *scale_inv_dev = 1/scale;
 *   out_i = encode_f( binary32(x_i) * scale ).
 * Tensors below 256 MB take ONE kernel, launched cooperatively (all of its blocks resident at once), which
 * crosses one grid-wide barrier between the two passes; the second pass re-reads the tail of x from L2.  A tensor
 * small enough for the shared memory of the whole GPU (about 33 MB on a B200) is kept there between the passes and
 * read from global memory only once.
 * Larger tensors (and pointers without 16-byte alignment) take the three streaming kernels back to back on the
 * stream, the conversion walking the tensor from its end, where the amax pass has just been: on long streams
 * that is the faster form, and the workspace is then not touched.
 *   workspace  device, fp8_quantize_current_workspace_bytes() bytes, 16-byte aligned, owned by the
 *              caller.  It must hold zeros before the first call; every call leaves it zeroed again,
 *              so one buffer serves any number of calls on one stream.  Calls that may overlap on the
 *              GPU (different streams) need different workspaces.
 * The grid barrier is a bounded wait (about two seconds).  If it expires in any block, fp8_async_status
 * reports FP8_ERR_TIMEOUT and the contents of out, amax_dev, scale_dev and scale_inv_dev are undefined (blocks
 * that gave up write nothing, blocks that got through may have written their share).  The workspace is left
 * zeroed in that case too: the last block to leave clears it whether or not the barrier held.
 */
fp8_status fp8_quantize_current(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o,
                                uint8_t* out, float* amax_dev, float* scale_dev, float* scale_inv_dev,
                                void* workspace, void* stream);

/* Size in bytes of the workspace fp8_quantize_current needs. */
size_t fp8_quantize_current_workspace_bytes(void);

/*
 * fp8_quantize_current_static — the paper has no counterpart; this entry point exists for callers
 * that cannot obtain device memory for a workspace.
 *
 * Who that is: code that runs where cudaMalloc is off limits or would fail — a plug-in called from
 * inside another framework's memory pool that already owns all of the GPU's memory, a latency-bound
 * serving loop in which an allocation (an implicit device synchronisation) is not acceptable, or a
 * component that is only ever handed its input and output buffers.  Such a caller still wants the
 * one-launch current-scaling conversion of fp8_quantize_current, but has no 16 spare bytes to pass.
 *
 * What it does: exactly fp8_quantize_current (same kernel, same results bit for bit), with the
 * kernel's three control words kept in a 256-byte array that is part of the library image.  Every GPU
 * that loads the library holds those 256 bytes until the process exits.  The call allocates nothing:
 * no cudaMalloc, no cudaFree, no allocating library routine.  The caller passes inputs and outputs only.
 *
 * Rules of use
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Each call clears the words it needs before its
 *     kernel runs, so a call never depends on what the previous one left behind; but two calls that
 *     overlap on the GPU (different streams, or different host threads on different streams) race on
 *     it and give undefined results.  Issue them on one stream, or serialise them yourself.
 *   - n may not exceed FP8_STATIC_MAX_ELEMENTS; larger tensors return FP8_ERR_UNSUPPORTED and nothing
 *     is enqueued.  (The scratch need of this kernel does not grow with n; the bound is simply the
 *     stated maximum of this entry point.)
 *   - Arguments, alignment rules and the bounded grid barrier are those of fp8_quantize_current.
 */
#define FP8_STATIC_MAX_ELEMENTS ((size_t)1 << 32)
fp8_status fp8_quantize_current_static(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o,
                                       uint8_t* out, float* amax_dev, float* scale_dev, float* scale_inv_dev,
                                       void* stream);

/*
 * fp8_dequantize — Section 2: convert back and multiply by the inverse of the
 * scale factor.  out_i = round_t( decode_f(c_i) * scale_inv ), one binary32
 * multiply, then round-to-nearest-even to bf16 when t is FP8_BF16.  NaN codes
 * give NaN (payload unspecified), E5M2 infinities give infinities.
 */
fp8_status fp8_dequantize(const uint8_t* c, size_t n, fp8_format f,
                          const float* scale_inv_dev, void* out, fp8_wide t, void* stream);

/*
 * fp8_fake_quantize — Section 4: the paper's own experiments simulated FP8: tensors were converted
 * to FP8 (scale factor, rounding and saturation included) and straight back to the wider type, and the
 * arithmetic stayed in that wider type.  This is that round trip in one pass over the tensor:
 *   out_i = round_t( decode_f( encode_f( binary32(x_i) * scale ) ) * scale_inv ),  out has the type of x.
 * Bit for bit the composition of fp8_quantize and fp8_dequantize, without the intermediate code tensor
 * (4 B per bf16 element of traffic instead of 6).
 */
fp8_status fp8_fake_quantize(const void* x, fp8_wide t, size_t n, fp8_format f, fp8_overflow o,
                             const float* scale_dev, const float* scale_inv_dev, void* out, void* stream);

/*
 * fp8_scale_pow2_from_amax — Section 3.2: a programmable exponent bias amounts to restricting the scale
 * factors to powers of two.  scale = the largest power of two not above fmax/amax (same guards
 * as fp8_scale_from_amax), scale_inv = 1/scale (exact).  Converting with this scale is converting to an
 * E4M3/E5M2 variant whose exponent bias is shifted by log2(scale) (the bias sweep of Section 4.3).
 */
fp8_status fp8_scale_pow2_from_amax(const float* amax_dev, fp8_format f,
                                    float* scale_dev, float* scale_inv_dev, void* stream);

/*
 * fp8_gemm — Sections 2, 3 and 4.1: the matrix multiply on FP8 inputs with a
 * higher-precision result, unscaled once per dot product.
 *   D[i,j] = round_out( (sum_k decode_fa(A[i,k]) * decode_fb(B[k,j])) * (sa_inv * sb_inv) )
 * with binary32 accumulation on the tensor cores.
 * Operand roles (Section 3: E4M3 for weights and activations, E5M2 for
 * gradients): forward  fa=E4M3, fb=E4M3;  dgrad  fa=E5M2 (dY), fb=E4M3 (W);
 * wgrad  fa=E4M3 (X^T), fb=E5M2 (dY).  Any of the four pairs is accepted.
 *   A   M x K codes.  ma == FP8_MAJOR_K : A[i,k] at A[i*lda + k] (lda >= K);
 *                     ma == FP8_MAJOR_MN: A[i,k] at A[k*lda + i] (lda >= M).
 *   B   K x N codes.  mb == FP8_MAJOR_K : B[k,j] at B[j*ldb + k] (ldb >= K);
 *                     mb == FP8_MAJOR_MN: B[k,j] at B[k*ldb + j] (ldb >= N).
 *   D   M x N, row-major, D[i,j] at D[i*ldd + j], of type `out` (ldd in elements).
 *   scale_inv_a_dev / scale_inv_b_dev  device floats (the operands' inverse scales).
 *   amax_d_dev  NULL, or a device float OVERWRITTEN with amax of D as stored
 *               (after rounding), same definition as fp8_amax.
 * Alignment: A, B, D base addresses, lda, ldb (bytes) and ldd*sizeof(out) must
 * be multiples of 16, else FP8_ERR_ALIGN.  M, N, K are otherwise arbitrary
 * (edges are zero-filled on load and clipped on store).  M*N == 0 is a no-op
 * (amax = 0); K == 0 writes zeros.
 * Accumulation (`acc`): the products are exact and the tensor core adds them, 32 of K at a time, into a
 * binary32 accumulator whose additions round toward zero.
 *   FP8_ACC_SPLIT  (0, the default of a zero-initialised descriptor) the accumulator is drained every 2048 of K and the
 *                  partial sums are added in registers with round-to-nearest: below 1e-5 * sum_k|a.b| for ANY data and
 *                  any K.  For K <= 2048 it is the single accumulator.
 *   FP8_ACC_FAST   one accumulator over all of K, 2.5-4 % faster at K = 4096 .. 49152.  The error is below
 *                  1e-5 * sum_k|a.b| for K <= 2048 on any data; on products of mixed sign (training tensors: zero-mean
 *                  weights and gradients) it grows slowly with K (measured 1.4e-7 at K = 49152 on the workloads'
 *                  tensors, 1.2e-5 at K = 2^20 on heavy-tailed codes); products that all share one sign lose up to
 *                  (K/32) * 2^-23 of their sum (measured 3.7-5.3e-5 at K = 49152).  For callers who know their operands.
 * Every GEMM entry point that takes this descriptor honours `acc`; other values give FP8_ERR_ENUM.
 * Reproducibility: a call is bit-reproducible for a given problem (shapes, layouts, data) on a given device.  The
 * order in which the K-blocks of an output tile are accumulated (from the start or from the end of K) depends on
 * the tile's place in the kernel's schedule, so two equal dot products in different tiles may differ in the last
 * bits, within the stated tolerance.
 */
typedef struct {
    int64_t M, N, K;
    fp8_format fa, fb;
    fp8_major ma, mb;
    int64_t lda, ldb, ldd;
    fp8_wide out;
    fp8_accumulate acc;
} fp8_gemm_desc;

fp8_status fp8_gemm(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, void* D,
                    const float* scale_inv_a_dev, const float* scale_inv_b_dev,
                    float* amax_d_dev, void* stream);

/*
 * fp8_gemm_fp8out — Section 2: operations on FP8 inputs produce higher-precision results, which may
 * be converted to FP8 before they are written to memory.  Same contraction as fp8_gemm, but the
 * epilogue converts instead of storing a wide value:
 *   v[i,j] = (sum_k decode_fa(A[i,k]) * decode_fb(B[k,j])) * (sa_inv * sb_inv)      (binary32)
 *   D[i,j] = encode_fd( v[i,j] * scale_d )       conversion rules of fp8_quantize (RNE, specials, `od`)
 *   *amax_d_dev = amax over v, i.e. BEFORE the output scale and the conversion: it is the quantity the
 *                 next scale factor for this tensor is chosen from (scale_d itself comes from an earlier
 *                 step, as the scale-history recipes the paper leaves to software do).
 *   D            M x N codes, D[i,j] at D[i*ldd + j]; d->out is ignored; D and ldd 16-byte aligned.
 *   scale_d_dev  device float.
 * Everything else (operands, layouts, alignment, edge cases) as fp8_gemm.
 */
fp8_status fp8_gemm_fp8out(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, uint8_t* D,
                           fp8_format fd, fp8_overflow od,
                           const float* scale_inv_a_dev, const float* scale_inv_b_dev, const float* scale_d_dev,
                           float* amax_d_dev, void* stream);

/*
 * fp8_quantize_transpose — Sections 3 and 4.1: the same FP8 tensor is consumed by two matrix multiplies
 * that contract over different axes (an activation by the forward product and by the weight-gradient
 * product, an output gradient by both backward products), so its codes are produced once in both
 * orientations:
 *   code(r,c) = encode_f( binary32(x[r*ldx + c]) * scale )        conversion rules of fp8_quantize
 *   out  [r*ldo + c] = code(r,c)        (rows x cols; `out` may be NULL: transposed copy only)
 *   out_t[c*ldt + r] = code(r,c)        (cols x rows)
 *   *amax_dev (nullable) OVERWRITTEN with amax of x, same pass (definition of fp8_amax).
 * x is rows x cols, row-major, pitch ldx elements; ldo >= cols, ldt >= rows (bytes), else FP8_ERR_SHAPE.
 * One pass: 128 x 128 tiles, transposed through shared memory, every global access a full 128-byte line.
 * The tiled path needs rows and cols multiples of 4, x aligned to 4 elements with ldx a multiple of 4, and
 * out / out_t / ldo / ldt multiples of 4 bytes; anything else takes an element-wise kernel with identical
 * results.  rows*cols == 0 is a no-op (amax = 0).
 */
fp8_status fp8_quantize_transpose(const void* x, fp8_wide t, int64_t rows, int64_t cols, int64_t ldx,
                                  fp8_format f, fp8_overflow o, const float* scale_dev,
                                  uint8_t* out, int64_t ldo, uint8_t* out_t, int64_t ldt,
                                  float* amax_dev, void* stream);

/*
 * Per-channel scale factors — Section 4.2: post-training quantization scales weights channel by channel and
 * activations with one factor per tensor.  A channel is a row or a column of a 2-D tensor
 * x (rows x cols, row-major, pitch ld elements): axis 0 = one channel per column, axis 1 = one per row.
 *
 * fp8_amax_channels      amax_vec[c] = amax over channel c (definition of fp8_amax), OVERWRITTEN.
 * fp8_scales_from_amax   `count` scale factors at once, arithmetic of fp8_scale_from_amax; pow2 != 0 gives
 *                        the power-of-two scales of fp8_scale_pow2_from_amax.
 * fp8_quantize_channels  out[r*ld_out + c] = encode_f( binary32(x[r*ld + c]) * scale_vec[channel of (r,c)] ),
 *                        conversion rules of fp8_quantize.
 * Fast paths need 16-byte aligned rows (base and pitch); anything else takes element-wise kernels with
 * identical results.
 */
fp8_status fp8_amax_channels(const void* x, fp8_wide t, int64_t rows, int64_t cols, int64_t ld, int axis,
                             float* amax_vec_dev, void* stream);
fp8_status fp8_scales_from_amax(const float* amax_vec_dev, int64_t count, fp8_format f, int pow2,
                                float* scale_vec_dev, float* scale_inv_vec_dev, void* stream);
fp8_status fp8_quantize_channels(const void* x, fp8_wide t, int64_t rows, int64_t cols, int64_t ld, int axis,
                                 fp8_format f, fp8_overflow o, const float* scale_vec_dev,
                                 uint8_t* out, int64_t ld_out, void* stream);

/*
 * fp8_gemm_channel_scales — fp8_gemm for a B operand (the weights) quantized with per-channel scales:
 *   D[i,j] = round_out( (sum_k decode(A[i,k]) * decode(B[k,j])) * (sa_inv * sb_inv_vec[j]) )
 * scale_inv_b_vec_dev holds N device floats, one per column j of B (per output channel).  A keeps its
 * per-tensor inverse scale.  Everything else as fp8_gemm.
 */
fp8_status fp8_gemm_channel_scales(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, void* D,
                                   const float* scale_inv_a_dev, const float* scale_inv_b_vec_dev,
                                   float* amax_d_dev, void* stream);

/*
 * fp8_gemm_batched — Section 4.2 quantizes the inputs of every matrix multiply, the batched
 * products of attention among them.  `batch` independent products with the same shape, layouts,
 * formats and per-tensor scales (one scale for the whole batched tensor), in one launch:
 *   D_b = (A_b . B_b) * (sa_inv * sb_inv),   A_b = A + b*stride_a, B_b = B + b*stride_b, D_b = D + b*stride_d
 * Strides are in elements of the respective tensor and 16-byte aligned (in bytes).  The members of D lie at
 * least one whole matrix apart (they are written); the members of A and of B are only read, so any positive
 * stride is accepted: members may interleave (heads stored side by side inside a row, slices of K of one
 * matrix) or overlap.  amax_d_dev (optional) receives the amax over all batch members.  batch == 0 is a no-op
 * (amax = 0); batch <= 65535.  Everything else as fp8_gemm.
 */
fp8_status fp8_gemm_batched(const fp8_gemm_desc* d, int64_t batch,
                            const uint8_t* A, int64_t stride_a, const uint8_t* B, int64_t stride_b,
                            void* D, int64_t stride_d,
                            const float* scale_inv_a_dev, const float* scale_inv_b_dev,
                            float* amax_d_dev, void* stream);

/*
 * fp8_gemm_splitk — fp8_gemm for problems with few output tiles and a long contraction (a weight-bandwidth-
 * bound product of a few rows with a wide weight matrix): K is cut into `splits` slices that run as members of
 * one batched launch, each writing an fp32 partial product (already multiplied by sa_inv * sb_inv) into the
 * caller's workspace, and a second kernel adds the partials in slice order, rounds to `out` and records amax.
 *   D[i,j] = round_out( sum_s fl32( (sum_{k in slice s} a.b) * (sa_inv * sb_inv) ) )
 * Same tolerance as fp8_gemm (the extra binary32 roundings are ~1e-7 relative).  Deterministic.
 * fp8_gemm_splitk_workspace reports, for a descriptor, the number of slices the library will use on the
 * current device and the workspace it needs: splits = 1 (bytes = 0) whenever a cost model of the kernel (operand
 * bytes over min(tiles x 90 GB/s, HBM), plus the second launch and the partials) predicts less than 15 % gain,
 * K < 2048, N is not a multiple of 4, or K does not divide into slices that are multiples of 256; then
 * fp8_gemm_splitk is exactly fp8_gemm.  Otherwise splits is a power of two up to 16 and
 * bytes = splits * M * N * 4.  workspace_dev: 16-byte aligned device memory of at least that size (else
 * FP8_ERR_ALIGN / FP8_ERR_SHAPE), owned by the caller, contents undefined afterwards.  With splits > 1, D needs
 * only element alignment and ldd >= N.
 */
fp8_status fp8_gemm_splitk_workspace(const fp8_gemm_desc* d, int* splits_out, size_t* bytes_out);
fp8_status fp8_gemm_splitk(const fp8_gemm_desc* d, const uint8_t* A, const uint8_t* B, void* D,
                           const float* scale_inv_a_dev, const float* scale_inv_b_dev, float* amax_d_dev,
                           void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * fp8_async_status — reads and clears the device-side error latch of the
 * current device (synchronises the device).  FP8_OK, or FP8_ERR_TIMEOUT if a
 * kernel gave up on a bounded wait since the last call; *detail (optional, host
 * pointer) receives a code naming the wait.  Not part of the paper: it exists
 * so that a pipeline fault ends in an error code instead of a hung GPU.
 */
fp8_status fp8_async_status(uint32_t* detail);

/*
 * fp8_self_test_expire_wait — the paper has no counterpart; a self-test of the library's safety net.  Every
 * device-side wait in the library (the mbarrier waits of the GEMM pipeline, the grid barrier of
 * fp8_quantize_current) counts SM clocks and gives up after a limit, so that a pipeline fault ends in
 * FP8_ERR_TIMEOUT instead of a hung GPU.  This call makes one such wait run out ON PURPOSE, in a way that
 * cannot hang or fault: it launches a small kernel whose wait can never be satisfied and whose limit is
 * `limit_cycles` SM clocks (1 .. 2e9, i.e. at most about a second; FP8_ERR_UNSUPPORTED otherwise).
 *   FP8_WAIT_MBARRIER      one block waits on an mbarrier nobody arrives on, through the same bounded-wait
 *                          routine the GEMM roles use; detail code 9.
 *   FP8_WAIT_GRID_BARRIER  the fp8_quantize_current kernel runs on an empty tensor with its grid barrier told to
 *                          expect one block more than the grid has: every block gives up, nothing is written, the
 *                          control words (those of fp8_quantize_current_static) are left zeroed; detail code 16.
 * Afterwards fp8_async_status returns FP8_ERR_TIMEOUT once, with the detail code above, then FP8_OK again;
 * the stream and the library remain fully usable.
 */
typedef enum { FP8_WAIT_MBARRIER = 0, FP8_WAIT_GRID_BARRIER = 1 } fp8_wait_kind;
fp8_status fp8_self_test_expire_wait(int which, uint64_t limit_cycles, void* stream);

/*
 * fp8_sm_clock_probe — the paper has no counterpart; a measurement aid.  Launches a one-warp kernel that reads the SM
 * cycle counter and the device's nanosecond timer, waits `duration_us` microseconds (1 .. 100000, else
 * FP8_ERR_UNSUPPORTED; the wait is bounded by an iteration count as well) and reads both again.
 *   out_dev  device, two 64-bit words, OVERWRITTEN: [0] = SM clocks elapsed, [1] = nanoseconds elapsed;
 *            clocks * 1000 / nanoseconds = SM clock in MHz during the window.
 * Enqueued on a second stream it runs beside other kernels (it needs one warp and no shared memory), which is how the
 * benchmark reads the clock the tensor cores actually ran at under the power cap: the management interface samples
 * too coarsely for that.
 */
fp8_status fp8_sm_clock_probe(uint64_t* out_dev, uint32_t duration_us, void* stream);

/* Human-readable name of a status code (static storage, never NULL). */
const char* fp8_status_string(fp8_status s);

/* Number of kernel launches (and memset nodes) the library has enqueued since
 * it was loaded; host-side counter used by benchmarks to report launch counts. */
uint64_t fp8_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* FP8_B200_H */
