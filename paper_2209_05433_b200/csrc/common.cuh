// Shared host/device plumbing of the fp8_b200 library: status latch, launch
// counter, device properties, small PTX wrappers.  No FP8 arithmetic here.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/fp8_b200.h"

namespace fp8b200 {

// ---- host side -------------------------------------------------------------

// Number of SMs of the current device (cached per device id).
int sm_count();

// Adds to the library-wide count of enqueued kernels / memset nodes.
void count_launches(int n);

// cudaGetLastError() folded into a status code.
inline fp8_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? FP8_OK : FP8_ERR_CUDA;
}

// Launch with programmatic stream serialization: the kernel may be scheduled while its predecessor in the
// stream is still draining (once every block of the predecessor has signalled or exited).  Such a kernel must
// execute grid_dependency_wait() before it touches memory an earlier kernel may still be writing.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_programmatic(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- device side -----------------------------------------------------------

// Blocks until every earlier kernel of the stream has completed and its writes are visible (no-op when the
// kernel was launched without programmatic serialization).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel of the stream be scheduled: called once a block has issued its last load.
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ uint32_t ld_nc_u32(const void* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}

__device__ __forceinline__ uint2 ld_nc_v2(const void* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Maximum over the warp of an unsigned value (redux.sync).
__device__ __forceinline__ uint32_t warp_max_u32(uint32_t v) {
    return __reduce_max_sync(0xFFFFFFFFu, v);
}

// Folds a magnitude bit pattern that is a NaN (above the infinity pattern) onto
// the one canonical NaN, so that an integer maximum propagates NaN.
__device__ __forceinline__ uint32_t canonical_nan_bits(uint32_t abs_bits) {
    return abs_bits > 0x7F800000u ? 0x7FC00000u : abs_bits;
}

// Block-wide maximum, then one atomicMax on the caller's float (as bits).
// Every thread of the block must call it; smem holds >= 32 words.
__device__ __forceinline__ void block_atomic_max_bits(uint32_t v, uint32_t* smem, uint32_t* out_bits) {
    v = warp_max_u32(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) smem[warp] = v;
    __syncthreads();
    if (warp == 0) {
        const int nwarps = (blockDim.x + 31) >> 5;
        uint32_t w = lane < nwarps ? smem[lane] : 0u;
        w = warp_max_u32(w);
        if (lane == 0 && w != 0u) atomicMax(out_bits, w);
    }
}

}  // namespace fp8b200
