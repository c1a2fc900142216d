// Shared host/device helpers of the lpdt CUDA library (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/lpdt.h"

#define LPDT_CHECK_ARG(cond)                       \
    do {                                           \
        if (!(cond)) return LPDT_ERR_INVALID_ARG;  \
    } while (0)

#define LPDT_CUDA(call)                                   \
    do {                                                  \
        if ((call) != cudaSuccess) return LPDT_ERR_CUDA;  \
    } while (0)

#define LPDT_LAUNCH_CHECK()                                       \
    do {                                                          \
        if (cudaPeekAtLastError() != cudaSuccess) {               \
            (void)cudaGetLastError();                             \
            return LPDT_ERR_CUDA;                                 \
        }                                                         \
    } while (0)

namespace lpdt {

static inline bool aligned(const void *p, size_t a) { return ((uintptr_t)p % a) == 0; }
static inline cudaStream_t as_stream(void *s) { return (cudaStream_t)s; }
static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

constexpr int kNumSMs = 148;  // B200

// double atomicAdd is native on sm_60+
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Block-wide max of non-negative values, then one atomicMax on the float's bit pattern
// (non-negative floats order like unsigned integers).  Every thread of the block must call.
__device__ __forceinline__ void block_amax_to(float v, float *dst) {
    __shared__ float s_blk_amax[32];
    v = warp_max(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) s_blk_amax[warp] = v;
    __syncthreads();
    if (warp == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        v = lane < nw ? s_blk_amax[lane] : 0.f;
        v = warp_max(v);
        if (lane == 0) atomicMax(reinterpret_cast<unsigned int *>(dst), __float_as_uint(v));
    }
}

}  // namespace lpdt
