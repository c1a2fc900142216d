// Shared host/device helpers of the lpdt CUDA library (not part of the ABI).
#pragma once
#include <cuda_runtime.h>
#include <atomic>
#include <stdint.h>
#include <stdlib.h>
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

// Name of the contraction kernel the calling host thread launched last (lpdt_last_kernel): lets a
// caller that times a call label the number with the kernel that actually ran.
inline thread_local const char *g_last_kernel = "";
// Kernels the calling host thread has enqueued through this library so far (lpdt_launch_count).
inline thread_local unsigned long long g_launch_count = 0;

// A kernel attribute (the opt-in dynamic shared memory limit) belongs to the device it was set on, so
// "already set" is remembered per device ordinal: one bit per device, devices beyond 63 set it every call.
struct PerDeviceOnce {
    std::atomic<unsigned long long> done{0};
    // true when the attribute still has to be set on the current device; *dev receives its ordinal
    bool pending(int *dev) {
        *dev = -1;
        if (cudaGetDevice(dev) != cudaSuccess || *dev < 0 || *dev >= 64) return true;
        return !((done.load(std::memory_order_acquire) >> *dev) & 1ull);
    }
    void mark(int dev) {
        if (dev >= 0 && dev < 64) done.fetch_or(1ull << dev, std::memory_order_release);
    }
};

// Programmatic dependent launch.  Every kernel of the library waits for the grids before it
// in the stream (griddepcontrol.wait returns once they have completed and their writes are
// visible) before it touches global memory, and then allows the grid after it to be scheduled.
// Launched through launch_k, a kernel's launch latency and its prologue (barrier set-up,
// tensor-memory allocation, descriptor prefetch) overlap the tail of its predecessor; stream
// order of every global access is unchanged.  LPDT_NO_PDL=1 launches without the attribute
// (the instructions are then no-ops).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_wait(); pdl_trigger(); }

static inline bool pdl_enabled() {
    static int on = -1;
    if (on < 0) { const char *e = getenv("LPDT_NO_PDL"); on = (e && e[0] == '1') ? 0 : 1; }
    return on == 1;
}

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                   Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl_enabled() ? 1 : 0;
    ++g_launch_count;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args &&>(args)...);
}

// The same with a thread-block cluster of `cluster_x` CTAs along x (grid.x must be a multiple of it).
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_k_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                           int cluster_x, Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[2];
    unsigned n = 0;
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = (unsigned)cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
        ++n;
    }
    if (pdl_enabled()) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    ++g_launch_count;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args &&>(args)...);
}

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
