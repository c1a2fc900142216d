// Per-tensor, per-node 8-bit quantizer: a range reduction followed by a
// scale-and-round pass (Section 3, "Low Precision Training").  Both passes are
// HBM-bound streaming kernels: 16-byte loads, warp-shuffle reduction of the
// range, one atomic per block; the second pass stores 4 codes per thread.
#include <atomic>
#include "common.cuh"

namespace lpdt {

// ---- Philox4x32-10 (Salmon et al., SC'11), from the published round function.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}
__device__ __forceinline__ float u24(uint32_t r) { return __uint2float_rn(r >> 8) * 0x1p-24f; }

// ws[2*node] = bits of max(0, max x) or of max|x|; ws[2*node+1] = bits of -min(0, min x).
// Non-negative floats order like their bit patterns, so atomicMax on uint works.
template <bool AFFINE, bool VEC>
__global__ void range_kernel(const float *__restrict__ x, int64_t n, int64_t stride,
                             uint32_t *__restrict__ ws) {
    pdl_enter();
    const int node = blockIdx.y;
    const float *xn = x + (int64_t)node * stride;
    float hi = 0.f, nlo = 0.f;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nth = (int64_t)gridDim.x * blockDim.x;
    if (VEC) {
        const float4 *x4 = reinterpret_cast<const float4 *>(xn);
        for (int64_t i = tid; i < n / 4; i += nth) {
            float4 v = __ldg(x4 + i);
            if (AFFINE) {
                hi = fmaxf(hi, fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)));
                nlo = fmaxf(nlo, -fminf(fminf(v.x, v.y), fminf(v.z, v.w)));
            } else {
                hi = fmaxf(hi, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
            }
        }
    } else {
        for (int64_t i = tid; i < n; i += nth) {
            float v = xn[i];
            if (AFFINE) { hi = fmaxf(hi, v); nlo = fmaxf(nlo, -v); }
            else hi = fmaxf(hi, fabsf(v));
        }
    }
    hi = warp_max(hi);
    if (AFFINE) nlo = warp_max(nlo);
    __shared__ float s_hi[32], s_lo[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { s_hi[warp] = hi; s_lo[warp] = nlo; }
    __syncthreads();
    if (warp == 0) {
        const int nw = blockDim.x >> 5;
        hi = lane < nw ? s_hi[lane] : 0.f;
        nlo = lane < nw ? s_lo[lane] : 0.f;
        hi = warp_max(hi);
        if (AFFINE) nlo = warp_max(nlo);
        if (lane == 0) {
            atomicMax(ws + 2 * node, __float_as_uint(hi));
            if (AFFINE) atomicMax(ws + 2 * node + 1, __float_as_uint(nlo));
        }
    }
}

struct SymParams { float inv; };

__device__ __forceinline__ int q_sym_rne(float x, float inv) {
    float r = rintf(__fmul_rn(x, inv));
    r = fminf(fmaxf(r, -127.f), 127.f);
    return (int)r;
}
__device__ __forceinline__ int q_sym_sr(float x, float inv, float u) {
    float t = __fmul_rn(x, inv);
    float fl = floorf(t);
    float f = __fsub_rn(t, fl);
    float r = fl + ((u < f) ? 1.f : 0.f);
    r = fminf(fmaxf(r, -127.f), 127.f);
    return (int)r;
}
__device__ __forceinline__ int q_affine(float x, float s, float zf) {
    float r = __fadd_rn(rintf(__fdiv_rn(x, s)), zf);
    r = fminf(fmaxf(r, 0.f), 255.f);
    return (int)r;
}

template <int MODE /*0 sym rne, 1 sym stochastic, 2 affine*/, bool VEC>
__global__ void quantize_kernel(const float *__restrict__ x, int64_t n, int64_t stride,
                                const uint32_t *__restrict__ ws, int8_t *__restrict__ q,
                                float *__restrict__ scale, int32_t *__restrict__ zero_point,
                                uint2 key, uint32_t ctr_offset, int wstride) {
    pdl_enter();
    const int node = blockIdx.y;
    const float *xn = x + (int64_t)node * stride;
    int8_t *qn = q + (int64_t)node * n;
    float s, inv = 0.f, zf = 0.f;
    if (MODE == 2) {
        const float hi = __uint_as_float(ws[wstride * node]);
        const float lo = -__uint_as_float(ws[wstride * node + 1]);
        s = (hi == lo) ? 1.f : __fdiv_rn(__fsub_rn(hi, lo), 255.f);
        zf = rintf(__fdiv_rn(-lo, s));
        zf = fminf(fmaxf(zf, 0.f), 255.f);
    } else {
        const float amax = __uint_as_float(ws[wstride * node]);
        if (amax == 0.f) { s = 1.f; inv = 0.f; }
        else { s = __fdiv_rn(amax, 127.f); inv = __fdiv_rn(127.f, amax); }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        scale[node] = s;
        if (MODE == 2) zero_point[node] = (int)zf;
    }
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t nth = (int64_t)gridDim.x * blockDim.x;
    if (VEC) {
        const float4 *x4 = reinterpret_cast<const float4 *>(xn);
        char4 *q4 = reinterpret_cast<char4 *>(qn);
        for (int64_t i = tid; i < n / 4; i += nth) {
            float4 v = __ldg(x4 + i);
            int a, b, c, d;
            if (MODE == 0) {
                a = q_sym_rne(v.x, inv); b = q_sym_rne(v.y, inv);
                c = q_sym_rne(v.z, inv); d = q_sym_rne(v.w, inv);
            } else if (MODE == 1) {
                uint4 r = philox4x32_10(make_uint4((uint32_t)i, (uint32_t)((uint64_t)i >> 32),
                                                   (uint32_t)node, ctr_offset), key);
                a = q_sym_sr(v.x, inv, u24(r.x)); b = q_sym_sr(v.y, inv, u24(r.y));
                c = q_sym_sr(v.z, inv, u24(r.z)); d = q_sym_sr(v.w, inv, u24(r.w));
            } else {
                a = q_affine(v.x, s, zf); b = q_affine(v.y, s, zf);
                c = q_affine(v.z, s, zf); d = q_affine(v.w, s, zf);
            }
            q4[i] = make_char4((signed char)a, (signed char)b, (signed char)c, (signed char)d);
        }
    } else {
        for (int64_t i = tid; i < n; i += nth) {
            float v = xn[i];
            int a;
            if (MODE == 0) a = q_sym_rne(v, inv);
            else if (MODE == 1) {
                uint4 r = philox4x32_10(make_uint4((uint32_t)(i >> 2), (uint32_t)((uint64_t)i >> 34),
                                                   (uint32_t)node, ctr_offset), key);
                uint32_t w = (i & 3) == 0 ? r.x : (i & 3) == 1 ? r.y : (i & 3) == 2 ? r.z : r.w;
                a = q_sym_sr(v, inv, u24(w));
            } else a = q_affine(v, s, zf);
            qn[i] = (int8_t)a;
        }
    }
}

template <bool AFFINE>
__global__ void dequantize_kernel(const int8_t *__restrict__ q, int64_t n,
                                  const float *__restrict__ scale,
                                  const int32_t *__restrict__ zp, float *__restrict__ y,
                                  int64_t ystride) {
    pdl_enter();
    const int node = blockIdx.y;
    const float s = scale[node];
    const int z = AFFINE ? zp[node] : 0;
    const int64_t base = (int64_t)node * n;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n;
         i += (int64_t)gridDim.x * blockDim.x) {
        int code = AFFINE ? (int)(uint8_t)q[base + i] - z : (int)q[base + i];
        y[(int64_t)node * ystride + i] = __fmul_rn(__int2float_rn(code), s);
    }
}

static int blocks_for(int64_t work_items, int nodes) {
    int64_t b = ceil_div(work_items, 256 * 4);
    int64_t cap = ceil_div((int64_t)kNumSMs * 8, nodes);
    if (b > cap) b = cap;
    if (b < 1) b = 1;
    return (int)b;
}

}  // namespace lpdt

using namespace lpdt;

extern "C" size_t lpdt_quantize_workspace_size(int32_t nodes) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * 2 * sizeof(uint32_t), 256);
}

extern "C" lpdt_status lpdt_quantize(const float *x, int32_t nodes, int64_t n, int64_t x_node_stride,
                                     lpdt_qmode mode, lpdt_round rounding, uint64_t seed,
                                     uint32_t ctr_offset, int8_t *q, float *scale,
                                     int32_t *zero_point, void *ws, size_t ws_bytes, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && n >= 0);
    if (nodes == 0 || n == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && q && scale);
    LPDT_CHECK_ARG(x_node_stride >= n || nodes == 1);
    LPDT_CHECK_ARG(mode == LPDT_SYM_S8 || mode == LPDT_AFFINE_U8);
    LPDT_CHECK_ARG(rounding == LPDT_ROUND_NEAREST_EVEN || rounding == LPDT_ROUND_STOCHASTIC);
    LPDT_CHECK_ARG(aligned(x, 4) && aligned(scale, 4));
    if (mode == LPDT_AFFINE_U8) {
        LPDT_CHECK_ARG(zero_point != nullptr);
        if (rounding != LPDT_ROUND_NEAREST_EVEN) return LPDT_ERR_UNSUPPORTED;
    }
    if (nodes > 65535) return LPDT_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < lpdt_quantize_workspace_size(nodes)) return LPDT_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    uint32_t *w = (uint32_t *)ws;
    LPDT_CUDA(cudaMemsetAsync(w, 0, (size_t)nodes * 2 * sizeof(uint32_t), st));
    const bool vec = aligned(x, 16) && (x_node_stride % 4 == 0) && (n % 4 == 0) && aligned(q, 4);
    dim3 grid(blocks_for(vec ? n / 4 : n, nodes), nodes), block(256);
    const uint2 key = make_uint2((uint32_t)seed, (uint32_t)(seed >> 32));
    if (mode == LPDT_AFFINE_U8) {
        if (vec) launch_k(range_kernel<true, true>, grid, block, 0, st, x, n, x_node_stride, w);
        else launch_k(range_kernel<true, false>, grid, block, 0, st, x, n, x_node_stride, w);
        LPDT_LAUNCH_CHECK();
        if (vec) launch_k(quantize_kernel<2, true>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, zero_point, key, ctr_offset, 2);
        else launch_k(quantize_kernel<2, false>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, zero_point, key, ctr_offset, 2);
    } else {
        if (vec) launch_k(range_kernel<false, true>, grid, block, 0, st, x, n, x_node_stride, w);
        else launch_k(range_kernel<false, false>, grid, block, 0, st, x, n, x_node_stride, w);
        LPDT_LAUNCH_CHECK();
        if (rounding == LPDT_ROUND_NEAREST_EVEN) {
            if (vec) launch_k(quantize_kernel<0, true>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, zero_point, key, ctr_offset, 2);
            else launch_k(quantize_kernel<0, false>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, zero_point, key, ctr_offset, 2);
        } else {
            if (vec) launch_k(quantize_kernel<1, true>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, zero_point, key, ctr_offset, 2);
            else launch_k(quantize_kernel<1, false>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, zero_point, key, ctr_offset, 2);
        }
    }
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_dequantize(const int8_t *q, int32_t nodes, int64_t n, const float *scale,
                                       const int32_t *zero_point, float *y, int64_t y_node_stride,
                                       void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && n >= 0);
    if (nodes == 0 || n == 0) return LPDT_OK;
    LPDT_CHECK_ARG(q && scale && y && nodes <= 65535 && (y_node_stride >= n || nodes == 1));
    dim3 grid(blocks_for(n, nodes), nodes), block(256);
    if (zero_point) launch_k(dequantize_kernel<true>, grid, block, 0, as_stream(stream), q, n, scale, zero_point, y, y_node_stride);
    else launch_k(dequantize_kernel<false>, grid, block, 0, as_stream(stream), q, n, scale, zero_point, y, y_node_stride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_quantize_with_range(const float *x, int32_t nodes, int64_t n, int64_t x_node_stride,
                                                const float *amax, lpdt_round rounding, uint64_t seed,
                                                uint32_t ctr_offset, int8_t *q, float *scale, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && n >= 0);
    if (nodes == 0 || n == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && q && scale && amax);
    LPDT_CHECK_ARG(x_node_stride >= n || nodes == 1);
    LPDT_CHECK_ARG(rounding == LPDT_ROUND_NEAREST_EVEN || rounding == LPDT_ROUND_STOCHASTIC);
    LPDT_CHECK_ARG(aligned(x, 4) && aligned(scale, 4) && aligned(amax, 4));
    if (nodes > 65535) return LPDT_ERR_UNSUPPORTED;
    cudaStream_t st = as_stream(stream);
    const uint32_t *w = reinterpret_cast<const uint32_t *>(amax);      // non-negative floats, read as bit patterns
    const bool vec = aligned(x, 16) && (x_node_stride % 4 == 0) && (n % 4 == 0) && aligned(q, 4);
    dim3 grid(blocks_for(vec ? n / 4 : n, nodes), nodes), block(256);
    const uint2 key = make_uint2((uint32_t)seed, (uint32_t)(seed >> 32));
    if (rounding == LPDT_ROUND_NEAREST_EVEN) {
        if (vec) launch_k(quantize_kernel<0, true>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, nullptr, key, ctr_offset, 1);
        else launch_k(quantize_kernel<0, false>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, nullptr, key, ctr_offset, 1);
    } else {
        if (vec) launch_k(quantize_kernel<1, true>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, nullptr, key, ctr_offset, 1);
        else launch_k(quantize_kernel<1, false>, grid, block, 0, st, x, n, x_node_stride, w, q, scale, nullptr, key, ctr_offset, 1);
    }
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

// ---------------------------------------------------------------------------
// Quantizer for callers that own no device scratch.
//
// lpdt_quantize needs a few bytes of caller-provided scratch for the per-node
// range words.  Some users of this library cannot supply any: an edge-device
// training loop that was given a fixed set of buffers at start-up and has no
// allocator afterwards, or a plug-in called from a host application whose device
// memory belongs to that application's own pool and which forbids device
// allocation on its hot path (cudaMalloc also synchronises the whole device).
// For them the range words live in the array below, which is part of the loaded
// library image: every GPU that loads the library holds these 8 KB until the
// process exits.
//
// In host code `g_static_range_words` is only a handle for the symbol, not a device
// address, so its address on the current device is looked up once per device with
// cudaGetSymbolAddress and that pointer is what the kernels receive.
constexpr int kStaticMaxNodes = LPDT_QUANTIZE_STATIC_MAX_NODES;
static __device__ __align__(256) uint32_t g_static_range_words[2 * kStaticMaxNodes];

// One cached address per device ordinal.  Two host threads that both make the first call on a device
// look the same address up and store the same value (an atomic pointer store), so the race is benign.
// The cache does not outlive a cudaDeviceReset: after one, the library must be reloaded.
constexpr int kMaxDevices = 64;
static std::atomic<uint32_t *> g_static_range_ptr[kMaxDevices];

static lpdt_status static_range_words(uint32_t **out) {
    int dev = -1;
    LPDT_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return LPDT_ERR_UNSUPPORTED;
    uint32_t *p = g_static_range_ptr[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress((void **)&p, g_static_range_words) != cudaSuccess || !p) {
            (void)cudaGetLastError();
            return LPDT_ERR_CUDA;
        }
        g_static_range_ptr[dev].store(p, std::memory_order_release);
    }
    *out = p;
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_quantize_static(const float *x, int32_t nodes, int64_t n_per_node,
                                            int64_t x_node_stride, lpdt_qmode mode, lpdt_round rounding,
                                            uint64_t seed, uint32_t ctr_offset, int8_t *q, float *scale,
                                            int32_t *zero_point, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && n_per_node >= 0);
    if (nodes > kStaticMaxNodes) return LPDT_ERR_WORKSPACE;     // the built-in scratch holds 1024 nodes
    if (nodes == 0 || n_per_node == 0) return LPDT_OK;          // nothing to do: no address lookup either
    uint32_t *words = nullptr;
    lpdt_status s = static_range_words(&words);
    if (s != LPDT_OK) return s;
    // Same two passes as lpdt_quantize; it zeroes the words it uses before the range pass,
    // so whatever the previous call left in the array does not matter.
    return lpdt_quantize(x, nodes, n_per_node, x_node_stride, mode, rounding, seed, ctr_offset, q, scale,
                         zero_point, words, sizeof(uint32_t) * 2 * kStaticMaxNodes, stream);
}

// ---------------------------------------------------------------------------
// Batched symmetric quantization of many small tensors that live inside one flat
// per-node parameter vector (all layer weights of a network): two launches in
// total instead of two per tensor.
namespace lpdt {

constexpr int kMaxBatchTensors = 64;
struct QuantBatch {
    int count;
    long long src_off[kMaxBatchTensors];    // element offset inside a node's parameter row
    long long size[kMaxBatchTensors];       // elements per node
    long long dst_off[kMaxBatchTensors];    // byte offset of the tensor's [nodes][size] block in q
};

// grid = (blocks, nodes, tensors); blocks beyond a tensor's length fall through
__global__ void batch_range_kernel(const float *__restrict__ params, long long row_stride, QuantBatch qb,
                                   uint32_t *__restrict__ ws) {
    pdl_enter();
    const int t = blockIdx.z, node = blockIdx.y;
    const long long n = qb.size[t];
    const float *x = params + (long long)node * row_stride + qb.src_off[t];
    float m = 0.f;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        m = fmaxf(m, fabsf(x[i]));
    if ((long long)blockIdx.x * blockDim.x >= n) return;
    block_amax_to(m, reinterpret_cast<float *>(ws + (size_t)t * gridDim.y + node));
}

__global__ void batch_quantize_kernel(const float *__restrict__ params, long long row_stride, QuantBatch qb,
                                      const uint32_t *__restrict__ ws, int8_t *__restrict__ q,
                                      float *__restrict__ scales) {
    pdl_enter();
    const int t = blockIdx.z, node = blockIdx.y, nodes = gridDim.y;
    const long long n = qb.size[t];
    const float *x = params + (long long)node * row_stride + qb.src_off[t];
    int8_t *dst = q + qb.dst_off[t] + (long long)node * n;
    const float amax = __uint_as_float(ws[(size_t)t * nodes + node]);
    float s = 1.f, inv = 0.f;
    if (amax != 0.f) { s = __fdiv_rn(amax, 127.f); inv = __fdiv_rn(127.f, amax); }
    if (blockIdx.x == 0 && threadIdx.x == 0) scales[(size_t)t * nodes + node] = s;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        dst[i] = (int8_t)q_sym_rne(x[i], inv);
}

}  // namespace lpdt

extern "C" size_t lpdt_quantize_batch_workspace_size(int32_t nodes, int32_t n_tensors) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)(n_tensors > 0 ? n_tensors : 1) * sizeof(uint32_t), 256);
}

extern "C" lpdt_status lpdt_quantize_batch(const float *params, int32_t nodes, int64_t row_stride, int32_t n_tensors,
                                           const int64_t *src_offsets, const int64_t *sizes,
                                           const int64_t *dst_offsets, int8_t *q, float *scales, void *ws,
                                           size_t ws_bytes, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && n_tensors >= 0);
    if (nodes == 0 || n_tensors == 0) return LPDT_OK;
    LPDT_CHECK_ARG(params && src_offsets && sizes && dst_offsets && q && scales);
    if (n_tensors > kMaxBatchTensors || nodes > 65535) return LPDT_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < lpdt_quantize_batch_workspace_size(nodes, n_tensors)) return LPDT_ERR_WORKSPACE;
    QuantBatch qb;
    qb.count = n_tensors;
    long long longest = 0;
    for (int t = 0; t < n_tensors; ++t) {
        LPDT_CHECK_ARG(src_offsets[t] >= 0 && sizes[t] >= 0 && dst_offsets[t] >= 0 && src_offsets[t] + sizes[t] <= row_stride);
        qb.src_off[t] = src_offsets[t]; qb.size[t] = sizes[t]; qb.dst_off[t] = dst_offsets[t];
        if (sizes[t] > longest) longest = sizes[t];
    }
    if (longest == 0) return LPDT_OK;
    cudaStream_t st = as_stream(stream);
    uint32_t *w = (uint32_t *)ws;
    LPDT_CUDA(cudaMemsetAsync(w, 0, (size_t)nodes * n_tensors * sizeof(uint32_t), st));
    int bx = (int)ceil_div(longest, 256 * 8);
    if (bx > 64) bx = 64;
    if (bx < 1) bx = 1;
    dim3 grid(bx, nodes, n_tensors);
    launch_k(batch_range_kernel, grid, 256, 0, st, params, row_stride, qb, w);
    LPDT_LAUNCH_CHECK();
    launch_k(batch_quantize_kernel, grid, 256, 0, st, params, row_stride, qb, w, q, scales);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
