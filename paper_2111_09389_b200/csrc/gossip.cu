// Gossip step of CHOCO-SGD (Algorithm 3) for all simulated nodes at once:
// exact top-k selection of x_half - x_hat per (node, segment) by radix select
// on the magnitude bits, then one fused streaming pass that updates the public
// copies and mixes.  The mix pass is HBM-bound: per parameter and node it reads
// x_half and x_hat and writes x_hat and x (16 bytes); the neighbours' updated
// x_hat values are exchanged through shared memory, never re-read from HBM.
#include "common.cuh"

namespace lpdt {

constexpr int kMaxSeg = 128;
constexpr int kMaxNodes = 64;

struct SegTable {
    int32_t n_seg;
    int64_t off[kMaxSeg + 1];
    int64_t k[kMaxSeg];
};

struct SelectOut {       // per (node, segment)
    uint32_t thr;        // magnitude bits of the k-th largest |delta|
    uint32_t dense;      // 1: keep everything
    int64_t cut;         // ties (== thr) are kept only below this index
};

__device__ __forceinline__ uint32_t mag_bits(float xh, float xhat) {
    return __float_as_uint(__fsub_rn(xh, xhat)) & 0x7fffffffu;
}

// One CTA per (node, segment).  Four 8-bit radix passes, most significant
// first, narrow the k-th largest key; a final ordered pass places the tie cut.
__global__ void __launch_bounds__(1024)
topk_select_kernel(const float *__restrict__ x_half, const float *__restrict__ x_hat, int64_t d,
                   SegTable seg, SelectOut *__restrict__ out) {
    const int s = blockIdx.x, node = blockIdx.y;
    const int64_t lo = seg.off[s], hi = seg.off[s + 1], len = hi - lo;
    const int64_t k = seg.k[s];
    SelectOut *o = out + (int64_t)node * seg.n_seg + s;
    if (k >= len) {
        if (threadIdx.x == 0) { o->thr = 0; o->dense = 1; o->cut = hi; }
        return;
    }
    __shared__ unsigned int hist[256];
    __shared__ uint32_t s_prefix, s_mask;
    __shared__ long long s_need;      // how many more keys to take inside the current prefix
    __shared__ long long s_eq;        // keys equal to the final threshold
    __shared__ long long s_run, s_cut;
    const float *xh = x_half + (int64_t)node * d, *xq = x_hat + (int64_t)node * d;
    if (threadIdx.x == 0) { s_prefix = 0; s_mask = 0; s_need = (k > 0 ? k : 0); }
    __syncthreads();
    if (k <= 0) {   // keep nothing: threshold above every finite key, no ties
        if (threadIdx.x == 0) { o->thr = 0xffffffffu; o->dense = 0; o->cut = lo; }
        return;
    }
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix, mask = s_mask;
        for (int64_t e = lo + threadIdx.x; e < hi; e += blockDim.x) {
            uint32_t key = mag_bits(xh[e], xq[e]);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            long long need = s_need;
            int b = 255;
            for (; b > 0; --b) {
                if ((long long)hist[b] >= need) break;
                need -= hist[b];
            }
            s_need = need;                       // 1 <= need <= hist[b]
            s_eq = hist[b];
            s_prefix = prefix | ((uint32_t)b << shift);
            s_mask = mask | (255u << shift);
        }
        __syncthreads();
    }
    const uint32_t thr = s_prefix;
    const long long need = s_need, eq = s_eq;
    if (eq == need) {        // every tie is taken
        if (threadIdx.x == 0) { o->thr = thr; o->dense = 0; o->cut = hi; }
        return;
    }
    // ordered pass: find the index just past the need-th key equal to thr
    if (threadIdx.x == 0) { s_run = 0; s_cut = -1; }
    __syncthreads();
    for (int64_t base = lo; base < hi; base += blockDim.x) {
        const int64_t e = base + threadIdx.x;
        const int flag = (e < hi) && (mag_bits(xh[e], xq[e]) == thr);
        const int cnt = __syncthreads_count(flag);
        const long long run = s_run;
        if (run + cnt >= need) {
            // the cut lies in this chunk: rank the flags with a ballot scan
            __shared__ int warp_cnt[32];
            const unsigned bal = __ballot_sync(0xffffffffu, flag);
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            if (lane == 0) warp_cnt[warp] = __popc(bal);
            __syncthreads();
            int before = 0;
            for (int w = 0; w < warp; ++w) before += warp_cnt[w];
            const int rank = before + __popc(bal & ((1u << lane) - 1u));   // ties before me in the chunk
            if (flag && run + rank + 1 == need) s_cut = e + 1;
            __syncthreads();
            break;
        }
        __syncthreads();
        if (threadIdx.x == 0) s_run = run + cnt;
        __syncthreads();
    }
    if (threadIdx.x == 0) { o->thr = thr; o->dense = 0; o->cut = s_cut; }
}

// Fused public-copy update + mixing.  Block = TE consecutive parameters of all nodes.
template <int TE>
__global__ void __launch_bounds__(TE)
gossip_mix_kernel(int nodes, int64_t d, const float *__restrict__ x_half, float *__restrict__ x_hat,
                  float *__restrict__ x_out, const float *__restrict__ Wmix, float gamma,
                  SegTable seg, const SelectOut *__restrict__ sel) {
    extern __shared__ float sm[];
    float *s_w = sm;                        // [nodes][nodes]
    float *s_hat = sm + nodes * nodes;      // [nodes][TE]
    for (int i = threadIdx.x; i < nodes * nodes; i += TE) s_w[i] = Wmix[i];
    const int64_t e = (int64_t)blockIdx.x * TE + threadIdx.x;
    const bool live = e < d;
    int s = 0;
    if (live) {   // segment of this parameter (segments tile [0,d))
        int a = 0, b = seg.n_seg;
        while (b - a > 1) { int m = (a + b) >> 1; if (seg.off[m] <= e) a = m; else b = m; }
        s = a;
    }
    for (int i = 0; i < nodes; ++i) {
        float hn = 0.f;
        if (live) {
            const float xh = x_half[(int64_t)i * d + e], xq = x_hat[(int64_t)i * d + e];
            const float delta = __fsub_rn(xh, xq);
            const SelectOut so = sel[(int64_t)i * seg.n_seg + s];
            const uint32_t key = __float_as_uint(delta) & 0x7fffffffu;
            const bool keep = so.dense || key > so.thr || (key == so.thr && e < so.cut);
            hn = keep ? __fadd_rn(xq, delta) : xq;
            x_hat[(int64_t)i * d + e] = hn;
        }
        s_hat[i * TE + threadIdx.x] = hn;
    }
    __syncthreads();
    if (!live) return;
    for (int i = 0; i < nodes; ++i) {
        const float hi_ = s_hat[i * TE + threadIdx.x];
        float acc = 0.f;
        for (int j = 0; j < nodes; ++j) {
            const float w = s_w[i * nodes + j];
            if (w != 0.f) acc = __fadd_rn(acc, __fmul_rn(w, __fsub_rn(s_hat[j * TE + threadIdx.x], hi_)));
        }
        const float xh = x_half[(int64_t)i * d + e];
        x_out[(int64_t)i * d + e] = __fadd_rn(xh, __fmul_rn(gamma, acc));
    }
}

}  // namespace lpdt

using namespace lpdt;

extern "C" size_t lpdt_gossip_mix_workspace_size(int32_t nodes, int64_t d, int32_t n_segments) {
    (void)d;
    size_t n = (size_t)(nodes > 0 ? nodes : 1) * (size_t)(n_segments > 0 ? n_segments : 1);
    return align_up(n * sizeof(SelectOut), 256);
}

extern "C" lpdt_status lpdt_gossip_mix(int32_t nodes, int64_t d, const float *x_half, float *x_hat,
                                       float *x_out, const float *Wmix, float gamma, int32_t n_segments,
                                       const int64_t *seg_offsets, const int64_t *seg_k, void *ws,
                                       size_t ws_bytes, int32_t *dev_status, void *stream) {
    (void)dev_status;
    LPDT_CHECK_ARG(nodes >= 0 && d >= 0 && n_segments >= 1);
    if (nodes == 0 || d == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x_half && x_hat && x_out && Wmix && seg_offsets && seg_k);
    LPDT_CHECK_ARG(x_hat != x_half && x_hat != x_out);
    if (nodes > kMaxNodes || n_segments > kMaxSeg) return LPDT_ERR_UNSUPPORTED;
    LPDT_CHECK_ARG(seg_offsets[0] == 0 && seg_offsets[n_segments] == d);
    SegTable seg;
    seg.n_seg = n_segments;
    for (int s = 0; s < n_segments; ++s) {
        LPDT_CHECK_ARG(seg_offsets[s + 1] > seg_offsets[s] && seg_k[s] >= 0);
        seg.off[s] = seg_offsets[s];
        seg.k[s] = seg_k[s];
    }
    seg.off[n_segments] = d;
    if (!ws || ws_bytes < lpdt_gossip_mix_workspace_size(nodes, d, n_segments) || !aligned(ws, 8))
        return LPDT_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    SelectOut *sel = (SelectOut *)ws;
    topk_select_kernel<<<dim3(n_segments, nodes), 1024, 0, st>>>(x_half, x_hat, d, seg, sel);
    LPDT_LAUNCH_CHECK();
    constexpr int TE = 256;
    size_t smem = ((size_t)nodes * nodes + (size_t)nodes * TE) * sizeof(float);
    static bool attr_set = false;
    if (!attr_set) {
        LPDT_CUDA(cudaFuncSetAttribute(gossip_mix_kernel<TE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (kMaxNodes * kMaxNodes + kMaxNodes * TE) * (int)sizeof(float)));
        attr_set = true;
    }
    gossip_mix_kernel<TE><<<(unsigned)ceil_div(d, TE), TE, smem, st>>>(nodes, d, x_half, x_hat, x_out, Wmix,
                                                                    gamma, seg, sel);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
