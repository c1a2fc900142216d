// Small element-wise and reduction kernels that surround the layers of one
// training step: SGD update, residual shortcuts, pooling, softmax
// cross-entropy, bias gradient.  All are HBM-bound streaming kernels.
#include <math.h>
#include "common.cuh"

namespace lpdt {

static inline unsigned grid1d(int64_t n, int threads = 256) {
    int64_t b = ceil_div(n, threads);
    int64_t cap = (int64_t)kNumSMs * 16;
    return (unsigned)(b < 1 ? 1 : (b > cap ? cap : b));
}

__global__ void sgd_kernel(int64_t n, const float *__restrict__ x, const float *__restrict__ g,
                           float lr, float *__restrict__ out) {
    pdl_enter();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        out[i] = __fsub_rn(x[i], __fmul_rn(lr, g[i]));
}

// grid.y = node; B = samples per node.  amax_out (nullable) receives max|y| per node.
__global__ void residual_add_kernel(int B, int H, int W, int Ca, int C, int stride, int ch_off,
                                    const float *__restrict__ r, const float *__restrict__ a,
                                    float *__restrict__ y, float *__restrict__ amax_out) {
    pdl_enter();
    const int Ho = (H + stride - 1) / stride, Wo = (W + stride - 1) / stride;
    const int64_t per_node = (int64_t)B * Ho * Wo * C;
    const int64_t base = (int64_t)blockIdx.y * per_node;
    float ymax = 0.f;
    for (int64_t ol = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; ol < per_node; ol += (int64_t)gridDim.x * blockDim.x) {
        const int64_t o = base + ol;
        int c = (int)(o % C);
        int64_t pix = o / C;
        int ow = (int)(pix % Wo); pix /= Wo;
        int oh = (int)(pix % Ho);
        int64_t nb = pix / Ho;
        float v = r[o];
        int ca = c - ch_off;
        if (ca >= 0 && ca < Ca)
            v = __fadd_rn(v, a[((nb * H + (int64_t)oh * stride) * W + (int64_t)ow * stride) * Ca + ca]);
        y[o] = v;
        ymax = fmaxf(ymax, fabsf(v));
    }
    if (amax_out) block_amax_to(ymax, amax_out + blockIdx.y);
}

// Vector forms: 4 consecutive channels per thread (C, Ca and ch_off multiples of 4).
__global__ void residual_add_v4_kernel(int B, int H, int W, int Ca4, int C4, int stride, int ch_off4,
                                       const float4 *__restrict__ r, const float4 *__restrict__ a,
                                       float4 *__restrict__ y, float *__restrict__ amax_out) {
    pdl_enter();
    const int Ho = (H + stride - 1) / stride, Wo = (W + stride - 1) / stride;
    const long long per_node = (long long)B * Ho * Wo * C4;
    const long long base = (long long)blockIdx.y * per_node;
    float ymax = 0.f;
    for (long long ol = (long long)blockIdx.x * blockDim.x + threadIdx.x; ol < per_node; ol += (long long)gridDim.x * blockDim.x) {
        const long long o = base + ol;
        const int c = (int)(o % C4);
        float4 v = r[o];
        const int ca = c - ch_off4;
        if (ca >= 0 && ca < Ca4) {
            long long pix = o / C4;
            const int ow = (int)(pix % Wo); pix /= Wo;
            const int oh = (int)(pix % Ho);
            const long long nb = pix / Ho;
            const float4 u = a[((nb * H + (long long)oh * stride) * W + (long long)ow * stride) * Ca4 + ca];
            v.x = __fadd_rn(v.x, u.x); v.y = __fadd_rn(v.y, u.y); v.z = __fadd_rn(v.z, u.z); v.w = __fadd_rn(v.w, u.w);
        }
        y[o] = v;
        ymax = fmaxf(ymax, fmaxf(fmaxf(fabsf(v.x), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w))));
    }
    if (amax_out) block_amax_to(ymax, amax_out + blockIdx.y);
}

__global__ void residual_add_bwd_v4_kernel(int NB, int H, int W, int Ca4, int C4, int stride, int ch_off4,
                                           const float4 *__restrict__ dy, const float4 *__restrict__ gm,
                                           float4 *__restrict__ da) {
    pdl_enter();
    const int Ho = (H + stride - 1) / stride, Wo = (W + stride - 1) / stride;
    const long long total = (long long)NB * H * W * Ca4;
    for (long long o = (long long)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (long long)gridDim.x * blockDim.x) {
        float4 v = gm[o];
        bool hit = stride == 1;
        long long src = o;
        if (stride != 1 || Ca4 != C4) {
            const int ca = (int)(o % Ca4);
            long long pix = o / Ca4;
            const int w = (int)(pix % W); pix /= W;
            const int h = (int)(pix % H);
            const long long nb = pix / H;
            hit = (h % stride == 0) && (w % stride == 0);
            src = ((nb * Ho + h / stride) * Wo + w / stride) * C4 + ca + ch_off4;
        }
        if (hit) {
            const float4 u = dy[src];
            v.x = __fadd_rn(v.x, u.x); v.y = __fadd_rn(v.y, u.y); v.z = __fadd_rn(v.z, u.z); v.w = __fadd_rn(v.w, u.w);
        }
        da[o] = v;
    }
}

__global__ void residual_add_bwd_kernel(int64_t NB, int H, int W, int Ca, int C, int stride, int ch_off,
                                        const float *__restrict__ dy, const float *__restrict__ gm,
                                        float *__restrict__ da) {
    pdl_enter();
    const int Ho = (H + stride - 1) / stride, Wo = (W + stride - 1) / stride;
    const int64_t total = NB * H * W * Ca;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int ca = (int)(o % Ca);
        int64_t pix = o / Ca;
        int w = (int)(pix % W); pix /= W;
        int h = (int)(pix % H);
        int64_t nb = pix / H;
        float v = gm[o];
        if (h % stride == 0 && w % stride == 0)
            v = __fadd_rn(v, dy[((nb * Ho + h / stride) * Wo + w / stride) * C + ca + ch_off]);
        da[o] = v;
    }
}

__global__ void avgpool_kernel(int64_t NB, int HW, int C, const float *__restrict__ x, float *__restrict__ y) {
    pdl_enter();
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= NB * C) return;
    int64_t nb = i / C; int c = (int)(i % C);
    double s = 0.0;
    for (int p = 0; p < HW; ++p) s += (double)x[(nb * HW + p) * C + c];
    y[i] = (float)(s / (double)HW);
}

__global__ void avgpool_bwd_kernel(int64_t NB, int HW, int C, const float *__restrict__ dy, float *__restrict__ dx) {
    pdl_enter();
    const int64_t total = NB * HW * C;
    const float fhw = (float)HW;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int c = (int)(o % C);
        int64_t nb = o / ((int64_t)HW * C);
        dx[o] = __fdiv_rn(dy[nb * C + c], fhw);
    }
}

__global__ void maxpool_kernel(int64_t NB, int H, int W, int C, const float *__restrict__ x,
                               float *__restrict__ y, int8_t *__restrict__ idx) {
    pdl_enter();
    const int Ho = H / 2, Wo = W / 2;
    const int64_t total = NB * Ho * Wo * C;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int c = (int)(o % C);
        int64_t pix = o / C;
        int ow = (int)(pix % Wo); pix /= Wo;
        int oh = (int)(pix % Ho);
        int64_t nb = pix / Ho;
        float best = 0.f; int bi = -1;
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            float v = x[((nb * H + 2 * oh + t / 2) * W + 2 * ow + t % 2) * C + c];
            if (bi < 0 || v > best) { best = v; bi = t; }
        }
        y[o] = best; idx[o] = (int8_t)bi;
    }
}

__global__ void maxpool_bwd_kernel(int64_t NB, int H, int W, int C, const float *__restrict__ dy,
                                   const int8_t *__restrict__ idx, float *__restrict__ dx) {
    pdl_enter();
    const int Ho = H / 2, Wo = W / 2;
    const int64_t total = NB * H * W * C;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int c = (int)(o % C);
        int64_t pix = o / C;
        int w = (int)(pix % W); pix /= W;
        int h = (int)(pix % H);
        int64_t nb = pix / H;
        int64_t po = ((nb * Ho + h / 2) * Wo + w / 2) * C + c;
        int t = (h & 1) * 2 + (w & 1);
        dx[o] = (idx[po] == t) ? dy[po] : 0.f;
    }
}

// Four channels per thread (C % 4 == 0, 16-byte aligned tensors): 16-byte loads and stores, one
// index decode per four elements.
__global__ void maxpool_v4_kernel(int64_t NB, int H, int W, int C4, const float4 *__restrict__ x,
                                  float4 *__restrict__ y, char4 *__restrict__ idx) {
    pdl_enter();
    const int Ho = H / 2, Wo = W / 2;
    const int64_t total = NB * Ho * Wo * C4;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(o % C4);
        int64_t pix = o / C4;
        const int ow = (int)(pix % Wo); pix /= Wo;
        const int oh = (int)(pix % Ho);
        const int64_t nb = pix / Ho;
        const int64_t base = ((nb * H + 2 * oh) * W + 2 * ow) * C4 + c;
        const float4 v0 = x[base], v1 = x[base + C4], v2 = x[base + (int64_t)W * C4], v3 = x[base + (int64_t)W * C4 + C4];
        float4 best = v0; char4 bi = make_char4(0, 0, 0, 0);
#define LPDT_MP_STEP(f, v, t) if (v.f > best.f) { best.f = v.f; bi.f = t; }
        LPDT_MP_STEP(x, v1, 1) LPDT_MP_STEP(y, v1, 1) LPDT_MP_STEP(z, v1, 1) LPDT_MP_STEP(w, v1, 1)
        LPDT_MP_STEP(x, v2, 2) LPDT_MP_STEP(y, v2, 2) LPDT_MP_STEP(z, v2, 2) LPDT_MP_STEP(w, v2, 2)
        LPDT_MP_STEP(x, v3, 3) LPDT_MP_STEP(y, v3, 3) LPDT_MP_STEP(z, v3, 3) LPDT_MP_STEP(w, v3, 3)
#undef LPDT_MP_STEP
        y[o] = best; idx[o] = bi;
    }
}

__global__ void maxpool_bwd_v4_kernel(int64_t NB, int H, int W, int C4, const float4 *__restrict__ dy,
                                      const char4 *__restrict__ idx, float4 *__restrict__ dx) {
    pdl_enter();
    const int Ho = H / 2, Wo = W / 2;
    const int64_t total = NB * H * W * C4;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int c = (int)(o % C4);
        int64_t pix = o / C4;
        const int w = (int)(pix % W); pix /= W;
        const int h = (int)(pix % H);
        const int64_t nb = pix / H;
        const int64_t po = ((nb * Ho + h / 2) * Wo + w / 2) * C4 + c;
        const int t = (h & 1) * 2 + (w & 1);
        const float4 g = dy[po];
        const char4 i = idx[po];
        dx[o] = make_float4(i.x == t ? g.x : 0.f, i.y == t ? g.y : 0.f, i.z == t ? g.z : 0.f, i.w == t ? g.w : 0.f);
    }
}

// One block per node, one thread per sample; double arithmetic, fixed-order tree.
// A label outside [0, K) is never used as an index: that sample adds nothing to the loss, its gradient is the
// plain softmax/B, and LPDT_ERR_INVALID_ARG is written to the status word.
__global__ void softmax_ce_kernel(int B, int K, const float *__restrict__ logits,
                                  const int32_t *__restrict__ labels, float *__restrict__ loss,
                                  float *__restrict__ dlogits, int32_t *__restrict__ dev_status) {
    pdl_enter();
    extern __shared__ double s_part[];
    const int n = blockIdx.x;
    double mine = 0.0;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        const float *z = logits + ((int64_t)n * B + b) * K;
        float *dz = dlogits + ((int64_t)n * B + b) * K;
        double zmax = z[0];
        for (int k = 1; k < K; ++k) if ((double)z[k] > zmax) zmax = z[k];
        double den = 0.0;
        for (int k = 0; k < K; ++k) den += exp((double)z[k] - zmax);
        const int lab = labels[(int64_t)n * B + b];
        const bool lab_ok = lab >= 0 && lab < K;
        if (lab_ok) mine += log(den) + zmax - (double)z[lab];
        else if (dev_status) atomicCAS(dev_status, 0, (int32_t)LPDT_ERR_INVALID_ARG);
        for (int k = 0; k < K; ++k) {
            double p = exp((double)z[k] - zmax) / den;
            dz[k] = (float)((p - (k == lab ? 1.0 : 0.0)) / (double)B);
        }
    }
    s_part[threadIdx.x] = mine;
    __syncthreads();
    for (int o = blockDim.x >> 1; o > 0; o >>= 1) {
        if (threadIdx.x < o) s_part[threadIdx.x] += s_part[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[n] = (float)(s_part[0] / (double)B);
}

__global__ void colsum_kernel(int nodes, int B, int C, const float *__restrict__ x,
                              float *__restrict__ out, int64_t ostride) {
    pdl_enter();
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nodes * C) return;
    int n = i / C, c = i % C;
    double s = 0.0;
    for (int b = 0; b < B; ++b) s += (double)x[((int64_t)n * B + b) * C + c];
    out[(int64_t)n * ostride + c] = (float)s;
}

}  // namespace lpdt

using namespace lpdt;

extern "C" lpdt_status lpdt_sgd_update(int64_t n, const float *x, const float *g, float lr, float *out,
                                       void *stream) {
    LPDT_CHECK_ARG(n >= 0);
    if (n == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && g && out);
    launch_k(sgd_kernel, grid1d(n), 256, 0, as_stream(stream), n, x, g, lr, out);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_residual_add(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t Ca,
                                         int32_t C, int32_t stride, int32_t ch_off, const float *r,
                                         const float *a, float *y, float *amax_out, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && Ca > 0 && C >= Ca && stride >= 1);
    LPDT_CHECK_ARG(ch_off >= 0 && ch_off + Ca <= C);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(r && a && y && nodes <= 65535);
    const int Ho = (H + stride - 1) / stride, Wo = (W + stride - 1) / stride;
    const int64_t per_node = (int64_t)B * Ho * Wo * C;
    auto gx = [&](int64_t n) {
        int64_t b = ceil_div(n, 256), cap = ceil_div((int64_t)kNumSMs * 16, nodes);
        return (unsigned)(b < 1 ? 1 : (b > cap ? cap : b));
    };
    if (C % 4 == 0 && Ca % 4 == 0 && ch_off % 4 == 0 && aligned(r, 16) && aligned(a, 16) && aligned(y, 16))
        launch_k(residual_add_v4_kernel, dim3(gx(per_node / 4), nodes), 256, 0, as_stream(stream), 
            B, H, W, Ca / 4, C / 4, stride, ch_off / 4, (const float4 *)r, (const float4 *)a, (float4 *)y, amax_out);
    else
        launch_k(residual_add_kernel, dim3(gx(per_node), nodes), 256, 0, as_stream(stream), 
            B, H, W, Ca, C, stride, ch_off, r, a, y, amax_out);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_residual_add_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t Ca,
                                             int32_t C, int32_t stride, int32_t ch_off, const float *dy,
                                             const float *g_main, float *da, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && Ca > 0 && C >= Ca && stride >= 1);
    LPDT_CHECK_ARG(ch_off >= 0 && ch_off + Ca <= C);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dy && g_main && da);
    if (C % 4 == 0 && Ca % 4 == 0 && ch_off % 4 == 0 && aligned(dy, 16) && aligned(g_main, 16) && aligned(da, 16) &&
        (int64_t)nodes * B < 0x7fffffff)
        launch_k(residual_add_bwd_v4_kernel, grid1d((int64_t)nodes * B * H * W * Ca / 4), 256, 0, as_stream(stream), 
            nodes * B, H, W, Ca / 4, C / 4, stride, ch_off / 4, (const float4 *)dy, (const float4 *)g_main, (float4 *)da);
    else
    launch_k(residual_add_bwd_kernel, grid1d((int64_t)nodes * B * H * W * Ca), 256, 0, as_stream(stream), 
        (int64_t)nodes * B, H, W, Ca, C, stride, ch_off, dy, g_main, da);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_avgpool(int32_t nodes, int32_t B, int32_t HW, int32_t C, const float *x,
                                    float *y, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && HW > 0 && C > 0);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && y);
    int64_t n = (int64_t)nodes * B * C;
    launch_k(avgpool_kernel, (unsigned)ceil_div(n, 256), 256, 0, as_stream(stream), (int64_t)nodes * B, HW, C, x, y);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_avgpool_bwd(int32_t nodes, int32_t B, int32_t HW, int32_t C, const float *dy,
                                        float *dx, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && HW > 0 && C > 0);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dy && dx);
    launch_k(avgpool_bwd_kernel, grid1d((int64_t)nodes * B * HW * C), 256, 0, as_stream(stream), 
        (int64_t)nodes * B, HW, C, dy, dx);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_maxpool2x2(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                       const float *x, float *y, int8_t *idx, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && H % 2 == 0 && W % 2 == 0);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && y && idx);
    if (C % 4 == 0 && aligned(x, 16) && aligned(y, 16) && aligned(idx, 4))
        launch_k(maxpool_v4_kernel, grid1d((int64_t)nodes * B * (H / 2) * (W / 2) * (C / 4)), 256, 0, as_stream(stream), 
            (int64_t)nodes * B, H, W, C / 4, reinterpret_cast<const float4 *>(x), reinterpret_cast<float4 *>(y),
            reinterpret_cast<char4 *>(idx));
    else
        launch_k(maxpool_kernel, grid1d((int64_t)nodes * B * (H / 2) * (W / 2) * C), 256, 0, as_stream(stream), 
            (int64_t)nodes * B, H, W, C, x, y, idx);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_maxpool2x2_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                           const float *dy, const int8_t *idx, float *dx, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && H % 2 == 0 && W % 2 == 0);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dy && idx && dx);
    if (C % 4 == 0 && aligned(dx, 16) && aligned(dy, 16) && aligned(idx, 4))
        launch_k(maxpool_bwd_v4_kernel, grid1d((int64_t)nodes * B * H * W * (C / 4)), 256, 0, as_stream(stream), 
            (int64_t)nodes * B, H, W, C / 4, reinterpret_cast<const float4 *>(dy), reinterpret_cast<const char4 *>(idx),
            reinterpret_cast<float4 *>(dx));
    else
        launch_k(maxpool_bwd_kernel, grid1d((int64_t)nodes * B * H * W * C), 256, 0, as_stream(stream), 
            (int64_t)nodes * B, H, W, C, dy, idx, dx);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_softmax_ce(int32_t nodes, int32_t B, int32_t K, const float *logits,
                                       const int32_t *labels, float *loss, float *dlogits, int32_t *dev_status,
                                       void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B > 0 && K > 0);
    if (nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(logits && labels && loss && dlogits);
    int threads = 32;
    while (threads < B && threads < 256) threads <<= 1;
    launch_k(softmax_ce_kernel, nodes, threads, threads * sizeof(double), as_stream(stream), B, K, logits, labels,
             loss, dlogits, dev_status);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_colsum(int32_t nodes, int32_t B, int32_t C, const float *x, float *out,
                                   int64_t out_node_stride, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && C > 0);
    if (nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && out && (out_node_stride >= C || nodes == 1));
    launch_k(colsum_kernel, (nodes * C + 255) / 256, 256, 0, as_stream(stream), nodes, B, C, x, out, out_node_stride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
