// CUDA-core int8 convolution kernels for shapes the tensor-core engine does
// not take (channel counts that are not multiples of 16, strided layers, tiny
// problems).  Plain implicit-GEMM loops with 4-way int8 dot products (dp4a)
// where the channel count allows; int32 accumulation is exact in any order.
#include "common.cuh"
#include "qconv_internal.cuh"

namespace lpdt {

__device__ __forceinline__ int dot_s8(const int8_t *__restrict__ a, const int8_t *__restrict__ b, int n,
                                      bool vec4) {
    int acc = 0;
    if (vec4) {
        const int *a4 = reinterpret_cast<const int *>(a);
        const int *b4 = reinterpret_cast<const int *>(b);
        for (int i = 0; i < n / 4; ++i) acc = __dp4a(__ldg(a4 + i), __ldg(b4 + i), acc);
    } else {
        for (int i = 0; i < n; ++i) acc += (int)a[i] * (int)b[i];
    }
    return acc;
}

// the same on unsigned codes
__device__ __forceinline__ int dot_u8(const uint8_t *__restrict__ a, const uint8_t *__restrict__ b, int n, bool vec4) {
    unsigned acc = 0;
    if (vec4) {
        const unsigned *a4 = reinterpret_cast<const unsigned *>(a);
        const unsigned *b4 = reinterpret_cast<const unsigned *>(b);
        for (int i = 0; i < n / 4; ++i) acc = __dp4a(__ldg(a4 + i), __ldg(b4 + i), acc);
    } else {
        for (int i = 0; i < n; ++i) acc += (unsigned)a[i] * (unsigned)b[i];
    }
    return (int)acc;
}

// One thread per output element (n, b, oh, ow, co); co fastest.
__global__ void conv_fwd_generic(lpdt_conv_desc d, int Ho, int Wo, const int8_t *__restrict__ A,
                                 const int8_t *__restrict__ Wq, int32_t *__restrict__ acc_out,
                                 float *__restrict__ Y, const float *__restrict__ s1,
                                 const float *__restrict__ s2, const float *__restrict__ bias,
                                 int64_t bias_stride, bool vec4, bool uns) {
    pdl_enter();
    const int64_t per_node = (int64_t)d.B * Ho * Wo * d.Cout;
    const int64_t total = per_node * d.nodes;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int co = (int)(o % d.Cout);
        int64_t pix = o / d.Cout;
        int ow = (int)(pix % Wo); pix /= Wo;
        int oh = (int)(pix % Ho); pix /= Ho;
        int b = (int)(pix % d.B);
        int n = (int)(pix / d.B);
        int acc = 0;
        for (int r = 0; r < d.R; ++r) {
            int ih = oh * d.stride + r - d.pad;
            if (ih < 0 || ih >= d.H) continue;
            for (int s = 0; s < d.S; ++s) {
                int iw = ow * d.stride + s - d.pad;
                if (iw < 0 || iw >= d.W) continue;
                const int8_t *a = A + ((((int64_t)n * d.B + b) * d.H + ih) * d.W + iw) * d.Cin;
                const int8_t *w = Wq + ((((int64_t)n * d.Cout + co) * d.R + r) * d.S + s) * d.Cin;
                acc += uns ? dot_u8(reinterpret_cast<const uint8_t *>(a), reinterpret_cast<const uint8_t *>(w), d.Cin, vec4)
                           : dot_s8(a, w, d.Cin, vec4);
            }
        }
        if (acc_out) acc_out[o] = acc;
        if (Y) {
            float v = __fmul_rn(__int2float_rn(acc), __fmul_rn(s1[n], s2[n]));
            if (bias) v = __fadd_rn(v, bias[(int64_t)n * bias_stride + co]);
            Y[o] = v;
        }
    }
}

// Wt[n][ci][r][s][co] = W[n][co][r][s][ci]
__global__ void transpose_weights_kernel(lpdt_conv_desc d, const int8_t *__restrict__ Wq,
                                         int8_t *__restrict__ Wt) {
    pdl_enter();
    const int64_t per_node = (int64_t)d.Cout * d.R * d.S * d.Cin;
    const int64_t total = per_node * d.nodes;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int co = (int)(o % d.Cout);
        int64_t t = o / d.Cout;
        int s = (int)(t % d.S); t /= d.S;
        int r = (int)(t % d.R); t /= d.R;
        int ci = (int)(t % d.Cin);
        int n = (int)(t / d.Cin);
        Wt[o] = Wq[((((int64_t)n * d.Cout + co) * d.R + r) * d.S + s) * d.Cin + ci];
    }
}

// One thread per input-gradient element (n, b, ih, iw, ci); ci fastest.
__global__ void conv_bwd_data_generic(lpdt_conv_desc d, int Ho, int Wo, const int8_t *__restrict__ E,
                                      const int8_t *__restrict__ Wt, int32_t *__restrict__ acc_out,
                                      float *__restrict__ dA, const float *__restrict__ s1,
                                      const float *__restrict__ s2, bool vec4, const float *__restrict__ addend,
                                      bool uns) {
    pdl_enter();
    const int64_t per_node = (int64_t)d.B * d.H * d.W * d.Cin;
    const int64_t total = per_node * d.nodes;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int ci = (int)(o % d.Cin);
        int64_t pix = o / d.Cin;
        int iw = (int)(pix % d.W); pix /= d.W;
        int ih = (int)(pix % d.H); pix /= d.H;
        int b = (int)(pix % d.B);
        int n = (int)(pix / d.B);
        int acc = 0;
        for (int r = 0; r < d.R; ++r) {
            int th = ih + d.pad - r;
            if (th < 0 || th % d.stride) continue;
            int oh = th / d.stride;
            if (oh >= Ho) continue;
            for (int s = 0; s < d.S; ++s) {
                int tw = iw + d.pad - s;
                if (tw < 0 || tw % d.stride) continue;
                int ow = tw / d.stride;
                if (ow >= Wo) continue;
                const int8_t *e = E + ((((int64_t)n * d.B + b) * Ho + oh) * Wo + ow) * d.Cout;
                const int8_t *w = Wt + ((((int64_t)n * d.Cin + ci) * d.R + r) * d.S + s) * d.Cout;
                acc += uns ? dot_u8(reinterpret_cast<const uint8_t *>(e), reinterpret_cast<const uint8_t *>(w), d.Cout, vec4)
                           : dot_s8(e, w, d.Cout, vec4);
            }
        }
        if (acc_out) acc_out[o] = acc;
        if (dA) {
            float v = __fmul_rn(__int2float_rn(acc), __fmul_rn(s1[n], s2[n]));
            if (addend) v = __fadd_rn(v, addend[o]);
            dA[o] = v;
        }
    }
}

// Split over pixels: block (chunk, node) accumulates every dW entry over its
// pixel chunk and adds the partial sums with integer atomics (exact).
__global__ void conv_bwd_weight_generic(lpdt_conv_desc d, int Ho, int Wo, int chunk,
                                        const int8_t *__restrict__ E, const int8_t *__restrict__ A,
                                        int32_t *__restrict__ acc_out, bool uns) {
    pdl_enter();
    const int n = blockIdx.y;
    const int64_t npix = (int64_t)d.B * Ho * Wo;
    const int64_t p0 = (int64_t)blockIdx.x * chunk;
    const int64_t p1 = (p0 + chunk < npix) ? p0 + chunk : npix;
    const int nout = d.Cout * d.R * d.S * d.Cin;
    for (int o = threadIdx.x; o < nout; o += blockDim.x) {
        int ci = o % d.Cin;
        int t = o / d.Cin;
        int s = t % d.S; t /= d.S;
        int r = t % d.R;
        int co = t / d.R;
        int acc = 0;
        for (int64_t p = p0; p < p1; ++p) {
            int ow = (int)(p % Wo);
            int64_t q = p / Wo;
            int oh = (int)(q % Ho);
            int b = (int)(q / Ho);
            int ih = oh * d.stride + r - d.pad, iw = ow * d.stride + s - d.pad;
            if (ih < 0 || ih >= d.H || iw < 0 || iw >= d.W) continue;
            const int8_t e = E[((int64_t)n * npix + p) * d.Cout + co];
            const int8_t a = A[((((int64_t)n * d.B + b) * d.H + ih) * d.W + iw) * d.Cin + ci];
            acc += uns ? (int)((unsigned)(uint8_t)e * (unsigned)(uint8_t)a) : (int)e * (int)a;
        }
        if (acc) atomicAdd(acc_out + (int64_t)n * nout + o, acc);
    }
}

__global__ void dequant_acc_kernel(const int32_t *__restrict__ acc, int nodes, int64_t per_node,
                                   const float *__restrict__ s1, const float *__restrict__ s2,
                                   float *__restrict__ out, int64_t out_stride) {
    pdl_enter();
    const int64_t total = per_node * nodes;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        int n = (int)(o / per_node);
        int64_t i = o % per_node;
        out[(int64_t)n * out_stride + i] = __fmul_rn(__int2float_rn(acc[o]), __fmul_rn(s1[n], s2[n]));
    }
}

// The same conversion for many tensors in one launch (all weight gradients of a network): the sums of
// tensor t are a contiguous [nodes][size[t]] block at acc + acc_off[t]; its fp32 values go to offset
// out_off[t] of every node's output row; each tensor has its own pair of per-node scales.
// grid = (blocks, nodes, tensors).
constexpr int kMaxDequantBatch = 64;
struct DequantBatch {
    int count;
    long long acc_off[kMaxDequantBatch], size[kMaxDequantBatch], out_off[kMaxDequantBatch];
    const float *s1[kMaxDequantBatch], *s2[kMaxDequantBatch];
};
__global__ void dequant_acc_batch_kernel(const int32_t *__restrict__ acc, DequantBatch db,
                                         float *__restrict__ out, long long out_stride) {
    pdl_enter();
    const int t = blockIdx.z, n = blockIdx.y;
    const long long size = db.size[t];
    const float sc = __fmul_rn(db.s1[t][n], db.s2[t][n]);
    const int32_t *a = acc + db.acc_off[t] + (long long)n * size;
    float *o = out + (long long)n * out_stride + db.out_off[t];
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < size; i += (long long)gridDim.x * blockDim.x)
        o[i] = __fmul_rn(__int2float_rn(a[i]), sc);
}

static unsigned grid_for(int64_t n);

lpdt_status dequant_acc_launch(const int32_t *acc, int nodes, int64_t per_node, const float *s1,
                               const float *s2, float *out, int64_t out_stride, cudaStream_t st) {
    launch_k(dequant_acc_kernel, grid_for(per_node * nodes), 256, 0, st, acc, nodes, per_node, s1, s2, out, out_stride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

static unsigned grid_for(int64_t n) {
    int64_t b = ceil_div(n, 256), cap = (int64_t)kNumSMs * 32;
    return (unsigned)(b < 1 ? 1 : (b > cap ? cap : b));
}

lpdt_status generic_fwd(const lpdt_conv_desc &d, const int8_t *A, const float *sA, const int8_t *Wq,
                        const float *sW, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                        cudaStream_t st, bool uns) {
    const int Ho = conv_out(d.H, d.pad, d.R, d.stride), Wo = conv_out(d.W, d.pad, d.S, d.stride);
    const int64_t total = (int64_t)d.nodes * d.B * Ho * Wo * d.Cout;
    const bool vec4 = d.Cin % 4 == 0 && aligned(A, 4) && aligned(Wq, 4);
    g_last_kernel = "lpdt::conv_fwd_generic";
    launch_k(conv_fwd_generic, grid_for(total), 256, 0, st, d, Ho, Wo, A, Wq, Yacc, Y, sA, sW, bias, bias_stride, vec4, uns);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

lpdt_status generic_bwd_data(const lpdt_conv_desc &d, const int8_t *E, const float *sE, const int8_t *Wq,
                             const float *sW, float *dA, int32_t *dAacc, const float *addend, void *ws, cudaStream_t st,
                             bool uns) {
    const int Ho = conv_out(d.H, d.pad, d.R, d.stride), Wo = conv_out(d.W, d.pad, d.S, d.stride);
    int8_t *Wt = (int8_t *)ws;
    const int64_t wn = (int64_t)d.nodes * d.Cout * d.R * d.S * d.Cin;
    launch_k(transpose_weights_kernel, grid_for(wn), 256, 0, st, d, Wq, Wt);
    LPDT_LAUNCH_CHECK();
    const int64_t total = (int64_t)d.nodes * d.B * d.H * d.W * d.Cin;
    const bool vec4 = d.Cout % 4 == 0 && aligned(E, 4) && aligned(Wt, 4);
    g_last_kernel = "lpdt::conv_bwd_data_generic";
    launch_k(conv_bwd_data_generic, grid_for(total), 256, 0, st, d, Ho, Wo, E, Wt, dAacc, dA, sE, sW, vec4, addend, uns);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

lpdt_status generic_bwd_weight(const lpdt_conv_desc &d, const int8_t *E, const float *sE, const int8_t *A,
                               const float *sA, float *dW, int64_t dw_stride, int32_t *dWacc, void *ws,
                               cudaStream_t st, bool uns) {
    const int Ho = conv_out(d.H, d.pad, d.R, d.stride), Wo = conv_out(d.W, d.pad, d.S, d.stride);
    const int64_t per_node = (int64_t)d.Cout * d.R * d.S * d.Cin;
    if (d.nodes > 65535) return LPDT_ERR_UNSUPPORTED;        // nodes ride in grid.y
    int32_t *acc = dWacc ? dWacc : (int32_t *)ws;
    LPDT_CUDA(cudaMemsetAsync(acc, 0, (size_t)d.nodes * per_node * sizeof(int32_t), st));
    const int64_t npix = (int64_t)d.B * Ho * Wo;
    if (npix > 0) {                      // an empty batch leaves the zeroed sums: the gradient of no samples
        int chunk = 4;
        while (ceil_div(npix, chunk) * d.nodes > (int64_t)kNumSMs * 16) chunk *= 2;
        g_last_kernel = "lpdt::conv_bwd_weight_generic";
        launch_k(conv_bwd_weight_generic, dim3((unsigned)ceil_div(npix, chunk), d.nodes), 256, 0, st, d, Ho, Wo, chunk, E, A, acc, uns);
        LPDT_LAUNCH_CHECK();
    }
    if (dW) {
        launch_k(dequant_acc_kernel, grid_for(per_node * d.nodes), 256, 0, st, acc, d.nodes, per_node, sE, sA, dW, dw_stride);
        LPDT_LAUNCH_CHECK();
    }
    return LPDT_OK;
}

}  // namespace lpdt

extern "C" lpdt_status lpdt_dequantize_acc_batch(const int32_t *acc, int32_t nodes, int32_t n_tensors,
                                                 const int64_t *acc_offsets, const int64_t *sizes,
                                                 const int64_t *out_offsets, const float *const *s1,
                                                 const float *const *s2, float *out, int64_t out_node_stride,
                                                 void *stream) {
    using namespace lpdt;
    LPDT_CHECK_ARG(nodes >= 0 && n_tensors >= 0);
    if (nodes == 0 || n_tensors == 0) return LPDT_OK;
    LPDT_CHECK_ARG(acc && acc_offsets && sizes && out_offsets && s1 && s2 && out);
    if (n_tensors > kMaxDequantBatch || nodes > 65535) return LPDT_ERR_UNSUPPORTED;
    DequantBatch db;
    db.count = n_tensors;
    long long longest = 0;
    for (int t = 0; t < n_tensors; ++t) {
        LPDT_CHECK_ARG(acc_offsets[t] >= 0 && out_offsets[t] >= 0 && sizes[t] >= 0 && s1[t] && s2[t]);
        LPDT_CHECK_ARG(out_offsets[t] + sizes[t] <= out_node_stride || nodes == 1);
        db.acc_off[t] = acc_offsets[t]; db.size[t] = sizes[t]; db.out_off[t] = out_offsets[t];
        db.s1[t] = s1[t]; db.s2[t] = s2[t];
        if (sizes[t] > longest) longest = sizes[t];
    }
    if (longest == 0) return LPDT_OK;
    int bx = (int)ceil_div(longest, 256 * 4);
    if (bx > 64) bx = 64;
    if (bx < 1) bx = 1;
    launch_k(dequant_acc_batch_kernel, dim3(bx, nodes, n_tensors), 256, 0, as_stream(stream), acc, db, out,
             out_node_stride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
