// Front end of the quantized contractions: argument validation, workspace
// accounting and the choice between the tensor-core engine and the CUDA-core
// kernels.  Layers whose input channel count is not a multiple of 16 (the RGB
// first layer) reach the tensor-core engine through zero-padded copies of the
// activations and weights held in the workspace: zero channels add nothing to an
// integer sum, so the result is unchanged.
#include <stdlib.h>
#include "common.cuh"
#include "qconv_internal.cuh"

using namespace lpdt;

namespace lpdt {

// dst[row][0..Cp) = src[row][0..C) followed by zeros.  One thread per 16-byte piece of a
// destination row (Cp is a multiple of 16), written with a single 16-byte store.
__global__ void pad_channels_kernel(const int8_t *__restrict__ src, int8_t *__restrict__ dst, int64_t rows,
                                    int C, int Cp) {
    pdl_enter();
    const int pieces = Cp / 16;
    const int64_t total = rows * pieces;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = o / pieces;
        const int c0 = (int)(o % pieces) * 16;
        union { int8_t b[16]; uint4 v; } u;
#pragma unroll
        for (int k = 0; k < 16; ++k) u.b[k] = (c0 + k < C) ? src[row * C + c0 + k] : (int8_t)0;
        *reinterpret_cast<uint4 *>(dst + row * Cp + c0) = u.v;
    }
}

}  // namespace lpdt

static unsigned grid_for(int64_t n) {
    int64_t b = ceil_div(n, 256), cap = (int64_t)kNumSMs * 32;
    return (unsigned)(b < 1 ? 1 : (b > cap ? cap : b));
}

// LPDT_DISABLE_TC=1 in the environment routes every shape to the CUDA-core kernels.
static bool tc_enabled() {
    static int disabled = -1;
    if (disabled < 0) {
        const char *e = getenv("LPDT_DISABLE_TC");
        disabled = (e && e[0] == '1') ? 1 : 0;
    }
    return !disabled;
}
static bool use_tc(const lpdt_conv_desc &d) { return tc_enabled() && tc::tc_supported(d); }
// LPDT_DISABLE_HALO=1 keeps 16-channel layers on the general tensor-core kernel.
static bool use_halo(const lpdt_conv_desc &d, int mode) {
    static int disabled = -1;
    if (disabled < 0) {
        const char *e = getenv("LPDT_DISABLE_HALO");
        disabled = (e && e[0] == '1') ? 1 : 0;
    }
    return !disabled && tc::halo_supported(d, mode);
}
static lpdt_status run_pix(const lpdt_conv_desc &d, int mode, const int8_t *A, const float *s1, const int8_t *Wq,
                           const float *s2, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                           int32_t *dev_status, cudaStream_t st, bool uns = false, const float *addend = nullptr) {
    if (use_halo(d, mode)) {
        lpdt_status r = tc::tc_pix_halo(d, mode, A, s1, Wq, s2, bias, bias_stride, Y, Yacc, dev_status, st, uns, addend);
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    }
    return tc::tc_pix(d, mode, A, s1, Wq, s2, bias, bias_stride, Y, Yacc, dev_status, st, uns, addend);
}

static int pad16(int c) { return (c + 15) / 16 * 16; }
// Input channels padded to a multiple of 16 make the shape eligible.
static bool use_tc_padded(const lpdt_conv_desc &d, lpdt_conv_desc *dp) {
    if (!tc_enabled() || d.Cin % 16 == 0) return false;
    *dp = d;
    dp->Cin = pad16(d.Cin);
    return tc::tc_supported(*dp);
}

static lpdt_status check_desc(const lpdt_conv_desc *d) {
    LPDT_CHECK_ARG(d != nullptr);
    LPDT_CHECK_ARG(d->nodes >= 0 && d->B >= 0 && d->H > 0 && d->W > 0 && d->Cin > 0 && d->Cout > 0);
    LPDT_CHECK_ARG(d->R > 0 && d->S > 0 && d->stride > 0 && d->pad >= 0);
    LPDT_CHECK_ARG(d->H + 2 * d->pad >= d->R && d->W + 2 * d->pad >= d->S);
    return LPDT_OK;
}

struct PadPlan { size_t a_bytes, w_bytes, acc_bytes; };
static PadPlan pad_plan(const lpdt_conv_desc &d) {
    const size_t Cp = pad16(d.Cin);
    PadPlan p;
    p.a_bytes = align_up((size_t)d.nodes * d.B * d.H * d.W * Cp, 256);
    p.w_bytes = align_up((size_t)d.nodes * d.Cout * d.R * d.S * Cp, 256);
    p.acc_bytes = align_up((size_t)d.nodes * d.Cout * d.R * d.S * Cp * sizeof(int32_t), 256);
    return p;
}

extern "C" size_t lpdt_qconv_workspace_size(const lpdt_conv_desc *d, int32_t which) {
    if (!d || d->nodes <= 0 || check_desc(d) != LPDT_OK) return 256;
    const size_t wn = (size_t)d->nodes * d->Cout * d->R * d->S * d->Cin;
    size_t need = 256;
    if (which == 1) need = align_up(wn, 256);                       // transposed weights
    if (which == 2) need = align_up(wn * sizeof(int32_t), 256);     // int32 partial sums
    if (d->Cin % 16) {
        const PadPlan p = pad_plan(*d);
        if (which == 0 && p.a_bytes + p.w_bytes > need) need = p.a_bytes + p.w_bytes;
        if (which == 2) need += p.a_bytes;                              // + zero-padded copy of the input
    }
    return need;
}

// Forward contraction on raw codes (signed, or unsigned when `uns`): kernel choice only.
static lpdt_status fwd_impl(const lpdt_conv_desc *d, const int8_t *A, const float *sA, const int8_t *Wq,
                            const float *sW, const float *bias, int64_t bias_node_stride, float *Y, int32_t *Yacc,
                            void *ws, size_t ws_bytes, int32_t *dev_status, cudaStream_t st, bool uns) {
    const bool out_ok = (!Y || aligned(Y, 16)) && (!Yacc || aligned(Yacc, 16));
    if (use_tc(*d) && aligned(A, 16) && aligned(Wq, 16) && out_ok)
        return run_pix(*d, 0, A, sA, Wq, sW, bias, bias_node_stride, Y, Yacc, dev_status, st, uns);
    lpdt_conv_desc dp;
    if (use_tc_padded(*d, &dp) && out_ok && ws && aligned(ws, 256) &&
        ws_bytes >= lpdt_qconv_workspace_size(d, 0)) {
        const PadPlan pp = pad_plan(*d);
        int8_t *Ap = (int8_t *)ws, *Wp = Ap + pp.a_bytes;
        const int64_t arows = (int64_t)d->nodes * d->B * d->H * d->W, wrows = (int64_t)d->nodes * d->Cout * d->R * d->S;
        launch_k(pad_channels_kernel, grid_for(arows * dp.Cin / 16), 256, 0, st, A, Ap, arows, d->Cin, dp.Cin);
        LPDT_LAUNCH_CHECK();
        launch_k(pad_channels_kernel, grid_for(wrows * dp.Cin / 16), 256, 0, st, Wq, Wp, wrows, d->Cin, dp.Cin);
        LPDT_LAUNCH_CHECK();
        return run_pix(dp, 0, Ap, sA, Wp, sW, bias, bias_node_stride, Y, Yacc, dev_status, st, uns);
    }
    return generic_fwd(*d, A, sA, Wq, sW, bias, bias_node_stride, Y, Yacc, st, uns);
}

extern "C" lpdt_status lpdt_qconv_fwd(const lpdt_conv_desc *d, const int8_t *A, const float *sA,
                                      const int8_t *Wq, const float *sW, const float *bias,
                                      int64_t bias_node_stride, float *Y, int32_t *Yacc, void *ws,
                                      size_t ws_bytes, int32_t *dev_status, void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0 || d->B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(A && Wq && (Y || Yacc));
    LPDT_CHECK_ARG(!Y || (sA && sW));
    LPDT_CHECK_ARG(!bias || bias_node_stride >= d->Cout || d->nodes == 1);
    return fwd_impl(d, A, sA, Wq, sW, bias, bias_node_stride, Y, Yacc, ws, ws_bytes, dev_status, as_stream(stream),
                    false);
}

// ---- affine (zero-point) operands -------------------------------------------------------------
// sum (qa - zA)(qw - zW) over the taps inside the image
//   = sum qa*qw  -  zW * sum qa  -  zA * sum qw  +  (taps inside * Cin) * zA * zW.
// The first term is the contraction engine on the unsigned codes (taps outside the image read code 0
// and add nothing); the other three come from per-pixel channel sums of the input and from prefix
// sums over the filter taps of the weights' channel sums (the taps inside the image form a rectangle
// of the filter).  All arithmetic is modulo 2^32, like the accumulators.
namespace lpdt {

// out[row] = sum of the `len` unsigned bytes of row `row`.  A group of G lanes (a power of two up to
// 32, chosen by the launcher from the row length) shares a row: 16-byte loads when the rows allow.
__global__ void row_sum_u8_kernel(const uint8_t *__restrict__ src, int64_t rows, int len, int G, bool vec16,
                                  int32_t *__restrict__ out) {
    pdl_enter();
    const int lane_in_group = threadIdx.x & (G - 1);
    const int64_t groups_total = ((int64_t)gridDim.x * blockDim.x) / G;
    for (int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;; row += groups_total) {
        if (row - (int)((threadIdx.x & 31) / G) >= rows) break;      // warp-uniform: the warp's first row is past the end
        const bool valid = row < rows;                               // lanes past the end still take part in the shuffles
        const uint8_t *a = src + (valid ? row : 0) * len;
        unsigned sum = 0;
        if (!valid) {
        } else if (vec16) {
            const uint4 *a16 = reinterpret_cast<const uint4 *>(a);
            for (int i = lane_in_group; i < len / 16; i += G) {
                const uint4 v = __ldg(a16 + i);
                sum = __dp4a(v.x, 0x01010101u, sum); sum = __dp4a(v.y, 0x01010101u, sum);
                sum = __dp4a(v.z, 0x01010101u, sum); sum = __dp4a(v.w, 0x01010101u, sum);
            }
        } else {
            for (int i = lane_in_group; i < len; i += G) sum += a[i];
        }
        for (int o = G >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (valid && lane_in_group == 0) out[row] = (int32_t)sum;
    }
}

// P[n][r][s][co] for 0 <= r <= R, 0 <= s <= S: sum of tapsum[n][co][r'][s'] over r' < r, s' < s.  The output
// channel is the fastest index, so the correction pass reads four neighbours with one 16-byte load.
__global__ void weight_prefix_kernel(const int32_t *__restrict__ tapsum, int nodes, int Cout, int R, int S,
                                     int32_t *__restrict__ P) {
    pdl_enter();
    const int row = blockIdx.x * blockDim.x + threadIdx.x;        // (node, co)
    if (row >= nodes * Cout) return;
    const int n = row / Cout, co = row % Cout, PS = S + 1;
    const int32_t *t = tapsum + (int64_t)row * R * S;
    int32_t *p = P + (int64_t)n * (R + 1) * PS * Cout + co;
    for (int s = 0; s <= S; ++s) p[(int64_t)s * Cout] = 0;
    for (int r = 1; r <= R; ++r) {
        p[(int64_t)(r * PS) * Cout] = 0;
        unsigned run = 0;                                     // taps (r-1, < s)
        for (int s = 1; s <= S; ++s) {
            run += (unsigned)t[(r - 1) * S + (s - 1)];
            p[(int64_t)(r * PS + s) * Cout] = (int32_t)((unsigned)p[(int64_t)((r - 1) * PS + s) * Cout] + run);
        }
    }
}

// One thread per (output pixel, V consecutive output channels); V = 4 with 16-byte accesses when the
// channel count allows, else 1.
template <int V>
__global__ void affine_fix_kernel(lpdt_conv_desc d, int Ho, int Wo, const int32_t *__restrict__ raw,
                                  const int32_t *__restrict__ asum, const int32_t *__restrict__ P,
                                  const int32_t *__restrict__ zA, const int32_t *__restrict__ zW,
                                  const float *__restrict__ sA, const float *__restrict__ sW,
                                  const float *__restrict__ bias, int64_t bias_stride, float *__restrict__ Y,
                                  int32_t *__restrict__ Yacc) {
    pdl_enter();
    const int chunks = d.Cout / V;
    const int64_t total = (int64_t)d.nodes * d.B * Ho * Wo * chunks;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int co0 = (int)(o % chunks) * V;
        const int64_t pix = o / chunks;
        const int ow = (int)(pix % Wo);
        const int oh = (int)((pix / Wo) % Ho);
        const int64_t nb = pix / ((int64_t)Wo * Ho);
        const int n = (int)(nb / d.B);
        // filter rows / columns whose tap lies inside the image
        int r_lo = d.pad - oh * d.stride; if (r_lo < 0) r_lo = 0;
        int r_hi = d.H + d.pad - oh * d.stride; if (r_hi > d.R) r_hi = d.R;
        int s_lo = d.pad - ow * d.stride; if (s_lo < 0) s_lo = 0;
        int s_hi = d.W + d.pad - ow * d.stride; if (s_hi > d.S) s_hi = d.S;
        if (r_hi < r_lo) r_hi = r_lo;
        if (s_hi < s_lo) s_hi = s_lo;
        unsigned ra = 0;
        for (int r = r_lo; r < r_hi; ++r)
            for (int s = s_lo; s < s_hi; ++s)
                ra += (unsigned)__ldg(asum + (nb * d.H + oh * d.stride + r - d.pad) * d.W + ow * d.stride + s - d.pad);
        const unsigned za = (unsigned)zA[n], zw = (unsigned)zW[n];
        const unsigned cnt = (unsigned)((r_hi - r_lo) * (s_hi - s_lo) * d.Cin);
        const unsigned fixed = cnt * za * zw - zw * ra;
        const float sc = Y ? __fmul_rn(sA[n], sW[n]) : 0.f;
        const int PS = d.S + 1;
        const int64_t oi = pix * d.Cout + co0;
        int rawv[V], acc[V];
        if (V == 4) { const int4 t = *reinterpret_cast<const int4 *>(raw + oi); rawv[0] = t.x; rawv[1] = t.y; rawv[2] = t.z; rawv[3] = t.w; }
        else rawv[0] = raw[oi];
        // rectangle sum of the weights' channel sums over the taps inside the image: four corners of the prefix table
        const int32_t *p = P + (int64_t)n * (d.R + 1) * PS * d.Cout + co0;
        int c11[V], c01[V], c10[V], c00[V];
        auto corner = [&](int r, int s2, int (&o)[V]) {
            const int32_t *q = p + (int64_t)(r * PS + s2) * d.Cout;
            if (V == 4) { const int4 t = __ldg(reinterpret_cast<const int4 *>(q)); o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w; }
            else o[0] = __ldg(q);
        };
        corner(r_hi, s_hi, c11); corner(r_lo, s_hi, c01); corner(r_hi, s_lo, c10); corner(r_lo, s_lo, c00);
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const unsigned rw = (unsigned)c11[k] - (unsigned)c01[k] - (unsigned)c10[k] + (unsigned)c00[k];
            acc[k] = (int)((unsigned)rawv[k] + fixed - za * rw);
        }
        if (Yacc) {
            if (V == 4) *reinterpret_cast<int4 *>(Yacc + oi) = make_int4(acc[0], acc[1], acc[2], acc[3]);
            else Yacc[oi] = acc[0];
        }
        if (Y) {
            float v[V];
#pragma unroll
            for (int k = 0; k < V; ++k) {
                v[k] = __fmul_rn(__int2float_rn(acc[k]), sc);
                if (bias) v[k] = __fadd_rn(v[k], bias[(int64_t)n * bias_stride + co0 + k]);
            }
            if (V == 4) *reinterpret_cast<float4 *>(Y + oi) = make_float4(v[0], v[1], v[2], v[3]);
            else Y[oi] = v[0];
        }
    }
}

// rows of `len` bytes -> out[row]; lanes per row grow with the row length
static lpdt_status row_sum_launch(const uint8_t *src, int64_t rows, int len, int32_t *out, cudaStream_t st) {
    const bool vec16 = len % 16 == 0 && aligned(src, 16);
    const int units = vec16 ? len / 16 : len;
    int G = 1;
    while (G < 32 && G * 4 <= units) G <<= 1;             // at least four loads per lane
    int64_t blocks = ceil_div(rows * G, 256);
    const int64_t cap = (int64_t)kNumSMs * 32;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    launch_k(row_sum_u8_kernel, (unsigned)blocks, 256, 0, st, src, rows, len, G, vec16, out);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

}  // namespace lpdt

static size_t affine_raw_bytes(const lpdt_conv_desc *d) {
    const int Ho = conv_out(d->H, d->pad, d->R, d->stride), Wo = conv_out(d->W, d->pad, d->S, d->stride);
    return align_up((size_t)d->nodes * d->B * Ho * Wo * d->Cout * sizeof(int32_t), 256);
}
static size_t affine_asum_bytes(const lpdt_conv_desc *d) {
    return align_up((size_t)d->nodes * d->B * d->H * d->W * sizeof(int32_t), 256);
}
static size_t affine_prefix_bytes(const lpdt_conv_desc *d) {     // prefix table + per-tap channel sums
    return align_up((size_t)d->nodes * d->Cout * (d->R + 1) * (d->S + 1) * sizeof(int32_t), 256) +
           align_up((size_t)d->nodes * d->Cout * d->R * d->S * sizeof(int32_t), 256);
}

extern "C" size_t lpdt_qconv_fwd_affine_workspace_size(const lpdt_conv_desc *d) {
    if (!d || d->nodes <= 0 || check_desc(d) != LPDT_OK) return 256;
    return affine_raw_bytes(d) + affine_asum_bytes(d) + affine_prefix_bytes(d) + lpdt_qconv_workspace_size(d, 0);
}

extern "C" lpdt_status lpdt_qconv_fwd_affine(const lpdt_conv_desc *d, const uint8_t *A, const float *sA,
                                             const int32_t *zA, const uint8_t *Wq, const float *sW,
                                             const int32_t *zW, const float *bias, int64_t bias_node_stride,
                                             float *Y, int32_t *Yacc, void *ws, size_t ws_bytes,
                                             int32_t *dev_status, void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0 || d->B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(A && Wq && zA && zW && (Y || Yacc));
    LPDT_CHECK_ARG(!Y || (sA && sW));
    LPDT_CHECK_ARG(!bias || bias_node_stride >= d->Cout || d->nodes == 1);
    if (!ws || !aligned(ws, 256) || ws_bytes < lpdt_qconv_fwd_affine_workspace_size(d)) return LPDT_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    const int Ho = conv_out(d->H, d->pad, d->R, d->stride), Wo = conv_out(d->W, d->pad, d->S, d->stride);
    int32_t *raw = (int32_t *)ws;
    int32_t *asum = (int32_t *)((char *)ws + affine_raw_bytes(d));
    int32_t *P = (int32_t *)((char *)asum + affine_asum_bytes(d));
    void *inner = (char *)P + affine_prefix_bytes(d);
    const int64_t pixels = (int64_t)d->nodes * d->B * d->H * d->W;
    s = row_sum_launch(A, pixels, d->Cin, asum, st);
    if (s != LPDT_OK) return s;
    const int rows = d->nodes * d->Cout;
    int32_t *tapsum = (int32_t *)((char *)P + align_up((size_t)rows * (d->R + 1) * (d->S + 1) * sizeof(int32_t), 256));
    s = row_sum_launch(Wq, (int64_t)rows * d->R * d->S, d->Cin, tapsum, st);
    if (s != LPDT_OK) return s;
    launch_k(weight_prefix_kernel, (rows + 127) / 128, 128, 0, st, tapsum, d->nodes, d->Cout, d->R, d->S, P);
    LPDT_LAUNCH_CHECK();
    // Tensor-core path: the zero-point terms are applied in the contraction's own epilogue (no raw sums in
    // memory, no second pass over the result).  LPDT_AFFINE_SEPARATE=1 keeps the separate correction pass.
    static int separate = -1;
    if (separate < 0) { const char *e = getenv("LPDT_AFFINE_SEPARATE"); separate = (e && e[0] == '1') ? 1 : 0; }
    if (!separate && use_tc(*d) && d->Cout % 4 == 0 && aligned(A, 16) && aligned(Wq, 16) && (!Y || aligned(Y, 16)) &&
        (!Yacc || aligned(Yacc, 16))) {
        const tc::AffineArgs aff = {asum, P, zA, zW};
        lpdt_status r = tc::tc_pix(*d, 0, reinterpret_cast<const int8_t *>(A), sA, reinterpret_cast<const int8_t *>(Wq), sW,
                                   bias, bias_node_stride, Y, Yacc, dev_status, st, true, nullptr, &aff);
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    }
    s = fwd_impl(d, reinterpret_cast<const int8_t *>(A), nullptr, reinterpret_cast<const int8_t *>(Wq), nullptr, nullptr,
                 0, nullptr, raw, inner, lpdt_qconv_workspace_size(d, 0), dev_status, st, true);
    if (s != LPDT_OK) return s;
    const bool v4 = d->Cout % 4 == 0 && (!Y || aligned(Y, 16)) && (!Yacc || aligned(Yacc, 16));
    const int64_t work = (int64_t)d->nodes * d->B * Ho * Wo * (d->Cout / (v4 ? 4 : 1));
    if (v4)
        launch_k(affine_fix_kernel<4>, grid_for(work), 256, 0, st, *d, Ho, Wo, raw, asum, P, zA, zW, sA, sW, bias,
                                                             bias_node_stride, Y, Yacc);
    else
        launch_k(affine_fix_kernel<1>, grid_for(work), 256, 0, st, *d, Ho, Wo, raw, asum, P, zA, zW, sA, sW, bias,
                                                             bias_node_stride, Y, Yacc);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

// Backward-data contraction on raw codes (signed, or unsigned when `uns`): kernel choice only.
static lpdt_status bwd_data_impl(const lpdt_conv_desc *d, const int8_t *E, const float *sE, const int8_t *Wq,
                                 const float *sW, float *dA, int32_t *dAacc, const float *addend, void *ws,
                                 int32_t *dev_status, cudaStream_t st, bool uns) {
    if (use_tc(*d) && aligned(E, 16) && aligned(Wq, 16) && (!dA || aligned(dA, 16)) && (!dAacc || aligned(dAacc, 16)))
        return run_pix(*d, 1, E, sE, Wq, sW, nullptr, 0, dA, dAacc, dev_status, st, uns, addend);
    return generic_bwd_data(*d, E, sE, Wq, sW, dA, dAacc, addend, ws, st, uns);
}

extern "C" lpdt_status lpdt_qconv_bwd_data(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                           const int8_t *Wq, const float *sW, float *dA, int32_t *dAacc,
                                           const float *addend, void *ws, size_t ws_bytes, int32_t *dev_status,
                                           void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0 || d->B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(E && Wq && (dA || dAacc));
    LPDT_CHECK_ARG(!dA || (sE && sW));
    LPDT_CHECK_ARG(!addend || (dA && addend != dA && aligned(addend, 16)));
    if (!ws || ws_bytes < lpdt_qconv_workspace_size(d, 1)) return LPDT_ERR_WORKSPACE;
    return bwd_data_impl(d, E, sE, Wq, sW, dA, dAacc, addend, ws, dev_status, as_stream(stream), false);
}

// Backward-weight contraction on raw codes.  Workspace: [int32 sums (used unless the caller gave dWacc) |
// zero-padded input copy].
static lpdt_status bwd_weight_impl(const lpdt_conv_desc *d, const int8_t *E, const float *sE, const int8_t *A,
                                   const float *sA, float *dW, int64_t dw_node_stride, int32_t *dWacc, void *ws,
                                   int32_t *dev_status, cudaStream_t st, bool uns) {
    const size_t acc_bytes = align_up((size_t)d->nodes * d->Cout * d->R * d->S * d->Cin * sizeof(int32_t), 256);
    int32_t *acc_ws = (int32_t *)ws;
    lpdt_conv_desc dp;
    if (use_tc(*d) && d->B > 0 && aligned(E, 16) && aligned(A, 16)) {
        lpdt_status r = tc::tc_wgrad(*d, d->Cin, E, sE, A, sA, dWacc, acc_ws, dW, dw_node_stride, dev_status, st, uns);
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    } else if (use_tc_padded(*d, &dp) && d->B > 0 && aligned(E, 16)) {
        int8_t *Ap = (int8_t *)((char *)ws + acc_bytes);
        const int64_t arows = (int64_t)d->nodes * d->B * d->H * d->W;
        launch_k(pad_channels_kernel, grid_for(arows * dp.Cin / 16), 256, 0, st, A, Ap, arows, d->Cin, dp.Cin);
        LPDT_LAUNCH_CHECK();
        lpdt_status r = tc::tc_wgrad(dp, d->Cin, E, sE, Ap, sA, dWacc, acc_ws, dW, dw_node_stride, dev_status, st, uns);
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    }
    return generic_bwd_weight(*d, E, sE, A, sA, dW, dw_node_stride, dWacc, acc_ws, st, uns);
}

extern "C" lpdt_status lpdt_qconv_bwd_weight(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                             const int8_t *A, const float *sA, float *dW,
                                             int64_t dw_node_stride, int32_t *dWacc, void *ws,
                                             size_t ws_bytes, int32_t *dev_status, void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG((d->B == 0 || (E && A)) && (dW || dWacc));      // an empty batch has no operands to point at
    LPDT_CHECK_ARG(!dW || (sE && sA));
    LPDT_CHECK_ARG(!dW || dw_node_stride >= (int64_t)d->Cout * d->R * d->S * d->Cin || d->nodes == 1);
    if (!ws || ws_bytes < lpdt_qconv_workspace_size(d, 2) || !aligned(ws, 256)) return LPDT_ERR_WORKSPACE;
    return bwd_weight_impl(d, E, sE, A, sA, dW, dw_node_stride, dWacc, ws, dev_status, as_stream(stream), false);
}

// ---- backward products on affine (zero-point) operands -----------------------------------------
// With e' = qe - zE, w' = qw - zW, a' = qa - zA and the sums running over the taps that exist,
//   sum e'w' = sum qe*qw - zW * sum qe - zE * sum qw + (terms) * zE*zW          (backward-data)
//   sum e'a' = sum qe*qa - zA * sum qe - zE * sum qa + (terms) * zE*zA          (backward-weight)
// the first term is the contraction engine on the unsigned codes; the others come from channel sums
// of the operands, gathered over the same taps.  All arithmetic is modulo 2^32.
namespace lpdt {

// wsum[n][r][s][ci] = sum over co of W[n][co][r][s][ci]; one thread per output, ci fastest.
__global__ void weight_cout_sum_kernel(lpdt_conv_desc d, const uint8_t *__restrict__ Wq, int32_t *__restrict__ wsum) {
    pdl_enter();
    const int per = d.R * d.S * d.Cin;
    const int64_t total = (int64_t)d.nodes * per;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(o / per), i = (int)(o % per);
        const uint8_t *w = Wq + (int64_t)n * d.Cout * per + i;
        unsigned sum = 0;
        for (int co = 0; co < d.Cout; ++co) sum += w[(int64_t)co * per];
        wsum[o] = (int32_t)sum;
    }
}

// One thread per (input pixel, V consecutive input channels).
template <int V>
__global__ void affine_fix_bwd_data_kernel(lpdt_conv_desc d, int Ho, int Wo, const int32_t *__restrict__ raw,
                                           const int32_t *__restrict__ esum, const int32_t *__restrict__ wsum,
                                           const int32_t *__restrict__ zE, const int32_t *__restrict__ zW,
                                           const float *__restrict__ sE, const float *__restrict__ sW,
                                           float *__restrict__ dA, int32_t *__restrict__ dAacc) {
    pdl_enter();
    const int chunks = d.Cin / V;
    const int64_t total = (int64_t)d.nodes * d.B * d.H * d.W * chunks;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int ci0 = (int)(o % chunks) * V;
        const int64_t pix = o / chunks;
        const int iw = (int)(pix % d.W);
        const int ih = (int)((pix / d.W) % d.H);
        const int64_t nb = pix / ((int64_t)d.W * d.H);
        const int n = (int)(nb / d.B);
        unsigned es = 0, cnt = 0, ws_[V];
#pragma unroll
        for (int k = 0; k < V; ++k) ws_[k] = 0;
        for (int r = 0; r < d.R; ++r) {
            const int th = ih + d.pad - r;
            if (th < 0 || th % d.stride) continue;
            const int oh = th / d.stride;
            if (oh >= Ho) continue;
            for (int s = 0; s < d.S; ++s) {
                const int tw = iw + d.pad - s;
                if (tw < 0 || tw % d.stride) continue;
                const int ow = tw / d.stride;
                if (ow >= Wo) continue;
                es += (unsigned)__ldg(esum + (nb * Ho + oh) * Wo + ow);
                cnt += (unsigned)d.Cout;
                const int32_t *wp = wsum + (((int64_t)n * d.R + r) * d.S + s) * d.Cin + ci0;
#pragma unroll
                for (int k = 0; k < V; ++k) ws_[k] += (unsigned)__ldg(wp + k);
            }
        }
        const unsigned ze = (unsigned)zE[n], zw = (unsigned)zW[n];
        const unsigned fixed = cnt * ze * zw - zw * es;
        const float sc = dA ? __fmul_rn(sE[n], sW[n]) : 0.f;
        const int64_t oi = pix * d.Cin + ci0;
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const int acc = (int)((unsigned)raw[oi + k] + fixed - ze * ws_[k]);
            if (dAacc) dAacc[oi + k] = acc;
            if (dA) dA[oi + k] = __fmul_rn(__int2float_rn(acc), sc);
        }
    }
}

// col[n][pos][c] = sum over the batch of src[n][b][pos][c] (unsigned codes); one thread per output, c fastest.
__global__ void batch_sum_u8_kernel(const uint8_t *__restrict__ src, int nodes, int B, int64_t per_image,
                                    int32_t *__restrict__ col) {
    pdl_enter();
    const int64_t total = (int64_t)nodes * per_image;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int64_t n = o / per_image, i = o % per_image;
        const uint8_t *p = src + n * B * per_image + i;
        unsigned sum = 0;
        for (int b = 0; b < B; ++b) sum += p[(int64_t)b * per_image];
        col[o] = (int32_t)sum;
    }
}

// Sums of a batch-summed image over the output positions whose tap (r, s) lies inside the input image:
//   of_input = 0: tab[n][r][s][c] = sum col[n][oh][ow][c]                        (col over the OUTPUT image, C = Cout)
//   of_input = 1: tab[n][r][s][c] = sum col[n][oh*st+r-pad][ow*st+s-pad][c]      (col over the INPUT image, C = Cin)
// block (tap, node), threads over channels.
__global__ void tap_table_kernel(lpdt_conv_desc d, int Ho, int Wo, int of_input, int C,
                                 const int32_t *__restrict__ col, int32_t *__restrict__ tab) {
    pdl_enter();
    const int tap = blockIdx.x, n = blockIdx.y, r = tap / d.S, s = tap % d.S;
    const int Hc = of_input ? d.H : Ho, Wc = of_input ? d.W : Wo;
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        unsigned sum = 0;
        for (int oh = 0; oh < Ho; ++oh) {
            const int ih = oh * d.stride + r - d.pad;
            if (ih < 0 || ih >= d.H) continue;
            for (int ow = 0; ow < Wo; ++ow) {
                const int iw = ow * d.stride + s - d.pad;
                if (iw < 0 || iw >= d.W) continue;
                const int ph = of_input ? ih : oh, pw = of_input ? iw : ow;
                sum += (unsigned)col[(((int64_t)n * Hc + ph) * Wc + pw) * C + c];
            }
        }
        tab[((int64_t)n * d.R * d.S + tap) * C + c] = (int32_t)sum;
    }
}

// One thread per weight-gradient entry (n, co, r, s, ci); ci fastest.
__global__ void affine_fix_bwd_weight_kernel(lpdt_conv_desc d, int Ho, int Wo, const int32_t *__restrict__ raw,
                                             const int32_t *__restrict__ tabE, const int32_t *__restrict__ tabA,
                                             const int32_t *__restrict__ zE, const int32_t *__restrict__ zA,
                                             const float *__restrict__ sE, const float *__restrict__ sA,
                                             float *__restrict__ dW, int64_t dw_stride, int32_t *__restrict__ dWacc) {
    pdl_enter();
    const int taps = d.R * d.S;
    const int64_t per_node = (int64_t)d.Cout * taps * d.Cin;
    const int64_t total = per_node * d.nodes;
    for (int64_t o = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; o < total; o += (int64_t)gridDim.x * blockDim.x) {
        const int n = (int)(o / per_node);
        const int64_t i = o % per_node;
        const int ci = (int)(i % d.Cin);
        const int tap = (int)((i / d.Cin) % taps);
        const int co = (int)(i / ((int64_t)d.Cin * taps));
        const int r = tap / d.S, s = tap % d.S;
        // output rows / columns whose tap lies inside the input image
        int nh = 0, nw = 0;
        for (int oh = 0; oh < Ho; ++oh) { const int ih = oh * d.stride + r - d.pad; nh += (ih >= 0 && ih < d.H); }
        for (int ow = 0; ow < Wo; ++ow) { const int iw = ow * d.stride + s - d.pad; nw += (iw >= 0 && iw < d.W); }
        const unsigned cnt = (unsigned)d.B * (unsigned)nh * (unsigned)nw;
        const unsigned ze = (unsigned)zE[n], za = (unsigned)zA[n];
        const unsigned te = (unsigned)tabE[((int64_t)n * taps + tap) * d.Cout + co];
        const unsigned ta = (unsigned)tabA[((int64_t)n * taps + tap) * d.Cin + ci];
        const int acc = (int)((unsigned)raw[o] - za * te - ze * ta + cnt * ze * za);
        if (dWacc) dWacc[o] = acc;
        if (dW) dW[(int64_t)n * dw_stride + i] = __fmul_rn(__int2float_rn(acc), __fmul_rn(sE[n], sA[n]));
    }
}

}  // namespace lpdt

static size_t affine_bwd_data_raw_bytes(const lpdt_conv_desc *d) {
    return align_up((size_t)d->nodes * d->B * d->H * d->W * d->Cin * sizeof(int32_t), 256);
}
static size_t affine_esum_bytes(const lpdt_conv_desc *d) {
    const int Ho = conv_out(d->H, d->pad, d->R, d->stride), Wo = conv_out(d->W, d->pad, d->S, d->stride);
    return align_up((size_t)d->nodes * d->B * Ho * Wo * sizeof(int32_t), 256);
}
static size_t affine_wsum_bytes(const lpdt_conv_desc *d) {
    return align_up((size_t)d->nodes * d->R * d->S * d->Cin * sizeof(int32_t), 256);
}

extern "C" size_t lpdt_qconv_bwd_data_affine_workspace_size(const lpdt_conv_desc *d) {
    if (!d || d->nodes <= 0 || check_desc(d) != LPDT_OK) return 256;
    return affine_bwd_data_raw_bytes(d) + affine_esum_bytes(d) + affine_wsum_bytes(d) + lpdt_qconv_workspace_size(d, 1);
}

extern "C" lpdt_status lpdt_qconv_bwd_data_affine(const lpdt_conv_desc *d, const uint8_t *E, const float *sE,
                                                  const int32_t *zE, const uint8_t *Wq, const float *sW,
                                                  const int32_t *zW, float *dA, int32_t *dAacc, void *ws,
                                                  size_t ws_bytes, int32_t *dev_status, void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0 || d->B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(E && Wq && zE && zW && (dA || dAacc));
    LPDT_CHECK_ARG(!dA || (sE && sW));
    if (!ws || !aligned(ws, 256) || ws_bytes < lpdt_qconv_bwd_data_affine_workspace_size(d)) return LPDT_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    const int Ho = conv_out(d->H, d->pad, d->R, d->stride), Wo = conv_out(d->W, d->pad, d->S, d->stride);
    int32_t *raw = (int32_t *)ws;
    int32_t *esum = (int32_t *)((char *)ws + affine_bwd_data_raw_bytes(d));
    int32_t *wsum = (int32_t *)((char *)esum + affine_esum_bytes(d));
    void *inner = (char *)wsum + affine_wsum_bytes(d);
    s = bwd_data_impl(d, reinterpret_cast<const int8_t *>(E), nullptr, reinterpret_cast<const int8_t *>(Wq), nullptr,
                      nullptr, raw, nullptr, inner, dev_status, st, true);
    if (s != LPDT_OK) return s;
    s = row_sum_launch(E, (int64_t)d->nodes * d->B * Ho * Wo, d->Cout, esum, st);
    if (s != LPDT_OK) return s;
    launch_k(weight_cout_sum_kernel, grid_for((int64_t)d->nodes * d->R * d->S * d->Cin), 256, 0, st, *d, Wq, wsum);
    LPDT_LAUNCH_CHECK();
    const bool v4 = d->Cin % 4 == 0;
    const int64_t work = (int64_t)d->nodes * d->B * d->H * d->W * (d->Cin / (v4 ? 4 : 1));
    if (v4)
        launch_k(affine_fix_bwd_data_kernel<4>, grid_for(work), 256, 0, st, *d, Ho, Wo, raw, esum, wsum, zE, zW, sE, sW, dA, dAacc);
    else
        launch_k(affine_fix_bwd_data_kernel<1>, grid_for(work), 256, 0, st, *d, Ho, Wo, raw, esum, wsum, zE, zW, sE, sW, dA, dAacc);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

static size_t affine_wg_raw_bytes(const lpdt_conv_desc *d) {
    return align_up((size_t)d->nodes * d->Cout * d->R * d->S * d->Cin * sizeof(int32_t), 256);
}
static size_t affine_colE_bytes(const lpdt_conv_desc *d) {
    const int Ho = conv_out(d->H, d->pad, d->R, d->stride), Wo = conv_out(d->W, d->pad, d->S, d->stride);
    return align_up((size_t)d->nodes * Ho * Wo * d->Cout * sizeof(int32_t), 256);
}
static size_t affine_colA_bytes(const lpdt_conv_desc *d) {
    return align_up((size_t)d->nodes * d->H * d->W * d->Cin * sizeof(int32_t), 256);
}
static size_t affine_tab_bytes(const lpdt_conv_desc *d, int C) {
    return align_up((size_t)d->nodes * d->R * d->S * C * sizeof(int32_t), 256);
}

extern "C" size_t lpdt_qconv_bwd_weight_affine_workspace_size(const lpdt_conv_desc *d) {
    if (!d || d->nodes <= 0 || check_desc(d) != LPDT_OK) return 256;
    return affine_wg_raw_bytes(d) + affine_colE_bytes(d) + affine_colA_bytes(d) + affine_tab_bytes(d, d->Cout) +
           affine_tab_bytes(d, d->Cin) + lpdt_qconv_workspace_size(d, 2);
}

extern "C" lpdt_status lpdt_qconv_bwd_weight_affine(const lpdt_conv_desc *d, const uint8_t *E, const float *sE,
                                                    const int32_t *zE, const uint8_t *A, const float *sA,
                                                    const int32_t *zA, float *dW, int64_t dw_node_stride,
                                                    int32_t *dWacc, void *ws, size_t ws_bytes, int32_t *dev_status,
                                                    void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG((d->B == 0 || (E && A)) && zE && zA && (dW || dWacc));
    LPDT_CHECK_ARG(!dW || (sE && sA));
    LPDT_CHECK_ARG(!dW || dw_node_stride >= (int64_t)d->Cout * d->R * d->S * d->Cin || d->nodes == 1);
    if (d->nodes > 65535) return LPDT_ERR_UNSUPPORTED;
    if (!ws || !aligned(ws, 256) || ws_bytes < lpdt_qconv_bwd_weight_affine_workspace_size(d)) return LPDT_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    const int Ho = conv_out(d->H, d->pad, d->R, d->stride), Wo = conv_out(d->W, d->pad, d->S, d->stride);
    int32_t *raw = (int32_t *)ws;
    int32_t *colE = (int32_t *)((char *)ws + affine_wg_raw_bytes(d));
    int32_t *colA = (int32_t *)((char *)colE + affine_colE_bytes(d));
    int32_t *tabE = (int32_t *)((char *)colA + affine_colA_bytes(d));
    int32_t *tabA = (int32_t *)((char *)tabE + affine_tab_bytes(d, d->Cout));
    void *inner = (char *)tabA + affine_tab_bytes(d, d->Cin);
    s = bwd_weight_impl(d, reinterpret_cast<const int8_t *>(E), nullptr, reinterpret_cast<const int8_t *>(A), nullptr,
                        nullptr, 0, raw, inner, dev_status, st, true);
    if (s != LPDT_OK) return s;
    launch_k(batch_sum_u8_kernel, grid_for((int64_t)d->nodes * Ho * Wo * d->Cout), 256, 0, st, E, d->nodes, d->B,
             (int64_t)Ho * Wo * d->Cout, colE);
    LPDT_LAUNCH_CHECK();
    launch_k(batch_sum_u8_kernel, grid_for((int64_t)d->nodes * d->H * d->W * d->Cin), 256, 0, st, A, d->nodes, d->B,
             (int64_t)d->H * d->W * d->Cin, colA);
    LPDT_LAUNCH_CHECK();
    const dim3 tgrid(d->R * d->S, d->nodes);
    launch_k(tap_table_kernel, tgrid, 128, 0, st, *d, Ho, Wo, 0, d->Cout, colE, tabE);
    LPDT_LAUNCH_CHECK();
    launch_k(tap_table_kernel, tgrid, 128, 0, st, *d, Ho, Wo, 1, d->Cin, colA, tabA);
    LPDT_LAUNCH_CHECK();
    launch_k(affine_fix_bwd_weight_kernel, grid_for((int64_t)d->nodes * d->Cout * d->R * d->S * d->Cin), 256, 0, st, *d, Ho,
             Wo, raw, tabE, tabA, zE, zA, sE, sA, dW, dw_node_stride, dWacc);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
