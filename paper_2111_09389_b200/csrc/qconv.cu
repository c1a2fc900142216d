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
                           int32_t *dev_status, cudaStream_t st) {
    if (use_halo(d, mode)) {
        lpdt_status r = tc::tc_pix_halo(d, mode, A, s1, Wq, s2, bias, bias_stride, Y, Yacc, dev_status, st);
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    }
    return tc::tc_pix(d, mode, A, s1, Wq, s2, bias, bias_stride, Y, Yacc, dev_status, st);
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
    cudaStream_t st = as_stream(stream);
    const bool out_ok = (!Y || aligned(Y, 16)) && (!Yacc || aligned(Yacc, 16));
    if (use_tc(*d) && aligned(A, 16) && aligned(Wq, 16) && out_ok)
        return run_pix(*d, 0, A, sA, Wq, sW, bias, bias_node_stride, Y, Yacc, dev_status, st);
    lpdt_conv_desc dp;
    if (use_tc_padded(*d, &dp) && out_ok && ws && aligned(ws, 256) &&
        ws_bytes >= lpdt_qconv_workspace_size(d, 0)) {
        const PadPlan pp = pad_plan(*d);
        int8_t *Ap = (int8_t *)ws, *Wp = Ap + pp.a_bytes;
        const int64_t arows = (int64_t)d->nodes * d->B * d->H * d->W, wrows = (int64_t)d->nodes * d->Cout * d->R * d->S;
        pad_channels_kernel<<<grid_for(arows * dp.Cin / 16), 256, 0, st>>>(A, Ap, arows, d->Cin, dp.Cin);
        LPDT_LAUNCH_CHECK();
        pad_channels_kernel<<<grid_for(wrows * dp.Cin / 16), 256, 0, st>>>(Wq, Wp, wrows, d->Cin, dp.Cin);
        LPDT_LAUNCH_CHECK();
        return run_pix(dp, 0, Ap, sA, Wp, sW, bias, bias_node_stride, Y, Yacc, dev_status, st);
    }
    return generic_fwd(*d, A, sA, Wq, sW, bias, bias_node_stride, Y, Yacc, st);
}

extern "C" lpdt_status lpdt_qconv_bwd_data(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                           const int8_t *Wq, const float *sW, float *dA, int32_t *dAacc,
                                           void *ws, size_t ws_bytes, int32_t *dev_status, void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0 || d->B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(E && Wq && (dA || dAacc));
    LPDT_CHECK_ARG(!dA || (sE && sW));
    if (!ws || ws_bytes < lpdt_qconv_workspace_size(d, 1)) return LPDT_ERR_WORKSPACE;
    if (use_tc(*d) && aligned(E, 16) && aligned(Wq, 16) && (!dA || aligned(dA, 16)) && (!dAacc || aligned(dAacc, 16)))
        return run_pix(*d, 1, E, sE, Wq, sW, nullptr, 0, dA, dAacc, dev_status, as_stream(stream));
    return generic_bwd_data(*d, E, sE, Wq, sW, dA, dAacc, ws, as_stream(stream));
}

extern "C" lpdt_status lpdt_qconv_bwd_weight(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                             const int8_t *A, const float *sA, float *dW,
                                             int64_t dw_node_stride, int32_t *dWacc, void *ws,
                                             size_t ws_bytes, int32_t *dev_status, void *stream) {
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(E && A && (dW || dWacc));
    LPDT_CHECK_ARG(!dW || (sE && sA));
    LPDT_CHECK_ARG(!dW || dw_node_stride >= (int64_t)d->Cout * d->R * d->S * d->Cin || d->nodes == 1);
    if (!ws || ws_bytes < lpdt_qconv_workspace_size(d, 2) || !aligned(ws, 256)) return LPDT_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    // workspace: [int32 sums (used unless the caller gave dWacc) | zero-padded input copy]
    const size_t acc_bytes = align_up((size_t)d->nodes * d->Cout * d->R * d->S * d->Cin * sizeof(int32_t), 256);
    int32_t *acc_ws = (int32_t *)ws;
    lpdt_conv_desc dp;
    if (use_tc(*d) && d->B > 0 && aligned(E, 16) && aligned(A, 16)) {
        lpdt_status r = tc::tc_wgrad(*d, d->Cin, E, sE, A, sA, dWacc, acc_ws, dW, dw_node_stride, dev_status, st);
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    } else if (use_tc_padded(*d, &dp) && d->B > 0 && aligned(E, 16)) {
        int8_t *Ap = (int8_t *)((char *)ws + acc_bytes);
        const int64_t arows = (int64_t)d->nodes * d->B * d->H * d->W;
        pad_channels_kernel<<<grid_for(arows * dp.Cin / 16), 256, 0, st>>>(A, Ap, arows, d->Cin, dp.Cin);
        LPDT_LAUNCH_CHECK();
        lpdt_status r = tc::tc_wgrad(dp, d->Cin, E, sE, Ap, sA, dWacc, acc_ws, dW, dw_node_stride, dev_status, st);
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    }
    return generic_bwd_weight(*d, E, sE, A, sA, dW, dw_node_stride, dWacc, acc_ws, st);
}
