// Front end of the quantized contractions: argument validation, workspace
// accounting and the choice between the tensor-core engine and the CUDA-core
// kernels.
#include "common.cuh"
#include "qconv_internal.cuh"

#include <stdlib.h>

using namespace lpdt;

// LPDT_DISABLE_TC=1 in the environment routes every shape to the CUDA-core kernels.
static bool use_tc(const lpdt_conv_desc &d) {
    static int disabled = -1;
    if (disabled < 0) {
        const char *e = getenv("LPDT_DISABLE_TC");
        disabled = (e && e[0] == '1') ? 1 : 0;
    }
    return !disabled && tc::tc_supported(d);
}

static lpdt_status check_desc(const lpdt_conv_desc *d) {
    LPDT_CHECK_ARG(d != nullptr);
    LPDT_CHECK_ARG(d->nodes >= 0 && d->B >= 0 && d->H > 0 && d->W > 0 && d->Cin > 0 && d->Cout > 0);
    LPDT_CHECK_ARG(d->R > 0 && d->S > 0 && d->stride > 0 && d->pad >= 0);
    LPDT_CHECK_ARG(d->H + 2 * d->pad >= d->R && d->W + 2 * d->pad >= d->S);
    return LPDT_OK;
}

extern "C" size_t lpdt_qconv_workspace_size(const lpdt_conv_desc *d, int32_t which) {
    if (!d || d->nodes <= 0) return 256;
    const size_t wn = (size_t)d->nodes * d->Cout * d->R * d->S * d->Cin;
    if (which == 1) return align_up(wn, 256);                       // transposed weights
    if (which == 2) return align_up(wn * sizeof(int32_t), 256);     // int32 partial sums
    return 256;
}

extern "C" lpdt_status lpdt_qconv_fwd(const lpdt_conv_desc *d, const int8_t *A, const float *sA,
                                      const int8_t *Wq, const float *sW, const float *bias,
                                      int64_t bias_node_stride, float *Y, int32_t *Yacc, void *ws,
                                      size_t ws_bytes, int32_t *dev_status, void *stream) {
    (void)ws; (void)ws_bytes; (void)dev_status;
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0 || d->B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(A && Wq && (Y || Yacc));
    LPDT_CHECK_ARG(!Y || (sA && sW));
    LPDT_CHECK_ARG(!bias || bias_node_stride >= d->Cout || d->nodes == 1);
    if (use_tc(*d) && aligned(A, 16) && aligned(Wq, 16) && (!Y || aligned(Y, 16)) && (!Yacc || aligned(Yacc, 16)))
        return tc::tc_pix(*d, 0, A, sA, Wq, sW, bias, bias_node_stride, Y, Yacc, dev_status, as_stream(stream));
    return generic_fwd(*d, A, sA, Wq, sW, bias, bias_node_stride, Y, Yacc, as_stream(stream));
}

extern "C" lpdt_status lpdt_qconv_bwd_data(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                           const int8_t *Wq, const float *sW, float *dA, int32_t *dAacc,
                                           void *ws, size_t ws_bytes, int32_t *dev_status, void *stream) {
    (void)dev_status;
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0 || d->B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(E && Wq && (dA || dAacc));
    LPDT_CHECK_ARG(!dA || (sE && sW));
    if (!ws || ws_bytes < lpdt_qconv_workspace_size(d, 1)) return LPDT_ERR_WORKSPACE;
    if (use_tc(*d) && aligned(E, 16) && aligned(Wq, 16) && (!dA || aligned(dA, 16)) && (!dAacc || aligned(dAacc, 16)))
        return tc::tc_pix(*d, 1, E, sE, Wq, sW, nullptr, 0, dA, dAacc, dev_status, as_stream(stream));
    return generic_bwd_data(*d, E, sE, Wq, sW, dA, dAacc, ws, as_stream(stream));
}

extern "C" lpdt_status lpdt_qconv_bwd_weight(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                             const int8_t *A, const float *sA, float *dW,
                                             int64_t dw_node_stride, int32_t *dWacc, void *ws,
                                             size_t ws_bytes, int32_t *dev_status, void *stream) {
    (void)dev_status;
    lpdt_status s = check_desc(d);
    if (s != LPDT_OK) return s;
    if (d->nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(E && A && (dW || dWacc));
    LPDT_CHECK_ARG(!dW || (sE && sA));
    LPDT_CHECK_ARG(!dW || dw_node_stride >= (int64_t)d->Cout * d->R * d->S * d->Cin || d->nodes == 1);
    if (!dWacc && (!ws || ws_bytes < lpdt_qconv_workspace_size(d, 2) || !aligned(ws, 4)))
        return LPDT_ERR_WORKSPACE;
    if (use_tc(*d) && d->B > 0 && aligned(E, 16) && aligned(A, 16)) {
        cudaStream_t st = as_stream(stream);
        const int64_t per_node = (int64_t)d->Cout * d->R * d->S * d->Cin;
        int32_t *acc = dWacc ? dWacc : (int32_t *)ws;
        LPDT_CUDA(cudaMemsetAsync(acc, 0, (size_t)d->nodes * per_node * sizeof(int32_t), st));
        lpdt_status r = tc::tc_wgrad(*d, E, A, acc, dev_status, st);
        if (r == LPDT_OK) {
            if (dW) return dequant_acc_launch(acc, d->nodes, per_node, sE, sA, dW, dw_node_stride, st);
            return LPDT_OK;
        }
        if (r != LPDT_ERR_UNSUPPORTED) return r;
    }
    return generic_bwd_weight(*d, E, sE, A, sA, dW, dw_node_stride, dWacc, ws, as_stream(stream));
}
