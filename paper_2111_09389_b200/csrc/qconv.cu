// Front end of the quantized contractions: argument validation, workspace
// accounting and the choice between the tensor-core engine and the CUDA-core
// kernels.
#include "common.cuh"
#include "qconv_internal.cuh"

using namespace lpdt;

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
    return generic_bwd_weight(*d, E, sE, A, sA, dW, dw_node_stride, dWacc, ws, as_stream(stream));
}
