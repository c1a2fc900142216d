// Internal interface between the convolution front end (argument checks,
// kernel choice) and its back ends.  Not part of the ABI.
#pragma once
#include "common.cuh"

namespace lpdt {

static inline int conv_out(int H, int pad, int R, int stride) { return (H + 2 * pad - R) / stride + 1; }

lpdt_status generic_fwd(const lpdt_conv_desc &d, const int8_t *A, const float *sA, const int8_t *Wq,
                        const float *sW, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                        cudaStream_t st);
lpdt_status generic_bwd_data(const lpdt_conv_desc &d, const int8_t *E, const float *sE, const int8_t *Wq,
                             const float *sW, float *dA, int32_t *dAacc, void *ws, cudaStream_t st);
lpdt_status generic_bwd_weight(const lpdt_conv_desc &d, const int8_t *E, const float *sE, const int8_t *A,
                               const float *sA, float *dW, int64_t dw_stride, int32_t *dWacc, void *ws,
                               cudaStream_t st);

}  // namespace lpdt
