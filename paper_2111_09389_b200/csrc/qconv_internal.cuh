// Internal interface between the convolution front end (argument checks,
// kernel choice) and its back ends.  Not part of the ABI.
#pragma once
#include "common.cuh"

namespace lpdt {

static inline int conv_out(int H, int pad, int R, int stride) { return (H + 2 * pad - R) / stride + 1; }

lpdt_status generic_fwd(const lpdt_conv_desc &d, const int8_t *A, const float *sA, const int8_t *Wq,
                        const float *sW, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                        cudaStream_t st, bool uns = false);
lpdt_status generic_bwd_data(const lpdt_conv_desc &d, const int8_t *E, const float *sE, const int8_t *Wq,
                             const float *sW, float *dA, int32_t *dAacc, const float *addend, void *ws, cudaStream_t st,
                             bool uns = false);
lpdt_status generic_bwd_weight(const lpdt_conv_desc &d, const int8_t *E, const float *sE, const int8_t *A,
                               const float *sA, float *dW, int64_t dw_stride, int32_t *dWacc, void *ws,
                               cudaStream_t st, bool uns = false);

lpdt_status dequant_acc_launch(const int32_t *acc, int nodes, int64_t per_node, const float *s1,
                               const float *s2, float *out, int64_t out_stride, cudaStream_t st);

namespace tc {
// Tensor-core engine (tcgen05 kind::i8): stride-1 convolutions and GEMMs whose
// channel counts are multiples of 16.  mode 0 = forward, 1 = backward-data.
bool tc_supported(const lpdt_conv_desc &d);
// Zero-point correction applied in the forward epilogue (unsigned operands): per-pixel channel sums of the
// input [nodes][B][H][W], prefix table of the weights' channel sums over the filter taps
// [nodes][R+1][S+1][Cout], and the per-node zero points.
struct AffineArgs { const int32_t *asum, *wpre, *zA, *zW; };
lpdt_status tc_pix(const lpdt_conv_desc &d, int mode, const int8_t *A, const float *s1, const int8_t *Wq,
                   const float *s2, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                   int32_t *dev_status, cudaStream_t st, bool uns = false, const float *addend = nullptr,
                   const AffineArgs *aff = nullptr);
// Halo-tile kernel for 16-channel operands at stride 1 (one TMA request per tile).
bool halo_supported(const lpdt_conv_desc &d, int mode);
lpdt_status tc_pix_halo(const lpdt_conv_desc &d, int mode, const int8_t *A, const float *s1, const int8_t *Wq,
                        const float *s2, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                        int32_t *dev_status, cudaStream_t st, bool uns = false, const float *addend = nullptr);
lpdt_status tc_wgrad(const lpdt_conv_desc &d, int cin_real, const int8_t *E, const float *sE, const int8_t *A,
                     const float *sA, int32_t *acc_user, int32_t *acc_ws, float *dW, int64_t dw_stride,
                     int32_t *dev_status, cudaStream_t st, bool uns = false);
}  // namespace tc

}  // namespace lpdt
