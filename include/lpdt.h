/*
 * lpdt.h — C ABI of the low-precision decentralized training step library
 * (8-bit training step of arXiv 2111.09389 on NVIDIA B200, sm_100a).
 *
 * Conventions (all entry points)
 *   - Every data pointer is a DEVICE pointer owned by the caller unless the
 *     argument is marked "host".  The library allocates no device memory;
 *     scratch comes from the caller's workspace `ws` (`ws_bytes` long, 256-byte
 *     aligned), whose required size the matching *_workspace_size call returns.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls only enqueue work; they never synchronise.  A workspace may be
 *     reused by the next call on the same stream.
 *   - The N simulated decentralized nodes are the leading dimension of every
 *     tensor; each node has its own values and its own quantization scale.
 *       activations  NHWC  [nodes][B][H][W][C]
 *       weights      KRSC  [nodes][Cout][R][S][Cin]
 *       parameters   flat  [nodes][d]; a tensor that lives inside the flat
 *                    parameter (or gradient) vector is addressed by a base
 *                    pointer plus a `*_node_stride` in elements.
 *   - Return value: LPDT_OK or an error code.  Argument errors are detected on
 *     the host before anything is enqueued.  Kernels never trap or spin
 *     without bound: a device-side wait that runs out writes a non-zero code
 *     into `dev_status` (one int32, caller-zeroed, nullable) and the kernel
 *     returns.
 *   - Integer accumulators are int32 and wrap modulo 2^32 like the hardware.
 *   - Floating point: element-wise arithmetic is a fixed sequence of
 *     individually rounded fp32 operations (no contraction, no fast math).
 *     Reductions that decide later integer codes (ranges, the Range-EvoNorm
 *     group sum) are exact or accumulated in fp64; the per-channel parameter
 *     gradient sums add fp32 runs of at most 16 terms into fp64 accumulators.
 *     Everything is rounded to fp32 once.
 */
#ifndef LPDT_H
#define LPDT_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t lpdt_status;
enum {
    LPDT_OK = 0,
    LPDT_ERR_INVALID_ARG = 1,   /* null pointer, bad size, misalignment */
    LPDT_ERR_UNSUPPORTED = 2,   /* valid request this build has no kernel for */
    LPDT_ERR_WORKSPACE = 3,     /* workspace missing or too small */
    LPDT_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed */
    LPDT_ERR_TIMEOUT = 5,       /* a bounded device-side wait expired */
    LPDT_ERR_OVERFLOW = 6
};

typedef enum { LPDT_SYM_S8 = 0, LPDT_AFFINE_U8 = 1 } lpdt_qmode;
typedef enum { LPDT_ROUND_NEAREST_EVEN = 0, LPDT_ROUND_STOCHASTIC = 1 } lpdt_round;

/* Convolution geometry.  Ho = (H + 2*pad - R)/stride + 1, likewise Wo.
 * A linear layer is R = S = H = W = 1, stride 1, pad 0 (B rows, Cin -> Cout). */
typedef struct {
    int32_t nodes, B, H, W, Cin, Cout, R, S, stride, pad;
} lpdt_conv_desc;

const char *lpdt_version(void);
const char *lpdt_status_string(lpdt_status s);
/* Name of the contraction kernel that the most recent lpdt_qconv_* call of the calling host thread
 * launched ("" before the first one): the tensor-core pixel-tile, halo-tile or weight-gradient kernel, or
 * a CUDA-core kernel.  For labelling timings; the choice depends on the shape, the alignment and on which
 * outputs were asked for. */
const char *lpdt_last_kernel(void);
/* Number of kernels the calling host thread has enqueued through this library so far (memsets and
 * copies not counted; a launch recorded during stream capture counts once, its replays do not). */
uint64_t lpdt_launch_count(void);
/* Enqueue a zero fill of `bytes` bytes at device pointer p (range accumulators, status words). */
lpdt_status lpdt_fill_zero(void *p, size_t bytes, void *stream);
/* Read a status word back: waits until everything enqueued on `stream` so far has finished (the one
 * call of this library that synchronises), then returns the value of *dev_status: LPDT_OK, or the
 * code a kernel recorded there (LPDT_ERR_TIMEOUT from a bounded wait that ran out,
 * LPDT_ERR_INVALID_ARG from an out-of-range label).  LPDT_ERR_CUDA if the copy or the wait fails.
 * The word is not cleared. */
lpdt_status lpdt_check_status(const int32_t *dev_status, void *stream);
/* Diagnostics (no counterpart in the paper): runs the bounded barrier wait of the tensor-core
 * kernels on a barrier that nothing arrives at, with a limit of limit_ns nanoseconds (1 us to
 * 50 ms; INVALID_ARG outside).  The one-CTA kernel returns once the limit has passed, writes
 * LPDT_ERR_TIMEOUT to *dev_status and 2 to *returned (nullable; 1 would mean the wait succeeded).
 * The production kernels use the same routine with a limit of two seconds. */
lpdt_status lpdt_selftest_bounded_wait(uint64_t limit_ns, int32_t *dev_status, int32_t *returned, void *stream);

/* ---------------------------------------------------------------------------
 * lpdt_quantize — per-tensor, per-node 8-bit quantization.
 * Paper: Section 3, "Low Precision Training" (weights, activations and layer
 * gradients are quantized to 8 bits in every iteration; the scheme is named by
 * citation only, the formulas below are this library's reading).
 *
 *   LPDT_SYM_S8 :  amax = max|x|; scale = amax/127; inv = 127/amax
 *       nearest-even : q = clamp(rne(x*inv), -127, 127)
 *       stochastic   : t = x*inv; q = floor(t) + [u < t - floor(t)], with u the
 *                      24-bit uniform from word (i mod 4) of Philox4x32-10 at
 *                      counter (i/4 low, i/4 high, node, ctr_offset), key = seed
 *       amax == 0 gives scale = 1 and q = 0.
 *   LPDT_AFFINE_U8 (nearest-even only): lo = min(0,min x), hi = max(0,max x),
 *       scale = (hi-lo)/255 (1 if hi == lo), zp = clamp(rne(-lo/scale),0,255),
 *       q = clamp(rne(x/scale) + zp, 0, 255), stored in the same byte array.
 *
 * x     : fp32, node n starts at x + n*x_node_stride, n_per_node elements each
 * q     : 8-bit codes, contiguous [nodes][n_per_node]
 * scale : fp32 [nodes];  zero_point : int32 [nodes], required for AFFINE_U8 only
 * ws    : lpdt_quantize_workspace_size(nodes) bytes
 * Errors: INVALID_ARG (null/negative/misaligned), WORKSPACE, CUDA.
 * n_per_node == 0 or nodes == 0 is a no-op returning LPDT_OK.
 */
size_t lpdt_quantize_workspace_size(int32_t nodes);
lpdt_status lpdt_quantize(const float *x, int32_t nodes, int64_t n_per_node, int64_t x_node_stride,
                          lpdt_qmode mode, lpdt_round rounding, uint64_t seed, uint32_t ctr_offset,
                          int8_t *q, float *scale, int32_t *zero_point,
                          void *ws, size_t ws_bytes, void *stream);

/* Symmetric quantization when the per-node range is already known: only the
 * scale-and-round pass of lpdt_quantize (LPDT_SYM_S8) runs.  amax : fp32 [nodes],
 * max|x| of each node's tensor, as the producers below can emit while they write
 * x (lpdt_range_evonorm_fwd/bwd, lpdt_residual_add: `amax_out`).  Same codes and
 * scales as lpdt_quantize, bit for bit, because a maximum does not depend on the
 * order it is taken in.  No workspace. */
lpdt_status lpdt_quantize_with_range(const float *x, int32_t nodes, int64_t n_per_node, int64_t x_node_stride,
                                     const float *amax, lpdt_round rounding, uint64_t seed,
                                     uint32_t ctr_offset, int8_t *q, float *scale, void *stream);

/* lpdt_quantize_batch - symmetric nearest-even quantization (as lpdt_quantize, LPDT_SYM_S8) of
 * n_tensors tensors that sit inside one flat per-node parameter vector, e.g. all layer
 * weights of a network, in two launches.  Tensor t of node n is read from
 * params + n*row_stride + src_offsets[t] (sizes[t] elements) and written as int8 to
 * q + dst_offsets[t] + n*sizes[t]  (each tensor contiguous [nodes][sizes[t]], as the
 * contractions expect); scales[t*nodes + n] receives its scale.  src_offsets, sizes and
 * dst_offsets are HOST arrays; n_tensors <= 64 (LPDT_ERR_UNSUPPORTED beyond).
 * ws : lpdt_quantize_batch_workspace_size(nodes, n_tensors) bytes. */
size_t lpdt_quantize_batch_workspace_size(int32_t nodes, int32_t n_tensors);
lpdt_status lpdt_quantize_batch(const float *params, int32_t nodes, int64_t row_stride, int32_t n_tensors,
                                const int64_t *src_offsets, const int64_t *sizes, const int64_t *dst_offsets,
                                int8_t *q, float *scales, void *ws, size_t ws_bytes, void *stream);

/* y = scale[n] * (q - zp[n]); zero_point == NULL means symmetric signed codes.
 * q is contiguous [nodes][n_per_node]; node n of y starts at y + n*y_node_stride. */
lpdt_status lpdt_dequantize(const int8_t *q, int32_t nodes, int64_t n_per_node,
                            const float *scale, const int32_t *zero_point,
                            float *y, int64_t y_node_stride, void *stream);

/* ---------------------------------------------------------------------------
 * lpdt_quantize_static - lpdt_quantize without a caller workspace.
 * (The paper has no counterpart: this entry point exists for integration only.)
 *
 * For callers that cannot hand the library any device scratch: a training loop
 * on a device whose buffers were all fixed at start-up, or code called from a
 * host application that owns the device memory pool and does not allow device
 * allocation where this call sits.  The per-node range words live in an 8 KB
 * array inside the library image instead (held by every GPU that loads the
 * library, until the process exits).  The call allocates nothing.
 *
 * Arguments, results and rounding are those of lpdt_quantize; ws/ws_bytes are
 * gone.  Limits and rules:
 *   - nodes <= LPDT_QUANTIZE_STATIC_MAX_NODES, otherwise LPDT_ERR_WORKSPACE
 *     (the built-in scratch is too small) and nothing is enqueued.
 *   - The first call on each device that has work to do (nodes > 0 and
 *     n_per_node > 0) looks up the array's device address; make that first call
 *     before any stream capture.  The device that owns `stream` must be the
 *     current device, as for every call of this library.  The looked-up address
 *     is cached per device ordinal and does not survive a cudaDeviceReset in
 *     the same process.
 *   - All calls share the one array, so two calls whose kernels may overlap on
 *     the GPU (different streams, no ordering between them) race; calls on one
 *     stream, or otherwise ordered, are safe.  The words a call uses are cleared
 *     at its start; it does not depend on what the previous call left behind.
 */
#define LPDT_QUANTIZE_STATIC_MAX_NODES 1024
lpdt_status lpdt_quantize_static(const float *x, int32_t nodes, int64_t n_per_node, int64_t x_node_stride,
                                 lpdt_qmode mode, lpdt_round rounding, uint64_t seed, uint32_t ctr_offset,
                                 int8_t *q, float *scale, int32_t *zero_point, void *stream);

/* ---------------------------------------------------------------------------
 * Quantized contractions on symmetric int8 operands (Section 3: the forward
 * product and both backward products run on 8-bit operands; the operation
 * count table's Conv and Linear rows count the three alike).  int32
 * accumulation; the fp32 result is (float)acc * (s1[n]*s2[n]) (+ bias).
 *
 * fwd        acc[n,b,oh,ow,co] = sum_{r,s,ci} A[n,b,oh*st+r-p,ow*st+s-p,ci] * W[n,co,r,s,ci]
 * bwd_data   dA[n,b,ih,iw,ci]  = sum_{r,s,co} E[n,b,oh,ow,co] * W[n,co,r,s,ci]
 *                                over (oh,ow) with ih = oh*st+r-p, iw = ow*st+s-p
 * bwd_weight dW[n,co,r,s,ci]   = sum_{b,oh,ow} E[n,b,oh,ow,co] * A[n,b,oh*st+r-p,ow*st+s-p,ci]
 * Taps that fall outside the image read zero.
 *
 * A, E, Wq : int8, contiguous in the layouts above;  sA, sE, sW : fp32 [nodes]
 * Y/dA/dW  : fp32 output (nullable);  Yacc/dAacc/dWacc : raw int32 accumulators
 *            (nullable; same shape, contiguous).  At least one must be given.
 * bias     : fp32, node n at bias + n*bias_node_stride, Cout entries (nullable)
 * dW       : node n at dW + n*dw_node_stride (weight gradients stay fp32:
 *            "gradient bifurcation"); dWacc is contiguous.
 * addend   : (bwd_data, nullable) fp32, shape of dA, 16-byte aligned, not dA itself: dA = dequantized
 *            sums + addend, one more fp32 addition.  This is the adjoint of a residual block's identity
 *            shortcut (the block-output gradient joins the gradient of the block's first convolution),
 *            fused into the contraction's epilogue; dAacc is not affected.
 * ws       : lpdt_qconv_workspace_size(desc, which) bytes, which = 0 fwd,
 *            1 bwd_data, 2 bwd_weight.
 * Errors: INVALID_ARG, UNSUPPORTED (shape outside every kernel's range),
 *         WORKSPACE, CUDA; TIMEOUT is reported through dev_status.
 */
size_t lpdt_qconv_workspace_size(const lpdt_conv_desc *d, int32_t which);
lpdt_status lpdt_qconv_fwd(const lpdt_conv_desc *d, const int8_t *A, const float *sA,
                           const int8_t *Wq, const float *sW,
                           const float *bias, int64_t bias_node_stride,
                           float *Y, int32_t *Yacc,
                           void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);
lpdt_status lpdt_qconv_bwd_data(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                const int8_t *Wq, const float *sW,
                                float *dA, int32_t *dAacc, const float *addend,
                                void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);
lpdt_status lpdt_qconv_bwd_weight(const lpdt_conv_desc *d, const int8_t *E, const float *sE,
                                  const int8_t *A, const float *sA,
                                  float *dW, int64_t dw_node_stride, int32_t *dWacc,
                                  void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);

/* Dequantize the raw int32 sums of up to 64 tensors in one launch (all weight gradients of a network, each
 * left by lpdt_qconv_bwd_weight through dWacc as a contiguous [nodes][sizes[t]] block at acc + acc_offsets[t]):
 *   out[n*out_node_stride + out_offsets[t] + i] = (float)acc[acc_offsets[t] + n*sizes[t] + i] * (s1[t][n]*s2[t][n])
 * for i < sizes[t]: the fp32 result of lpdt_qconv_bwd_weight, bit for bit.  acc_offsets, sizes and out_offsets
 * are HOST arrays (elements); s1 and s2 are HOST arrays of device pointers to the per-node scales of each
 * tensor's two operands.  Errors: INVALID_ARG, UNSUPPORTED (more than 64 tensors), CUDA. */
lpdt_status lpdt_dequantize_acc_batch(const int32_t *acc, int32_t nodes, int32_t n_tensors,
                                      const int64_t *acc_offsets, const int64_t *sizes, const int64_t *out_offsets,
                                      const float *const *s1, const float *const *s2,
                                      float *out, int64_t out_node_stride, void *stream);

/* ---------------------------------------------------------------------------
 * Forward contraction on affine (zero-point) operands: the quantization scheme
 * Section 3 names maps a real tensor to unsigned 8-bit codes with a scale and a
 * zero point, real = scale*(code - zero_point) (lpdt_quantize, LPDT_AFFINE_U8).
 * The convolution pads with real zeros, so taps outside the image add nothing:
 *
 *   acc[n,b,oh,ow,co] = sum_{(r,s) inside the image, ci}
 *                       (A[n,b,oh*st+r-p,ow*st+s-p,ci] - zA[n]) * (W[n,co,r,s,ci] - zW[n])
 *   Y = (float)acc * (sA[n]*sW[n]) (+ bias)
 *
 * A, Wq   : uint8 codes in the layouts of lpdt_qconv_fwd;  zA, zW : int32 [nodes],
 *           each in [0, 255];  sA, sW : fp32 [nodes] (needed only for Y)
 * Y, Yacc : as in lpdt_qconv_fwd (at least one); int32 results wrap modulo 2^32
 * ws      : lpdt_qconv_fwd_affine_workspace_size(desc) bytes, 256-byte aligned
 * The integer contraction of the codes runs on the same kernels as
 * lpdt_qconv_fwd (unsigned operand format); the zero-point terms are applied
 * in the tensor-core kernel's epilogue (forward product) or by a correction
 * pass over the int32 sums (shapes outside the tensor-core path, and both
 * backward products).
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA; TIMEOUT through dev_status.
 *
 * The two backward products in the same form (the adjoints of the forward product: a tap
 * outside the image is absent from the sums), with E the layer gradient as unsigned codes
 * with zero point zE and scale sE:
 *   dA[n,b,ih,iw,ci] = sum_{(oh,ow,r,s) with ih = oh*st+r-p, iw = ow*st+s-p; co}
 *                      (E[n,b,oh,ow,co] - zE[n]) * (W[n,co,r,s,ci] - zW[n])
 *   dW[n,co,r,s,ci]  = sum_{(b,oh,ow) with the tap (r,s) inside the image}
 *                      (E[n,b,oh,ow,co] - zE[n]) * (A[n,b,oh*st+r-p,ow*st+s-p,ci] - zA[n])
 *   fp32 results: (float)sum * (sE[n]*sW[n]) and (float)sum * (sE[n]*sA[n]).
 * Layouts, nullable outputs and dw_node_stride as in lpdt_qconv_bwd_data / _bwd_weight;
 * ws: the matching *_affine_workspace_size(desc) bytes, 256-byte aligned.
 */
size_t lpdt_qconv_fwd_affine_workspace_size(const lpdt_conv_desc *d);
lpdt_status lpdt_qconv_fwd_affine(const lpdt_conv_desc *d, const uint8_t *A, const float *sA, const int32_t *zA,
                                  const uint8_t *Wq, const float *sW, const int32_t *zW,
                                  const float *bias, int64_t bias_node_stride,
                                  float *Y, int32_t *Yacc,
                                  void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);
size_t lpdt_qconv_bwd_data_affine_workspace_size(const lpdt_conv_desc *d);
lpdt_status lpdt_qconv_bwd_data_affine(const lpdt_conv_desc *d, const uint8_t *E, const float *sE, const int32_t *zE,
                                       const uint8_t *Wq, const float *sW, const int32_t *zW,
                                       float *dA, int32_t *dAacc,
                                       void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);
size_t lpdt_qconv_bwd_weight_affine_workspace_size(const lpdt_conv_desc *d);
lpdt_status lpdt_qconv_bwd_weight_affine(const lpdt_conv_desc *d, const uint8_t *E, const float *sE, const int32_t *zE,
                                         const uint8_t *A, const float *sA, const int32_t *zA,
                                         float *dW, int64_t dw_node_stride, int32_t *dWacc,
                                         void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------
 * Range-EvoNorm (Eq. "ren"), forward and backward.
 * For node n, sample b, group G of cpg = C/groups consecutive channels:
 *   mx, mn = max/min of x over (h, w, c in G);  D = Cst*(mx-mn) + eps,
 *   Cst = 1/sqrt(2 ln cpg);  u = v_c*x;  hs = clamp((u+3)/6, 0, 1);  m = x*hs;
 *   y = (gamma_c*m)*(1/D) + beta_c
 * Backward (t = dy*gamma_c, hp = 1/6 on -3<u<3 else 0, S = sum_G t*m):
 *   dx = (t*(hs + u*hp))*(1/D), then dx[argmax] -= Cst*S/D^2, dx[argmin] += Cst*S/D^2
 *   (skipped when argmax == argmin);  dbeta_c = sum dy;  dgamma_c = sum dy*(m/D);
 *   dv_c = sum t*x*x*hp/D, sums over the node's (b,h,w).
 * argmax/argmin: lowest (h*W+w)*C+c index attaining the extremum.
 *
 * x, y, dy, dx : fp32 NHWC;  v, gamma, beta : fp32, node n at p + n*param_node_stride
 * gmin, gmax : fp32 [nodes][B][groups];  argmin, argmax : int32, same shape
 * dv, dgamma, dbeta : fp32, node n at p + n*grad_node_stride, C entries
 * res (forward, nullable) : fp32, shape of y; when given the identity shortcut of a residual
 *            block is fused: y = RangeEvoNorm(x) + res (the sum is one more fp32 addition)
 * amax_out (nullable) : fp32 [nodes], caller-zeroed; receives max|y| (forward) or max|dx|
 *            (backward) per node by atomic maximum, for lpdt_quantize_with_range
 * Requires C % groups == 0 and cpg >= 2 (Cst is infinite for cpg = 1).
 * Backward with dv = dgamma = dbeta = NULL writes dx only and leaves the parameter-gradient sums as
 * per-sample partial sums in ws; lpdt_range_evonorm_bwd_params(nodes, B, C, ws, ...) then adds them over
 * the batch (fixed order, same result as the one-call form).  The second call may run on another
 * stream once the first has finished, which takes the small reduction off the backward pass's critical
 * path; ws must not be reused in between.
 * Errors: INVALID_ARG, UNSUPPORTED (C beyond the kernels' range), WORKSPACE, CUDA.
 */
lpdt_status lpdt_range_evonorm_fwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                   int32_t groups, float eps, const float *x,
                                   const float *v, const float *gamma, const float *beta,
                                   int64_t param_node_stride, float *y,
                                   float *gmin, float *gmax, int32_t *argmin, int32_t *argmax,
                                   float *amax_out, const float *res, void *stream);
size_t lpdt_range_evonorm_bwd_workspace_size(int32_t nodes, int32_t B, int32_t C);
lpdt_status lpdt_range_evonorm_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                   int32_t groups, float eps, const float *dy, const float *x,
                                   const float *v, const float *gamma, int64_t param_node_stride,
                                   const float *gmin, const float *gmax,
                                   const int32_t *argmin, const int32_t *argmax,
                                   float *dx, float *dv, float *dgamma, float *dbeta,
                                   int64_t grad_node_stride, float *amax_out,
                                   void *ws, size_t ws_bytes, void *stream);
lpdt_status lpdt_range_evonorm_bwd_params(int32_t nodes, int32_t B, int32_t C, const void *ws, size_t ws_bytes,
                                          float *dv, float *dgamma, float *dbeta, int64_t grad_node_stride,
                                          void *stream);
/* The second call for up to 64 layers in one launch (a network's norm layers at the end of its backward
 * pass).  Layer l has C[l] channels, its partial sums in ws[l] (as left by lpdt_range_evonorm_bwd with null
 * gradient pointers; same nodes and B for all layers), and its three gradient vectors back to back - dv,
 * dgamma, dbeta, C[l] entries each - at grads + n*grad_node_stride + grad_offsets[l].  C, ws and
 * grad_offsets are HOST arrays (ws holds device pointers).  Same sums, same order, same results as
 * n_layers single calls.  Errors: INVALID_ARG, UNSUPPORTED (more than 64 layers), CUDA. */
lpdt_status lpdt_range_evonorm_bwd_params_batch(int32_t nodes, int32_t B, int32_t n_layers, const int32_t *C,
                                                const void *const *ws, const int64_t *grad_offsets,
                                                float *grads, int64_t grad_node_stride, void *stream);

/* Range-EvoNorm with the requantize step inside (Section 3, "Low Precision Training": activations and layer
 * gradients travel between layers as 8-bit tensors).  lpdt_range_evonorm_fwd_q8 computes y as
 * lpdt_range_evonorm_fwd does and ALSO writes y's symmetric 8-bit codes q (int8, shape of y) and per-node scale
 * (fp32 [nodes]): exactly what lpdt_quantize_with_range(y, max|y|, LPDT_ROUND_NEAREST_EVEN) would write.  y may
 * be NULL when only the codes are wanted.  lpdt_range_evonorm_bwd_q8 computes dx as lpdt_range_evonorm_bwd does
 * but writes only its codes q and scale; the parameter gradients (or, with the three pointers NULL, the partial
 * sums in ws) are those of lpdt_range_evonorm_bwd.  amax_out (nullable, fp32 [nodes]) is overwritten with
 * max|y| / max|dx| (no caller zeroing here).
 * One CTA per sample keeps the sample's fp32 result in shared memory until the node-wide range is known; the
 * CTAs of a node meet through the control block ctl (device memory, lpdt_range_evonorm_q8_ctl_size(nodes)
 * bytes, 4-byte aligned): ZERO it once before the first call; every call that completes leaves it zero again,
 * so consecutive calls may share it, concurrent calls may not.  The meeting is a bounded wait: if it ever ran
 * out, dev_status (nullable device int32) would receive LPDT_ERR_TIMEOUT, the codes of the affected nodes
 * would be left unwritten and ctl would have to be zeroed again.
 * lpdt_range_evonorm_fwd_q8_fits / _bwd_q8_fits return 1 when the shape is served: a sample (H*W*C fp32) fits
 * one CTA's shared memory beside the kernel's scratch, C/groups is a multiple of 4, and the device has room for
 * 2*B resident CTAs; otherwise the call returns UNSUPPORTED and the two-call form (lpdt_range_evonorm_*
 * followed by lpdt_quantize_with_range) serves.  x, dy, res, y 16-byte aligned, q 4-byte aligned.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE (ws or ctl missing or too small), CUDA. */
size_t lpdt_range_evonorm_q8_ctl_size(int32_t nodes);
int32_t lpdt_range_evonorm_fwd_q8_fits(int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups);
lpdt_status lpdt_range_evonorm_fwd_q8(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                      int32_t groups, float eps, const float *x,
                                      const float *v, const float *gamma, const float *beta,
                                      int64_t param_node_stride, float *y,
                                      float *gmin, float *gmax, int32_t *argmin, int32_t *argmax,
                                      float *amax_out, const float *res, int8_t *q, float *scale,
                                      void *ctl, size_t ctl_bytes, int32_t *dev_status, void *stream);
int32_t lpdt_range_evonorm_bwd_q8_fits(int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups);
lpdt_status lpdt_range_evonorm_bwd_q8(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                      int32_t groups, float eps, const float *dy, const float *x,
                                      const float *v, const float *gamma, int64_t param_node_stride,
                                      const float *gmin, const float *gmax,
                                      const int32_t *argmin, const int32_t *argmax,
                                      int8_t *q, float *scale, float *dv, float *dgamma, float *dbeta,
                                      int64_t grad_node_stride, float *amax_out,
                                      void *ws, size_t ws_bytes, void *ctl, size_t ctl_bytes,
                                      int32_t *dev_status, void *stream);

/* ---------------------------------------------------------------------------
 * Comparison layers of Section 3 (the normalization study; not on the 8-bit path).
 *
 * lpdt_evonorm_s0_fwd / _bwd — EvoNorm-S0 (Eq. "en"), the layer the paper trains with at full
 * precision.  Per node, sample and group of cpg = C/groups consecutive channels:
 *   mu, var = mean and divide-by-count variance of x over the group's (h, w, c)
 *   D = sqrt(var + eps);   y = gamma_c * (x * sigmoid(v_c*x)) / D + beta_c
 * (the equation has no eps: eps = 0 reproduces it).  Backward, derived, with t = dy*gamma_c,
 * sig = sigmoid(v_c*x), m = x*sig, cnt = H*W*cpg and S = sum over the group of t*m:
 *   dx = t*(sig + v_c*x*sig*(1 - sig))/D - S*(x - mu)/(cnt*D^3)
 *   dbeta_c = sum dy;  dgamma_c = sum dy*m/D;  dv_c = sum t*x*x*sig*(1 - sig)/D   (over b, h, w)
 * Layouts as lpdt_range_evonorm_*: x, y, dy, dx fp32 NHWC; parameters per node at p + n*param_node_stride;
 * gmean, gvar : fp32 [nodes][B][groups], written by the forward, read by the backward.
 * Statistics and parameter-gradient sums are accumulated in double; elementwise work is fp32.
 * Errors: INVALID_ARG, UNSUPPORTED (more than 256 channel vectors), WORKSPACE, CUDA.
 */
lpdt_status lpdt_evonorm_s0_fwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups,
                                float eps, const float *x, const float *v, const float *gamma, const float *beta,
                                int64_t param_node_stride, float *y, float *gmean, float *gvar, void *stream);
size_t lpdt_evonorm_s0_bwd_workspace_size(int32_t nodes, int32_t B, int32_t C);
lpdt_status lpdt_evonorm_s0_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups,
                                float eps, const float *dy, const float *x, const float *v, const float *gamma,
                                int64_t param_node_stride, const float *gmean, const float *gvar,
                                float *dx, float *dv, float *dgamma, float *dbeta, int64_t grad_node_stride,
                                void *ws, size_t ws_bytes, void *stream);

/* lpdt_range_bn_fwd / _bwd — range batch-norm (Eq. "rbn").  Per node and channel over the node's
 * batch (b, h, w), P = B*H*W positions:
 *   mu = mean of x;  D = Cb*(max x - min x) + eps,  Cb = 1/sqrt(2 ln B)   (the equation's C(b), b = the
 *   batch size; B >= 2);   y = gamma_c*(x - mu)/D + beta_c
 * Backward, derived, with t = dy*gamma_c and xc = x - mu:
 *   dx = t/D - (sum t)/(P*D) - Cb*(sum t*xc)/D^2 * ([p = argmax] - [p = argmin])   (no last term if they coincide)
 *   dbeta_c = sum dy;  dgamma_c = sum dy*xc/D
 * cmean, cmin, cmax : fp32 [nodes][C];  argmin, argmax : int32 [nodes][C], the lowest position b*H*W + h*W + w
 * attaining the extremum; all five written by the forward and read by the backward.
 * ws : lpdt_range_bn_workspace_size(nodes, C) bytes (cross-CTA sums and extrema; cleared by the call).
 * Errors: INVALID_ARG (B < 2 included), UNSUPPORTED, WORKSPACE, CUDA.
 */
size_t lpdt_range_bn_workspace_size(int32_t nodes, int32_t C);
lpdt_status lpdt_range_bn_fwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, float eps,
                              const float *x, const float *gamma, const float *beta, int64_t param_node_stride,
                              float *y, float *cmean, float *cmin, float *cmax, int32_t *argmin, int32_t *argmax,
                              void *ws, size_t ws_bytes, void *stream);
lpdt_status lpdt_range_bn_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, float eps,
                              const float *dy, const float *x, const float *gamma, int64_t param_node_stride,
                              const float *cmean, const float *cmin, const float *cmax,
                              const int32_t *argmin, const int32_t *argmax,
                              float *dx, float *dgamma, float *dbeta, int64_t grad_node_stride,
                              void *ws, size_t ws_bytes, void *stream);

/* ---------------------------------------------------------------------------
 * lpdt_gossip_mix — compression, public-copy update and gossip averaging of
 * CHOCO-SGD (Algorithm 3: "compute and compress", the x_hat update, and the
 * gossip update), for all nodes at once:
 *   delta_i = x_half_i - x_hat_i
 *   q_i     = delta_i on the seg_k[s] largest |delta_i| of every segment s
 *             (equal magnitudes: lower index kept), 0 elsewhere;
 *             seg_k[s] >= segment length means no compression
 *   x_hat_i <- x_hat_i + q_i
 *   x_out_i = x_half_i + gamma * sum_j Wmix[i][j] * (x_hat_j - x_hat_i)   (updated x_hat)
 * x_half, x_hat (in/out), x_out : fp32 [nodes][d];  x_out may alias x_half.
 * Wmix : fp32 [nodes][nodes] row-major, row i = the weights node i applies.
 * seg_offsets (n_segments+1 entries) and seg_k (n_segments) are HOST arrays;
 * segments must tile [0,d).  n_segments = 1 is the flattened vector.
 * Errors: INVALID_ARG, UNSUPPORTED (nodes > 64), WORKSPACE, CUDA.
 */
size_t lpdt_gossip_mix_workspace_size(int32_t nodes, int64_t d, int32_t n_segments);
lpdt_status lpdt_gossip_mix(int32_t nodes, int64_t d, const float *x_half, float *x_hat,
                            float *x_out, const float *Wmix, float gamma,
                            int32_t n_segments, const int64_t *seg_offsets, const int64_t *seg_k,
                            void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);

/* The same step with 8-bit messages (the quantized exchange behind the factor of four
 * in the Data column of the CIFAR table; the paper prints no formula, this is the reading
 * taken): the compressed difference of each (node, segment) is sent as signed 8-bit codes
 * with one range, by the symmetric quantizer of lpdt_quantize:
 *   amax = max |x_half - x_hat| over the segment (0 if seg_k = 0),
 *   scale = amax/127, inv = 127/amax (both 1 if amax = 0),
 *   message_e = (float)clamp(rne((x_half_e - x_hat_e) * inv), -127, 127) * scale on the kept entries,
 * and x_hat absorbs the dequantized message, so the rounding error stays in the next
 * difference.  msg_scale : fp32 [nodes][n_segments], out (the step each node transmits).
 * A node's message is k codes (+ k indices when k < segment length) + one scale.
 * Everything else as lpdt_gossip_mix (same workspace size). */
lpdt_status lpdt_gossip_mix_q8(int32_t nodes, int64_t d, const float *x_half, float *x_hat, float *x_out,
                               const float *Wmix, float gamma, int32_t n_segments,
                               const int64_t *seg_offsets, const int64_t *seg_k, float *msg_scale,
                               void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);

/* Bytes one node hands to EACH neighbour in one gossip step (host arithmetic, no device work), the
 * quantity behind the Data column of the paper's CIFAR table (data sent per node over a run =
 * this x iterations; the table's full-precision rows are 32-bit values, its low-precision rows
 * exactly a quarter of them):
 *   sum over segments of  k_s*value_bits + (k_s < len_s ? k_s*index_bits : 0) + (value_bits == 8 && k_s > 0 ? 32 : 0)
 * bits, rounded up to bytes, with k_s = min(seg_k[s], len_s): kept values, their positions inside
 * the segment when the segment is compressed, and the fp32 step of a segment sent as 8-bit codes.
 * seg_offsets / seg_k : HOST arrays as in lpdt_gossip_mix;  value_bits 32, 16 or 8;  index_bits 0..64
 * (0 = count values only).  Returns -1 for invalid arguments. */
int64_t lpdt_message_bytes(int64_t d, int32_t n_segments, const int64_t *seg_offsets, const int64_t *seg_k,
                           int32_t value_bits, int32_t index_bits);

/* Deep-Squeeze gossip step (supplementary Algorithm 2, steps 5-10) for all nodes:
 *   v_i = x_half_i + delta_i;  c_i = C[v_i];  delta_i <- v_i - c_i;
 *   x_i = x_half_i + eta * (sum_j W_ij c_j - c_i)
 * C keeps, per segment, the seg_k entries of largest |v| (ties: lower index); with
 * message_bits = 8 the kept entries are sent as 8-bit codes (one range per node and
 * segment, as in lpdt_gossip_mix_q8) and delta keeps the rounding error too.
 * delta     : fp32 [nodes][d], in/out (the error buffer; zeros at the start of training)
 * message_bits : 32 or 8;  msg_scale : fp32 [nodes][n_segments], out, required for 8 bits
 * Everything else, the workspace size included, as lpdt_gossip_mix. */
lpdt_status lpdt_deepsqueeze_mix(int32_t nodes, int64_t d, const float *x_half, float *delta, float *x_out,
                                 const float *Wmix, float eta, int32_t n_segments,
                                 const int64_t *seg_offsets, const int64_t *seg_k,
                                 int32_t message_bits, float *msg_scale,
                                 void *ws, size_t ws_bytes, int32_t *dev_status, void *stream);

/* The SGD half-step and the UNCOMPRESSED gossip step in one launch (Algorithm 1 "update the model", then
 * Algorithm 3 with every entry of the difference kept):
 *   x_half_i = x_i - lr*g_i;  x_hat_i <- x_hat_i + (x_half_i - x_hat_i);
 *   x_out_i  = x_half_i + gamma * sum_j Wmix[i][j] * (x_hat_j - x_hat_i)
 * the same fp32 operations in the same order as lpdt_sgd_update followed by lpdt_gossip_mix with
 * seg_k >= segment length, without the separate update pass over the parameters.
 * x, g : fp32 [nodes][d] (parameters, gradients);  x_half (out), x_hat (in/out), x_out (out) : fp32 [nodes][d];
 * the five arrays are distinct.  No workspace.  Errors: INVALID_ARG, UNSUPPORTED (nodes > 64), CUDA.
 */
lpdt_status lpdt_sgd_gossip_mix(int32_t nodes, int64_t d, const float *x, const float *g, float lr,
                                float *x_half, float *x_hat, float *x_out, const float *Wmix, float gamma,
                                void *stream);

/* Push-sum bias weights and de-biasing (supplementary Algorithms 4 and 5, Sparse-Push and
 * Quant-SGP: second line of the gossip update, then the de-biasing step), for column-stochastic
 * mixing matrices on directed graphs:
 *   u_new_i = u_i + eta * (sum_j Wmix[i][j]*u_j - u_i)     (j ascending, each step rounded to fp32)
 *   z_i     = x_i / u_new_i                                 (the model the next gradient is taken at)
 * x is the mixed model of the same step: x_out of lpdt_deepsqueeze_mix (Sparse-Push) or of
 * lpdt_gossip_mix / lpdt_gossip_mix_q8 (Quant-SGP) called with the same Wmix and eta.
 * x, z : fp32 [nodes][d] (z may alias x);  u, u_new : fp32 [nodes], distinct arrays (u starts at 1);
 * Wmix : fp32 [nodes][nodes] row-major, row i = the weights node i applies to what it receives.
 * d = 0 updates the bias weights alone.  Errors: INVALID_ARG, UNSUPPORTED (nodes > 64), CUDA.
 */
lpdt_status lpdt_pushsum_debias(int32_t nodes, int64_t d, const float *x, const float *u, const float *Wmix,
                                float eta, float *u_new, float *z, void *stream);

/* ---------------------------------------------------------------------------
 * Glue around the layers of one training step.
 */

/* Local SGD update (Algorithm 1, "update the model"): out = x - lr*g on the
 * fp32 master weights.  out may alias x. */
lpdt_status lpdt_sgd_update(int64_t n, const float *x, const float *g, float lr, float *out,
                            void *stream);

/* Residual connection y = r + P(a): P subsamples a [nodes*B][H][W][Ca]
 * spatially by `stride` and places its channels at ch_off within C channels
 * (identity shortcut: stride 1, Ca = C, ch_off 0).  y may alias r.  amax_out (nullable,
 * fp32 [nodes], caller-zeroed) receives max|y| per node. */
lpdt_status lpdt_residual_add(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t Ca,
                              int32_t C, int32_t stride, int32_t ch_off,
                              const float *r, const float *a, float *y, float *amax_out, void *stream);
/* Adjoint: da = g_main + P^T(dy).  da may alias g_main. */
lpdt_status lpdt_residual_add_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t Ca,
                                  int32_t C, int32_t stride, int32_t ch_off,
                                  const float *dy, const float *g_main, float *da, void *stream);

/* Global average pool over HW positions and its adjoint (dx = dy/HW). */
lpdt_status lpdt_avgpool(int32_t nodes, int32_t B, int32_t HW, int32_t C,
                         const float *x, float *y, void *stream);
lpdt_status lpdt_avgpool_bwd(int32_t nodes, int32_t B, int32_t HW, int32_t C,
                             const float *dy, float *dx, void *stream);

/* 2x2/stride-2 max-pool on fp32 NHWC; idx (int8, output shape) records the
 * winning tap 0..3 (row-major, first maximum wins).  H and W must be even. */
lpdt_status lpdt_maxpool2x2(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                            const float *x, float *y, int8_t *idx, void *stream);
lpdt_status lpdt_maxpool2x2_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                const float *dy, const int8_t *idx, float *dx, void *stream);

/* Softmax cross-entropy per node (mean over the node's batch):
 * loss[n], dlogits = (softmax - onehot)/B.  logits fp32 [nodes][B][K], labels int32 [nodes][B].
 * Labels must lie in [0, K).  The kernel checks each one before using it: a sample whose label
 * is out of range adds nothing to its node's loss, gets dlogits = softmax/B (no one-hot term), and
 * LPDT_ERR_INVALID_ARG is written to dev_status (one int32, caller-zeroed, nullable); no memory
 * outside the logits row is touched. */
lpdt_status lpdt_softmax_ce(int32_t nodes, int32_t B, int32_t K, const float *logits,
                            const int32_t *labels, float *loss, float *dlogits, int32_t *dev_status,
                            void *stream);

/* out[n][c] = sum_b x[n][b][c] (bias gradient); node n of out at out + n*out_node_stride. */
lpdt_status lpdt_colsum(int32_t nodes, int32_t B, int32_t C, const float *x,
                        float *out, int64_t out_node_stride, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LPDT_H */
