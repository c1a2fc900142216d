/*
 * lpdt_oracle.c — CPU oracle for the 8-bit decentralized training step
 * (arXiv 2111.09389).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow restatement of what the
 * method computes, used only to check the CUDA library and to be timed as the
 * CPU baseline.  It shares no code with the CUDA path and the product never
 * calls it.
 *
 * Conventions
 *   nodes        : the N simulated decentralized nodes; always the leading
 *                  dimension, each node has its own tensors and scales.
 *   activations  : NHWC   [nodes][B][H][W][C]
 *   weights      : KRSC   [nodes][Cout][R][S][Cin]
 *   integer sums : int32 result, with an int64 shadow; any accumulator that
 *                  leaves the int32 range is counted in *overflow.
 *   floating point: where a value decides an integer downstream (a quantised
 *                  code) the arithmetic is a stated sequence of individually
 *                  rounded fp32 operations; every reduction is accumulated in
 *                  double and rounded once.  The *_f64 variants evaluate the
 *                  same formulas entirely in double (the plain definition).
 *
 * Parity status of the pins (tests/test_oracle_*.py):
 *   quantizer, integer contractions, Range-EvoNorm fwd/bwd, gossip, Philox:
 *   pinned (hand examples, closed forms, brute force, invariants, finite
 *   differences, published known-answer vectors).
 *   Range-EvoNorm backward at tied extrema: pinned only to the stated
 *   subgradient rule (lowest index wins) — the paper gives no rule.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef long long i64;

/* Threads the contraction loops will use (1 without OpenMP). */
int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------
 * Philox4x32-10 counter-based generator (Salmon, Moraes, Dror, Shaw:
 * "Parallel random numbers: as easy as 1, 2, 3", SC'11), written from the
 * published round function: two 32x32->64 multiplies, a word permutation
 * with the key xored in, and a Weyl key schedule; ten rounds.
 * ---------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Uniform in [0,1) with 24 random bits for element i of node `node`:
 * word (i mod 4) of the block whose counter is (i/4 low, i/4 high, node,
 * ctr_offset) under key (seed low, seed high). */
static float philox_uniform(i64 i, int node, uint64_t seed, uint32_t ctr_offset)
{
    uint64_t blk = (uint64_t)i >> 2;
    uint32_t ctr[4] = { (uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)node, ctr_offset };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t r[4];
    orc_philox4x32_10(ctr, key, r);
    return (float)(r[i & 3] >> 8) * 0x1p-24f;
}

/* ------------------------------------------------------------------------
 * Quantizer (Section 3, "Low Precision Training": 8-bit integer
 * quantization of weights, activations and layer gradients; the paper names
 * the scheme only by citation, so the formulas below are this build's
 * reading: one range per tensor per node, uniform grid).
 *
 * Symmetric signed mode:  amax = max|x|, scale = amax/127, inv = 127/amax,
 *   nearest : q = clamp(rne(x*inv), -127, 127)
 *   stochastic: t = x*inv, f = t - floor(t),  q = floor(t) + [u < f]
 * with u the Philox uniform above.  amax == 0 gives scale 1 and q = 0.
 * Every operation is a single fp32 operation.
 * rounding: 0 = nearest-even, 1 = stochastic.
 * ---------------------------------------------------------------------- */
void orc_quantize_sym_s8(const float *x, int nodes, i64 n, int rounding,
                         uint64_t seed, uint32_t ctr_offset,
                         int8_t *q, float *scale)
{
    for (int nd = 0; nd < nodes; ++nd) {
        const float *xn = x + (i64)nd * n;
        int8_t *qn = q + (i64)nd * n;
        float amax = 0.0f;
        for (i64 i = 0; i < n; ++i) {
            float a = fabsf(xn[i]);
            if (a > amax) amax = a;
        }
        if (amax == 0.0f) {
            scale[nd] = 1.0f;
            memset(qn, 0, (size_t)n);
            continue;
        }
        float s = amax / 127.0f;
        float inv = 127.0f / amax;
        scale[nd] = s;
        for (i64 i = 0; i < n; ++i) {
            float t = xn[i] * inv;
            float r;
            if (rounding == 0) {
                r = nearbyintf(t);          /* default mode: ties to even */
            } else {
                float fl = floorf(t);
                float f = t - fl;           /* exact */
                float u = philox_uniform(i, nd, seed, ctr_offset);
                r = fl + ((u < f) ? 1.0f : 0.0f);
            }
            if (r > 127.0f) r = 127.0f;
            if (r < -127.0f) r = -127.0f;
            qn[i] = (int8_t)r;
        }
    }
}

/* Affine unsigned mode (zero-point form of the cited scheme):
 *   lo = min(0, min x), hi = max(0, max x), scale = (hi-lo)/255 (1 if equal)
 *   zp = clamp(rne(-lo/scale), 0, 255),  q = clamp(rne(x/scale) + zp, 0, 255)
 * so that real zero is exactly representable. */
void orc_quantize_affine_u8(const float *x, int nodes, i64 n,
                            uint8_t *q, float *scale, int32_t *zero_point)
{
    for (int nd = 0; nd < nodes; ++nd) {
        const float *xn = x + (i64)nd * n;
        uint8_t *qn = q + (i64)nd * n;
        float lo = 0.0f, hi = 0.0f;
        for (i64 i = 0; i < n; ++i) {
            if (xn[i] < lo) lo = xn[i];
            if (xn[i] > hi) hi = xn[i];
        }
        float s = (hi == lo) ? 1.0f : (hi - lo) / 255.0f;
        float zf = nearbyintf(-lo / s);
        if (zf < 0.0f) zf = 0.0f;
        if (zf > 255.0f) zf = 255.0f;
        scale[nd] = s;
        zero_point[nd] = (int32_t)zf;
        for (i64 i = 0; i < n; ++i) {
            float r = nearbyintf(xn[i] / s) + zf;
            if (r < 0.0f) r = 0.0f;
            if (r > 255.0f) r = 255.0f;
            qn[i] = (uint8_t)r;
        }
    }
}

/* Dequantize: x' = scale * (q - zp); zero_point may be NULL (symmetric). */
void orc_dequantize_s8(const int8_t *q, int nodes, i64 n, const float *scale, float *y)
{
    for (int nd = 0; nd < nodes; ++nd)
        for (i64 i = 0; i < n; ++i)
            y[(i64)nd * n + i] = (float)q[(i64)nd * n + i] * scale[nd];
}

void orc_dequantize_u8(const uint8_t *q, int nodes, i64 n, const float *scale,
                       const int32_t *zero_point, float *y)
{
    for (int nd = 0; nd < nodes; ++nd)
        for (i64 i = 0; i < n; ++i)
            y[(i64)nd * n + i] =
                (float)((int32_t)q[(i64)nd * n + i] - zero_point[nd]) * scale[nd];
}

/* ------------------------------------------------------------------------
 * Integer contractions: the plain definitions of the convolution and of its
 * two adjoints (Section 3: forward, layer-gradient and weight-gradient
 * products all run on 8-bit operands; Table "hardware_training" Conv row
 * counts the three as equal).  A linear layer is the case R=S=H=W=1.
 * Out-of-image taps read zero.  Ho = (H + 2*pad - R)/stride + 1.
 * ---------------------------------------------------------------------- */
static int32_t wrap32(i64 v, i64 *overflow)
{
    if (v > INT32_MAX || v < INT32_MIN) {
        #pragma omp atomic
        (*overflow)++;
    }
    return (int32_t)(uint32_t)(uint64_t)v;
}

void orc_qconv_fwd(int nodes, int B, int H, int W, int Cin, int Cout, int R, int S,
                   int stride, int pad, const int8_t *A, const int8_t *Wq,
                   int32_t *acc, i64 *overflow)
{
    const int Ho = (H + 2 * pad - R) / stride + 1;
    const int Wo = (W + 2 * pad - S) / stride + 1;
    *overflow = 0;
    #pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < nodes; ++n)
    for (int b = 0; b < B; ++b)
    for (int oh = 0; oh < Ho; ++oh)
    for (int ow = 0; ow < Wo; ++ow)
    for (int co = 0; co < Cout; ++co) {
        i64 sum = 0;
        for (int r = 0; r < R; ++r) {
            int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < S; ++s) {
                int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= W) continue;
                const int8_t *a = A + ((((i64)n * B + b) * H + ih) * W + iw) * Cin;
                const int8_t *w = Wq + ((((i64)n * Cout + co) * R + r) * S + s) * Cin;
                for (int ci = 0; ci < Cin; ++ci)
                    sum += (int32_t)a[ci] * (int32_t)w[ci];
            }
        }
        acc[((((i64)n * B + b) * Ho + oh) * Wo + ow) * Cout + co] = wrap32(sum, overflow);
    }
}

/* Forward contraction on affine (zero-point) 8-bit operands, the quantization scheme
 * Section 3 names: real a = sA*(qa - zA), real w = sW*(qw - zW), qa and qw unsigned
 * codes, one zero point per node and tensor.  The convolution pads with real zeros,
 * so a tap outside the image contributes nothing:
 *   acc[n,b,oh,ow,co] = sum over taps inside the image, ci of (qa - zA[n]) * (qw - zW[n]). */
void orc_qconv_fwd_affine(int nodes, int B, int H, int W, int Cin, int Cout, int R, int S,
                          int stride, int pad, const uint8_t *A, const int32_t *zA,
                          const uint8_t *Wq, const int32_t *zW, int32_t *acc, i64 *overflow)
{
    const int Ho = (H + 2 * pad - R) / stride + 1;
    const int Wo = (W + 2 * pad - S) / stride + 1;
    *overflow = 0;
    #pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < nodes; ++n)
    for (int b = 0; b < B; ++b)
    for (int oh = 0; oh < Ho; ++oh)
    for (int ow = 0; ow < Wo; ++ow)
    for (int co = 0; co < Cout; ++co) {
        i64 sum = 0;
        for (int r = 0; r < R; ++r) {
            int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= H) continue;
            for (int s = 0; s < S; ++s) {
                int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= W) continue;
                const uint8_t *a = A + ((((i64)n * B + b) * H + ih) * W + iw) * Cin;
                const uint8_t *w = Wq + ((((i64)n * Cout + co) * R + r) * S + s) * Cin;
                for (int ci = 0; ci < Cin; ++ci)
                    sum += ((int32_t)a[ci] - zA[n]) * ((int32_t)w[ci] - zW[n]);
            }
        }
        acc[((((i64)n * B + b) * Ho + oh) * Wo + ow) * Cout + co] = wrap32(sum, overflow);
    }
}

/* dA[n,b,ih,iw,ci] = sum over (oh,ow,r,s,co) with ih = oh*stride + r - pad,
 * iw = ow*stride + s - pad of E[n,b,oh,ow,co] * W[n,co,r,s,ci]. */
void orc_qconv_bwd_data(int nodes, int B, int H, int W, int Cin, int Cout, int R, int S,
                        int stride, int pad, const int8_t *E, const int8_t *Wq,
                        int32_t *dA, i64 *overflow)
{
    const int Ho = (H + 2 * pad - R) / stride + 1;
    const int Wo = (W + 2 * pad - S) / stride + 1;
    *overflow = 0;
    #pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < nodes; ++n)
    for (int b = 0; b < B; ++b)
    for (int ih = 0; ih < H; ++ih)
    for (int iw = 0; iw < W; ++iw)
    for (int ci = 0; ci < Cin; ++ci) {
        i64 sum = 0;
        for (int r = 0; r < R; ++r) {
            int th = ih + pad - r;
            if (th < 0 || th % stride != 0) continue;
            int oh = th / stride;
            if (oh >= Ho) continue;
            for (int s = 0; s < S; ++s) {
                int tw = iw + pad - s;
                if (tw < 0 || tw % stride != 0) continue;
                int ow = tw / stride;
                if (ow >= Wo) continue;
                const int8_t *e = E + ((((i64)n * B + b) * Ho + oh) * Wo + ow) * Cout;
                for (int co = 0; co < Cout; ++co)
                    sum += (int32_t)e[co] *
                           (int32_t)Wq[((((i64)n * Cout + co) * R + r) * S + s) * Cin + ci];
            }
        }
        dA[((((i64)n * B + b) * H + ih) * W + iw) * Cin + ci] = wrap32(sum, overflow);
    }
}

/* dW[n,co,r,s,ci] = sum over (b,oh,ow) of E[n,b,oh,ow,co] * A[n,b,oh*stride+r-pad,
 * ow*stride+s-pad,ci]. */
void orc_qconv_bwd_weight(int nodes, int B, int H, int W, int Cin, int Cout, int R, int S,
                          int stride, int pad, const int8_t *E, const int8_t *A,
                          int32_t *dW, i64 *overflow)
{
    const int Ho = (H + 2 * pad - R) / stride + 1;
    const int Wo = (W + 2 * pad - S) / stride + 1;
    *overflow = 0;
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < nodes; ++n)
    for (int co = 0; co < Cout; ++co)
    for (int r = 0; r < R; ++r)
    for (int s = 0; s < S; ++s)
    for (int ci = 0; ci < Cin; ++ci) {
        i64 sum = 0;
        for (int b = 0; b < B; ++b)
        for (int oh = 0; oh < Ho; ++oh) {
            int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= H) continue;
            for (int ow = 0; ow < Wo; ++ow) {
                int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= W) continue;
                sum += (int32_t)E[((((i64)n * B + b) * Ho + oh) * Wo + ow) * Cout + co] *
                       (int32_t)A[((((i64)n * B + b) * H + ih) * W + iw) * Cin + ci];
            }
        }
        dW[((((i64)n * Cout + co) * R + r) * S + s) * Cin + ci] = wrap32(sum, overflow);
    }
}

/* Backward products on affine (zero-point) 8-bit operands (Section 3 names the scheme; the layer
 * gradient, the weights and the saved activations are unsigned codes with one zero point per node and
 * tensor: real = scale*(code - zero point)).  They are the adjoints of orc_qconv_fwd_affine: a tap that
 * lies outside the image pairs nothing with nothing, so it is simply absent from the sums.
 *   dA[n,b,ih,iw,ci] = sum over (oh,ow,r,s,co) with ih = oh*stride + r - pad, iw = ow*stride + s - pad
 *                      of (E[n,b,oh,ow,co] - zE[n]) * (W[n,co,r,s,ci] - zW[n]) */
void orc_qconv_bwd_data_affine(int nodes, int B, int H, int W, int Cin, int Cout, int R, int S,
                               int stride, int pad, const uint8_t *E, const int32_t *zE,
                               const uint8_t *Wq, const int32_t *zW, int32_t *dA, i64 *overflow)
{
    const int Ho = (H + 2 * pad - R) / stride + 1;
    const int Wo = (W + 2 * pad - S) / stride + 1;
    *overflow = 0;
    #pragma omp parallel for collapse(3) schedule(static)
    for (int n = 0; n < nodes; ++n)
    for (int b = 0; b < B; ++b)
    for (int ih = 0; ih < H; ++ih)
    for (int iw = 0; iw < W; ++iw)
    for (int ci = 0; ci < Cin; ++ci) {
        i64 sum = 0;
        for (int r = 0; r < R; ++r) {
            int th = ih + pad - r;
            if (th < 0 || th % stride != 0) continue;
            int oh = th / stride;
            if (oh >= Ho) continue;
            for (int s = 0; s < S; ++s) {
                int tw = iw + pad - s;
                if (tw < 0 || tw % stride != 0) continue;
                int ow = tw / stride;
                if (ow >= Wo) continue;
                const uint8_t *e = E + ((((i64)n * B + b) * Ho + oh) * Wo + ow) * Cout;
                for (int co = 0; co < Cout; ++co)
                    sum += ((int32_t)e[co] - zE[n]) *
                           ((int32_t)Wq[((((i64)n * Cout + co) * R + r) * S + s) * Cin + ci] - zW[n]);
            }
        }
        dA[((((i64)n * B + b) * H + ih) * W + iw) * Cin + ci] = wrap32(sum, overflow);
    }
}

/*   dW[n,co,r,s,ci] = sum over (b,oh,ow) whose tap (r,s) lies inside the image of
 *                     (E[n,b,oh,ow,co] - zE[n]) * (A[n,b,oh*stride+r-pad,ow*stride+s-pad,ci] - zA[n]) */
void orc_qconv_bwd_weight_affine(int nodes, int B, int H, int W, int Cin, int Cout, int R, int S,
                                 int stride, int pad, const uint8_t *E, const int32_t *zE,
                                 const uint8_t *A, const int32_t *zA, int32_t *dW, i64 *overflow)
{
    const int Ho = (H + 2 * pad - R) / stride + 1;
    const int Wo = (W + 2 * pad - S) / stride + 1;
    *overflow = 0;
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < nodes; ++n)
    for (int co = 0; co < Cout; ++co)
    for (int r = 0; r < R; ++r)
    for (int s = 0; s < S; ++s)
    for (int ci = 0; ci < Cin; ++ci) {
        i64 sum = 0;
        for (int b = 0; b < B; ++b)
        for (int oh = 0; oh < Ho; ++oh) {
            int ih = oh * stride + r - pad;
            if (ih < 0 || ih >= H) continue;
            for (int ow = 0; ow < Wo; ++ow) {
                int iw = ow * stride + s - pad;
                if (iw < 0 || iw >= W) continue;
                sum += ((int32_t)E[((((i64)n * B + b) * Ho + oh) * Wo + ow) * Cout + co] - zE[n]) *
                       ((int32_t)A[((((i64)n * B + b) * H + ih) * W + iw) * Cin + ci] - zA[n]);
            }
        }
        dW[((((i64)n * Cout + co) * R + r) * S + s) * Cin + ci] = wrap32(sum, overflow);
    }
}

/* Dequantize accumulators: sc = s1[n]*s2[n] (one fp32 multiply),
 * y = (float)acc * sc, then + bias[n][i mod C] when bias != NULL. */
void orc_dequant_acc(const int32_t *acc, int nodes, i64 n_per_node, int C,
                     const float *s1, const float *s2, const float *bias, float *y)
{
    for (int nd = 0; nd < nodes; ++nd) {
        float sc = s1[nd] * s2[nd];
        for (i64 i = 0; i < n_per_node; ++i) {
            float v = (float)acc[(i64)nd * n_per_node + i] * sc;
            if (bias) v = v + bias[(i64)nd * C + (i % C)];
            y[(i64)nd * n_per_node + i] = v;
        }
    }
}

/* ------------------------------------------------------------------------
 * Range-EvoNorm (Eq. "ren") forward and backward, instantiated twice from
 * ren_body.inc: REAL = float (each operation individually rounded; the
 * precision the kernels take their decisions in) and REAL = double (the
 * closed form).
 * ---------------------------------------------------------------------- */
#define REAL float
#define SUFFIX(name) name##_f32
#include "ren_body.inc"
#undef REAL
#undef SUFFIX

#define REAL double
#define SUFFIX(name) name##_f64
#include "ren_body.inc"
#undef REAL
#undef SUFFIX

/* ------------------------------------------------------------------------
 * The comparison layers of Section 3 (Eq. "en" and Eq. "rbn"), in double.
 * ---------------------------------------------------------------------- */

/* EvoNorm-S0 (Eq. "en"), per node n, sample b, group G of cpg = C/groups consecutive channels:
 *     mu, var = mean and (biased) variance of x over the group's (h, w, c)
 *     D       = sqrt(var + eps)
 *     y       = gamma_c * (x * sigmoid(v_c * x)) / D + beta_c
 * The equation has no eps (eps = 0 reproduces it) and does not say which variance; the divide-by-count
 * form is the reading taken.  gmean / gvar [nodes][B][groups] receive the statistics. */
void orc_evonorm_s0_fwd(int nodes, int B, int H, int W, int C, int groups, double eps,
                        const float *x, const float *v, const float *gamma, const float *beta,
                        double *y, double *gmean, double *gvar)
{
    const int cpg = C / groups;
    const double cnt = (double)H * W * cpg;
    for (int n = 0; n < nodes; ++n)
    for (int b = 0; b < B; ++b)
    for (int g = 0; g < groups; ++g) {
        const float *xs = x + ((i64)n * B + b) * H * W * C;
        double *ys = y + ((i64)n * B + b) * H * W * C;
        double sum = 0.0;
        for (int p = 0; p < H * W; ++p)
            for (int c = g * cpg; c < (g + 1) * cpg; ++c) sum += (double)xs[p * C + c];
        const double mu = sum / cnt;
        double sq = 0.0;
        for (int p = 0; p < H * W; ++p)
            for (int c = g * cpg; c < (g + 1) * cpg; ++c) {
                double dlt = (double)xs[p * C + c] - mu;
                sq += dlt * dlt;
            }
        const double var = sq / cnt;
        const i64 sg = ((i64)n * B + b) * groups + g;
        gmean[sg] = mu; gvar[sg] = var;
        const double D = sqrt(var + eps);
        for (int p = 0; p < H * W; ++p)
            for (int c = g * cpg; c < (g + 1) * cpg; ++c) {
                double xv = (double)xs[p * C + c];
                double sig = 1.0 / (1.0 + exp(-(double)v[(i64)n * C + c] * xv));
                ys[p * C + c] = (double)gamma[(i64)n * C + c] * (xv * sig) / D + (double)beta[(i64)n * C + c];
            }
    }
}

/* Backward of EvoNorm-S0 (derived from the forward; the paper prints none).  With t = dy*gamma_c,
 * sig = sigmoid(v_c x), m = x*sig, cnt = H*W*cpg and S = sum over the group of t*m:
 *     dx      = t * (sig + v_c*x*sig*(1 - sig)) / D  -  S * (x - mu) / (cnt * D^3)
 *     dbeta_c = sum dy;  dgamma_c = sum dy * m / D;  dv_c = sum t * x*x*sig*(1 - sig) / D
 * (sums over the node's b, h, w).  gmean / gvar are the forward's statistics as the caller stored them. */
void orc_evonorm_s0_bwd(int nodes, int B, int H, int W, int C, int groups, double eps,
                        const float *dy, const float *x, const float *v, const float *gamma,
                        const float *gmean, const float *gvar,
                        double *dx, double *dv, double *dgamma, double *dbeta)
{
    const int cpg = C / groups;
    const double cnt = (double)H * W * cpg;
    for (i64 i = 0; i < (i64)nodes * C; ++i) { dv[i] = 0.0; dgamma[i] = 0.0; dbeta[i] = 0.0; }
    for (int n = 0; n < nodes; ++n)
    for (int b = 0; b < B; ++b)
    for (int g = 0; g < groups; ++g) {
        const float *xs = x + ((i64)n * B + b) * H * W * C;
        const float *dys = dy + ((i64)n * B + b) * H * W * C;
        double *dxs = dx + ((i64)n * B + b) * H * W * C;
        const i64 sg = ((i64)n * B + b) * groups + g;
        const double mu = (double)gmean[sg], D = sqrt((double)gvar[sg] + eps);
        double S = 0.0;
        for (int p = 0; p < H * W; ++p)
            for (int c = g * cpg; c < (g + 1) * cpg; ++c) {
                double xv = (double)xs[p * C + c], vc = (double)v[(i64)n * C + c];
                double sig = 1.0 / (1.0 + exp(-vc * xv));
                S += (double)dys[p * C + c] * (double)gamma[(i64)n * C + c] * (xv * sig);
            }
        for (int p = 0; p < H * W; ++p)
            for (int c = g * cpg; c < (g + 1) * cpg; ++c) {
                double xv = (double)xs[p * C + c], vc = (double)v[(i64)n * C + c];
                double gc = (double)gamma[(i64)n * C + c], dyv = (double)dys[p * C + c];
                double sig = 1.0 / (1.0 + exp(-vc * xv));
                double m = xv * sig, t = dyv * gc, sp = sig * (1.0 - sig);
                dxs[p * C + c] = t * (sig + vc * xv * sp) / D - S * (xv - mu) / (cnt * D * D * D);
                dbeta[(i64)n * C + c] += dyv;
                dgamma[(i64)n * C + c] += dyv * m / D;
                dv[(i64)n * C + c] += t * xv * xv * sp / D;
            }
    }
}

/* Range batch-norm (Eq. "rbn"), per node n and channel c over the node's batch (b, h, w):
 *     mu    = mean of x;  range = max(x - mu) - min(x - mu) = max x - min x
 *     D     = Cb * range + eps,  Cb = 1/sqrt(2 ln B)  (the equation's C(b), b = batch size; B >= 2)
 *     y     = gamma_c * (x - mu) / D + beta_c
 * cmean / cmin / cmax [nodes][C] receive the statistics, argmin / argmax the lowest (b*H*W + p)
 * position attaining the extremum (for the backward's sub-gradient, as in Range-EvoNorm). */
void orc_range_bn_fwd(int nodes, int B, int H, int W, int C, double eps,
                      const float *x, const float *gamma, const float *beta,
                      double *y, double *cmean, float *cmin, float *cmax, int32_t *argmin, int32_t *argmax)
{
    const double Cb = 1.0 / sqrt(2.0 * log((double)B));
    const i64 P = (i64)B * H * W;
    for (int n = 0; n < nodes; ++n)
    for (int c = 0; c < C; ++c) {
        const float *xs = x + (i64)n * P * C;
        double *ys = y + (i64)n * P * C;
        double sum = 0.0;
        float mx = 0, mn = 0; int32_t amx = -1, amn = -1;
        for (i64 p = 0; p < P; ++p) {
            float val = xs[p * C + c];
            sum += (double)val;
            if (amx < 0 || val > mx) { mx = val; amx = (int32_t)p; }
            if (amn < 0 || val < mn) { mn = val; amn = (int32_t)p; }
        }
        const double mu = sum / (double)P;
        cmean[(i64)n * C + c] = mu; cmin[(i64)n * C + c] = mn; cmax[(i64)n * C + c] = mx;
        argmin[(i64)n * C + c] = amn; argmax[(i64)n * C + c] = amx;
        const double D = Cb * ((double)mx - (double)mn) + eps;
        for (i64 p = 0; p < P; ++p)
            ys[p * C + c] = (double)gamma[(i64)n * C + c] * ((double)xs[p * C + c] - mu) / D + (double)beta[(i64)n * C + c];
    }
}

/* Backward of range batch-norm (derived).  With t = dy*gamma_c, P = B*H*W, xc = x - mu:
 *     dx      = t / D - (sum t) / (P * D) - Cb * (sum t*xc) / D^2 * ([p = argmax] - [p = argmin])
 *     dbeta_c = sum dy;  dgamma_c = sum dy * xc / D
 * (the last dx term is skipped when argmax = argmin). */
void orc_range_bn_bwd(int nodes, int B, int H, int W, int C, double eps,
                      const float *dy, const float *x, const float *gamma,
                      const float *cmean, const float *cmin, const float *cmax,
                      const int32_t *argmin, const int32_t *argmax,
                      double *dx, double *dgamma, double *dbeta)
{
    const double Cb = 1.0 / sqrt(2.0 * log((double)B));
    const i64 P = (i64)B * H * W;
    for (int n = 0; n < nodes; ++n)
    for (int c = 0; c < C; ++c) {
        const float *xs = x + (i64)n * P * C;
        const float *dys = dy + (i64)n * P * C;
        double *dxs = dx + (i64)n * P * C;
        const i64 nc = (i64)n * C + c;
        const double mu = (double)cmean[nc], gc = (double)gamma[nc];
        const double D = Cb * ((double)cmax[nc] - (double)cmin[nc]) + eps;
        double sdy = 0.0, sdx = 0.0;          /* sum dy, sum dy*xc */
        for (i64 p = 0; p < P; ++p) {
            double dyv = (double)dys[p * C + c], xc = (double)xs[p * C + c] - mu;
            sdy += dyv; sdx += dyv * xc;
        }
        const double st = gc * sdy, stx = gc * sdx;
        for (i64 p = 0; p < P; ++p)
            dxs[p * C + c] = (double)dys[p * C + c] * gc / D - st / ((double)P * D);
        if (argmax[nc] != argmin[nc]) {
            const double coef = Cb * stx / (D * D);
            dxs[(i64)argmax[nc] * C + c] -= coef;
            dxs[(i64)argmin[nc] * C + c] += coef;
        }
        dbeta[nc] = sdy;
        dgamma[nc] = sdx / D;
    }
}

/* ------------------------------------------------------------------------
 * Gossip with compressed model updates (Algorithm 3, CHOCO-SGD, the steps
 * "compute and compress", "update the public copies", "gossip update").
 *   delta_i = xhalf_i - xhat_i                      (fp32: it decides the top-k)
 *   q_i     = delta_i on the k_s largest |delta_i| of each segment s
 *             (equal magnitudes: the lower index is kept), else 0
 *   xhat_i <- xhat_i + q_i                          (one fp32 add)
 *   x_i     = xhalf_i + gamma * sum_j W[i][j] * (xhat_j - xhat_i)   (double,
 *             with the UPDATED xhat, j ascending), rounded to fp32 once.
 * q_out (nullable) receives q.  seg_off has n_seg+1 entries, seg_k n_seg.
 * ---------------------------------------------------------------------- */
typedef struct { float mag; i64 idx; } mag_idx;

static int cmp_mag_desc(const void *pa, const void *pb)
{
    const mag_idx *a = (const mag_idx *)pa, *b = (const mag_idx *)pb;
    if (a->mag > b->mag) return -1;
    if (a->mag < b->mag) return 1;
    return (a->idx < b->idx) ? -1 : (a->idx > b->idx);
}

void orc_gossip_mix(int nodes, i64 d, const float *x_half, float *x_hat, float *x_out,
                    const float *Wmix, float gamma, int n_seg, const i64 *seg_off,
                    const i64 *seg_k, float *q_out)
{
    float *q = (float *)calloc((size_t)nodes * (size_t)d, sizeof(float));
    mag_idx *tmp = (mag_idx *)malloc((size_t)d * sizeof(mag_idx));
    for (int i = 0; i < nodes; ++i) {
        for (int s = 0; s < n_seg; ++s) {
            i64 lo = seg_off[s], hi = seg_off[s + 1], len = hi - lo, k = seg_k[s];
            if (k >= len) {
                for (i64 e = lo; e < hi; ++e)
                    q[i * d + e] = x_half[i * d + e] - x_hat[i * d + e];
                continue;
            }
            for (i64 e = lo; e < hi; ++e) {
                float delta = x_half[i * d + e] - x_hat[i * d + e];
                tmp[e - lo].mag = fabsf(delta);
                tmp[e - lo].idx = e;
            }
            qsort(tmp, (size_t)len, sizeof(mag_idx), cmp_mag_desc);
            for (i64 t = 0; t < k; ++t) {
                i64 e = tmp[t].idx;
                q[i * d + e] = x_half[i * d + e] - x_hat[i * d + e];
            }
        }
    }
    for (i64 t = 0; t < (i64)nodes * d; ++t) x_hat[t] = x_hat[t] + q[t];
    for (int i = 0; i < nodes; ++i)
        for (i64 e = 0; e < d; ++e) {
            double acc = 0.0;
            for (int j = 0; j < nodes; ++j)
                acc += (double)Wmix[i * nodes + j] *
                       ((double)x_hat[j * d + e] - (double)x_hat[i * d + e]);
            x_out[i * d + e] = (float)((double)x_half[i * d + e] + (double)gamma * acc);
        }
    if (q_out) memcpy(q_out, q, (size_t)nodes * (size_t)d * sizeof(float));
    free(tmp);
    free(q);
}

/* The same gossip step with 8-bit messages (the contributions list and the Data column of
 * the CIFAR table: quantized exchange is a quarter of the fp32 volume, alone or on top of
 * top-k).  The paper gives no formula for the message; the reading taken: the compressed
 * difference q is sent as signed 8-bit codes with one range per (node, segment), by the
 * same symmetric quantizer as every other tensor:
 *   amax = max |q| over the segment (the kept entries are the largest, so this is max |delta|),
 *   scale = amax / 127, inv = 127 / amax (scale = 1 when amax = 0),
 *   code = clamp(rne(delta * inv), -127, 127) on the kept entries, q = (float)code * scale,
 * each operation rounded to fp32 on its own.  The public copy absorbs the DEQUANTIZED message,
 * so sender and receivers hold the same x_hat and the rounding error stays in the next
 * difference (error feedback).  codes_out (nullable) receives the codes (0 where nothing is
 * sent), scale_out [nodes][n_seg] the scales. */
void orc_gossip_mix_q8(int nodes, i64 d, const float *x_half, float *x_hat, float *x_out,
                       const float *Wmix, float gamma, int n_seg, const i64 *seg_off,
                       const i64 *seg_k, float *q_out, int8_t *codes_out, float *scale_out)
{
    float *q = (float *)calloc((size_t)nodes * (size_t)d, sizeof(float));
    unsigned char *keep = (unsigned char *)calloc((size_t)d, 1);
    mag_idx *tmp = (mag_idx *)malloc((size_t)d * sizeof(mag_idx));
    if (codes_out) memset(codes_out, 0, (size_t)nodes * (size_t)d);
    for (int i = 0; i < nodes; ++i) {
        for (int s = 0; s < n_seg; ++s) {
            i64 lo = seg_off[s], hi = seg_off[s + 1], len = hi - lo, k = seg_k[s];
            if (k > len) k = len;
            for (i64 e = lo; e < hi; ++e) {
                float delta = x_half[i * d + e] - x_hat[i * d + e];
                tmp[e - lo].mag = fabsf(delta);
                tmp[e - lo].idx = e;
                keep[e] = 0;
            }
            if (k < len) qsort(tmp, (size_t)len, sizeof(mag_idx), cmp_mag_desc);
            float amax = 0.f;
            for (i64 t = 0; t < k; ++t) {
                keep[tmp[t].idx] = 1;
                if (tmp[t].mag > amax) amax = tmp[t].mag;
            }
            float scale = 1.f, inv = 1.f;
            if (amax > 0.f) { scale = amax / 127.0f; inv = 127.0f / amax; }
            scale_out[(i64)i * n_seg + s] = scale;
            for (i64 e = lo; e < hi; ++e) {
                if (!keep[e]) continue;
                float delta = x_half[i * d + e] - x_hat[i * d + e];
                float t = delta * inv;
                float r = rintf(t);                /* round half to even */
                if (r > 127.f) r = 127.f;
                if (r < -127.f) r = -127.f;
                q[i * d + e] = r * scale;
                if (codes_out) codes_out[i * d + e] = (int8_t)r;
            }
        }
    }
    for (i64 t = 0; t < (i64)nodes * d; ++t) x_hat[t] = x_hat[t] + q[t];
    for (int i = 0; i < nodes; ++i)
        for (i64 e = 0; e < d; ++e) {
            double acc = 0.0;
            for (int j = 0; j < nodes; ++j)
                acc += (double)Wmix[i * nodes + j] *
                       ((double)x_hat[j * d + e] - (double)x_hat[i * d + e]);
            x_out[i * d + e] = (float)((double)x_half[i * d + e] + (double)gamma * acc);
        }
    if (q_out) memcpy(q_out, q, (size_t)nodes * (size_t)d * sizeof(float));
    free(tmp);
    free(keep);
    free(q);
}

/* Deep-Squeeze gossip step (supplementary Algorithm 2, steps 5-10), all nodes at once:
 *   v_i = x_half_i + delta_i                       (error compensated update)
 *   c_i = C[v_i]: per segment the k entries of largest |v| (ties: lower index), the rest 0;
 *         with 8-bit messages the kept entries go through the symmetric quantizer
 *         (one range per node and segment), as in orc_gossip_mix_q8
 *   delta_i <- v_i - c_i                           (what was not sent is carried over)
 *   x_i = x_half_i + eta * sum_j (W_ij - I_ij) c_j = x_half_i + eta * (sum_j W_ij c_j - c_i)
 * delta is updated in place; c_out (nullable) receives the messages, scale_out (nullable
 * unless bits = 8) the quantizer steps.  fp32 elementwise steps, double for the mix sum. */
void orc_deepsqueeze_mix(int nodes, i64 d, const float *x_half, float *delta, float *x_out,
                         const float *Wmix, float eta, int n_seg, const i64 *seg_off,
                         const i64 *seg_k, int bits, float *c_out, float *scale_out)
{
    float *c = (float *)calloc((size_t)nodes * (size_t)d, sizeof(float));
    unsigned char *keep = (unsigned char *)calloc((size_t)d, 1);
    mag_idx *tmp = (mag_idx *)malloc((size_t)d * sizeof(mag_idx));
    for (int i = 0; i < nodes; ++i) {
        for (int s = 0; s < n_seg; ++s) {
            i64 lo = seg_off[s], hi = seg_off[s + 1], len = hi - lo, k = seg_k[s];
            if (k > len) k = len;
            for (i64 e = lo; e < hi; ++e) {
                float v = x_half[i * d + e] + delta[i * d + e];
                tmp[e - lo].mag = fabsf(v);
                tmp[e - lo].idx = e;
                keep[e] = 0;
            }
            if (k < len) qsort(tmp, (size_t)len, sizeof(mag_idx), cmp_mag_desc);
            float amax = 0.f;
            for (i64 t = 0; t < k; ++t) {
                keep[tmp[t].idx] = 1;
                if (tmp[t].mag > amax) amax = tmp[t].mag;
            }
            float scale = 1.f, inv = 1.f;
            if (amax > 0.f) { scale = amax / 127.0f; inv = 127.0f / amax; }
            if (scale_out) scale_out[(i64)i * n_seg + s] = scale;
            for (i64 e = lo; e < hi; ++e) {
                float v = x_half[i * d + e] + delta[i * d + e];
                float msg = 0.f;
                if (keep[e]) {
                    msg = v;
                    if (bits == 8) {
                        float r = rintf(v * inv);
                        if (r > 127.f) r = 127.f;
                        if (r < -127.f) r = -127.f;
                        msg = r * scale;
                    }
                }
                c[i * d + e] = msg;
                delta[i * d + e] = v - msg;
            }
        }
    }
    for (int i = 0; i < nodes; ++i)
        for (i64 e = 0; e < d; ++e) {
            double acc = 0.0;
            for (int j = 0; j < nodes; ++j)
                acc += (double)Wmix[i * nodes + j] * (double)c[j * d + e];
            acc -= (double)c[i * d + e];
            x_out[i * d + e] = (float)((double)x_half[i * d + e] + (double)eta * acc);
        }
    if (c_out) memcpy(c_out, c, (size_t)nodes * (size_t)d * sizeof(float));
    free(tmp);
    free(keep);
    free(c);
}

/* Push-sum bias weights and de-biasing (supplementary Algorithms 4 and 5, the second line of
 * step 9 and step 10), for column-stochastic mixing matrices on directed graphs:
 *   u_new_i = u_i + eta * (sum_j W_ij u_j - u_i)        j ascending, fp32 steps
 *   z_i = x_i / u_new_i                                  the model the next gradient is taken at
 * x is the mixed model of the same step (from the Deep-Squeeze or CHOCO mix with the same W). */
void orc_pushsum_debias(int nodes, i64 d, const float *x, const float *u, const float *Wmix,
                        float eta, float *u_new, float *z)
{
    for (int i = 0; i < nodes; ++i) {
        float acc = 0.f;
        for (int j = 0; j < nodes; ++j) {
            float t = Wmix[i * nodes + j] * u[j];
            acc = acc + t;
        }
        acc = acc - u[i];
        float step = eta * acc;
        u_new[i] = u[i] + step;
    }
    for (int i = 0; i < nodes; ++i)
        for (i64 e = 0; e < d; ++e) z[i * d + e] = x[i * d + e] / u_new[i];
}

/* ------------------------------------------------------------------------
 * Glue around the layers of the step.
 * ---------------------------------------------------------------------- */

/* Local SGD update (Algorithm 1, "update the model"): out = x - lr*g,
 * a multiply then a subtract in fp32 on the fp32 master weights. */
void orc_sgd_update(i64 n, const float *x, const float *g, float lr, float *out)
{
    for (i64 i = 0; i < n; ++i) {
        float step = lr * g[i];
        out[i] = x[i] - step;
    }
}

/* Residual connection with the parameter-free shortcut: y = r + P(a), where P
 * subsamples a [B][H][W][Ca] spatially by `stride` and places its channels at
 * offset ch_off inside C >= Ca channels (zero elsewhere).  stride=1, Ca=C,
 * ch_off=0 is the identity shortcut.  Ho = ceil(H/stride). */
void orc_residual_add(int nodes, int B, int H, int W, int Ca, int C, int stride, int ch_off,
                      const float *r, const float *a, float *y)
{
    const int Ho = (H + stride - 1) / stride, Wo = (W + stride - 1) / stride;
    for (i64 nb = 0; nb < (i64)nodes * B; ++nb)
    for (int oh = 0; oh < Ho; ++oh)
    for (int ow = 0; ow < Wo; ++ow)
    for (int c = 0; c < C; ++c) {
        i64 o = ((nb * Ho + oh) * Wo + ow) * C + c;
        int ca = c - ch_off;
        float v = r[o];
        if (ca >= 0 && ca < Ca)
            v = v + a[((nb * H + (i64)oh * stride) * W + (i64)ow * stride) * Ca + ca];
        y[o] = v;
    }
}

/* Adjoint of the shortcut path: da = g_main + P^T(dy), with g_main the
 * gradient that reached `a` through the block's convolutions. */
void orc_residual_add_bwd(int nodes, int B, int H, int W, int Ca, int C, int stride, int ch_off,
                          const float *dy, const float *g_main, float *da)
{
    const int Ho = (H + stride - 1) / stride, Wo = (W + stride - 1) / stride;
    for (i64 nb = 0; nb < (i64)nodes * B; ++nb)
    for (int h = 0; h < H; ++h)
    for (int w = 0; w < W; ++w)
    for (int ca = 0; ca < Ca; ++ca) {
        i64 o = ((nb * H + h) * W + w) * Ca + ca;
        float v = g_main[o];
        if (h % stride == 0 && w % stride == 0)
            v = v + dy[((nb * Ho + h / stride) * Wo + w / stride) * C + ca + ch_off];
        da[o] = v;
    }
}

/* Global average pool over H*W (double sum, one division, rounded once). */
void orc_avgpool(int nodes, int B, int HW, int C, const float *x, float *y)
{
    for (i64 nb = 0; nb < (i64)nodes * B; ++nb)
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            for (int p = 0; p < HW; ++p) s += (double)x[(nb * HW + p) * C + c];
            y[nb * C + c] = (float)(s / (double)HW);
        }
}

void orc_avgpool_bwd(int nodes, int B, int HW, int C, const float *dy, float *dx)
{
    for (i64 nb = 0; nb < (i64)nodes * B; ++nb)
        for (int p = 0; p < HW; ++p)
            for (int c = 0; c < C; ++c)
                dx[(nb * HW + p) * C + c] = dy[nb * C + c] / (float)HW;
}

/* 2x2 max-pool, stride 2, NHWC fp32; idx records which of the four taps
 * (0..3, row-major, first maximum wins) carried the maximum. */
void orc_maxpool2x2(int nodes, int B, int H, int W, int C, const float *x, float *y, int8_t *idx)
{
    const int Ho = H / 2, Wo = W / 2;
    for (i64 nb = 0; nb < (i64)nodes * B; ++nb)
    for (int oh = 0; oh < Ho; ++oh)
    for (int ow = 0; ow < Wo; ++ow)
    for (int c = 0; c < C; ++c) {
        float best = 0.0f; int bi = -1;
        for (int t = 0; t < 4; ++t) {
            float v = x[((nb * H + 2 * oh + t / 2) * W + 2 * ow + t % 2) * C + c];
            if (bi < 0 || v > best) { best = v; bi = t; }
        }
        i64 o = ((nb * Ho + oh) * Wo + ow) * C + c;
        y[o] = best; idx[o] = (int8_t)bi;
    }
}

void orc_maxpool2x2_bwd(int nodes, int B, int H, int W, int C, const float *dy,
                        const int8_t *idx, float *dx)
{
    const int Ho = H / 2, Wo = W / 2;
    memset(dx, 0, (size_t)nodes * B * H * W * C * sizeof(float));
    for (i64 nb = 0; nb < (i64)nodes * B; ++nb)
    for (int oh = 0; oh < Ho; ++oh)
    for (int ow = 0; ow < Wo; ++ow)
    for (int c = 0; c < C; ++c) {
        i64 o = ((nb * Ho + oh) * Wo + ow) * C + c;
        int t = idx[o];
        dx[((nb * H + 2 * oh + t / 2) * W + 2 * ow + t % 2) * C + c] = dy[o];
    }
}

/* Softmax cross-entropy per node, mean over the node's batch:
 * loss[n] = mean_b( logsumexp(z_b) - z_b[label] ),
 * dz = (softmax(z) - onehot)/B.  Double arithmetic, rounded once. */
void orc_softmax_ce(int nodes, int B, int K, const float *logits, const int32_t *labels,
                    float *loss, float *dlogits)
{
    for (int n = 0; n < nodes; ++n) {
        double total = 0.0;
        for (int b = 0; b < B; ++b) {
            const float *z = logits + ((i64)n * B + b) * K;
            float *dz = dlogits + ((i64)n * B + b) * K;
            double zmax = z[0];
            for (int k = 1; k < K; ++k) if (z[k] > zmax) zmax = z[k];
            double den = 0.0;
            for (int k = 0; k < K; ++k) den += exp((double)z[k] - zmax);
            int lab = labels[(i64)n * B + b];
            total += log(den) + zmax - (double)z[lab];
            for (int k = 0; k < K; ++k) {
                double p = exp((double)z[k] - zmax) / den;
                dz[k] = (float)((p - (k == lab ? 1.0 : 0.0)) / (double)B);
            }
        }
        loss[n] = (float)(total / (double)B);
    }
}

/* Column sums over the batch (bias gradient of the linear layer):
 * out[n][c] = sum_b x[n][b][c], double accumulate, rounded once. */
void orc_colsum(int nodes, int B, int C, const float *x, float *out)
{
    for (int n = 0; n < nodes; ++n)
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            for (int b = 0; b < B; ++b) s += (double)x[((i64)n * B + b) * C + c];
            out[(i64)n * C + c] = (float)s;
        }
}
