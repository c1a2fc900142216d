// Tensor-core engine of the quantized contractions: implicit-GEMM convolution
// (stride 1) and GEMM on tcgen05.mma kind::i8 with TMA-staged operands, int32
// accumulators in TMEM and a fused dequantize epilogue.
//
// Data movement.  Activations stay NHWC int8 in HBM.  A TMA box of
// {16 channels, TW, TH, TB pixels} lands in shared memory as 128 rows of 16
// bytes, i.e. sixteen 8x16-byte core matrices of the no-swizzle canonical
// layout.  One such box is a "slice" (16 bytes of the channel dimension at one
// filter tap, shifted by the tap offset; out-of-image pixels are zero-filled by
// TMA, which is exact for symmetric int8).  The same shared-memory image serves
//   - as a K-major operand  (K = (tap, channel): forward and backward-data), and
//   - as an MN-major operand (K = pixels: backward-weight),
// only the descriptor's leading/stride offsets trade places.
//
// Kernels.  conv_pix_kernel: M = 128 output pixels, N = channels, K = taps x
// channels; persistent over tiles, double-buffered TMEM accumulator so the
// epilogue of tile i overlaps the MMAs of tile i+1.  conv_wgrad_kernel: M = (tap,
// input channel), N = output channels, K = pixels, split over CTAs with exact
// int32 atomics.  Warp roles: warp 0 issues TMA, warp 1 owns TMEM and issues the
// MMAs, warps 2-5 run the epilogue (one TMEM lane quarter each).
#include "qconv_internal.cuh"
#include "tc_common.cuh"

namespace lpdt {
namespace tc {

constexpr int kSliceBytes = 2048;     // 128 rows x 16 bytes
constexpr int kThreads = 192;

// A tile belongs to one "class" of M-space pixels.  Stride-1 problems have one
// class holding every filter tap.  The stride-2 backward-data problem splits the
// input pixels by the parity of (ih, iw): each parity class sees its own subset of
// taps and is a stride-1 problem on the error image.
constexpr int kMaxTaps = 64;
struct TapTable {
    int ntaps;
    signed char wtap[kMaxTaps];   // tap index in the weight tensor (r*S + s)
    signed char dh[kMaxTaps], dw[kMaxTaps];   // operand-A pixel offset of the tap
};
struct PixParams {
    int mode;                 // 0 forward, 1 backward-data
    int nodes, B, Hm, Wm;     // M-space grid of one class
    int Hout, Wout;           // full output image; output pixel = out_mul*m + class parity
    int out_mul, cmul;        // cmul scales tile origins into operand-A coordinates (forward stride)
    int ncls, cls_ph[4], cls_pw[4], cls_iters[4];
    TapTable tt[4];
    int Nc, Kc;               // N channels, K channels per tap
    int TB, TH, TW, tilesB, tilesH, tilesW, tilesN, BN;
    int S_slices, stages, tmem_cols;
    int w_rows_per_node;      // Cout: rows of the weight map per node
    float *Y; int32_t *Yacc;
    const float *s1, *s2, *bias; long long bias_stride;
    int32_t *dev_status;
};

struct SharedCtl {
    unsigned long long full[8], empty[8], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

__global__ void __launch_bounds__(kThreads, 1)
conv_pix_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapW,
                const PixParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    SharedCtl *ctl = reinterpret_cast<SharedCtl *>(smem);
    unsigned char *data = smem + 1024;
    const int stage_bytes = p.S_slices * (kSliceBytes + p.BN * 16);
    const int a_bytes = p.S_slices * kSliceBytes;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = p.nodes * p.tilesB * p.tilesH * p.tilesW * p.tilesN * p.ncls;

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.stages; ++i) { mbar_init(smem_u32(&ctl->full[i]), 1); mbar_init(smem_u32(&ctl->empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&ctl->tmem_full[i]), 1); mbar_init(smem_u32(&ctl->tmem_empty[i]), 4); }
        ctl->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&ctl->tmem_base), p.tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;
    const int cpt = p.Kc / 16;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&mapA); tma_prefetch_desc(&mapW);
            uint32_t g = 0;     // global stage counter
            for (int tile = blockIdx.x; tile < total_tiles && !ctl->abort_flag; tile += gridDim.x) {
                int t = tile;
                const int cls = t % p.ncls; t /= p.ncls;
                const int nt = t % p.tilesN; t /= p.tilesN;
                const int tw = t % p.tilesW; t /= p.tilesW;
                const int th = t % p.tilesH; t /= p.tilesH;
                const int tb = t % p.tilesB; const int node = t / p.tilesB;
                const int n0 = nt * p.BN, w0 = tw * p.TW * p.cmul, h0 = th * p.TH * p.cmul, b0 = tb * p.TB;
                const TapTable &tt = p.tt[cls];
                for (int it = 0; it < p.cls_iters[cls]; ++it, ++g) {
                    const int st = g % p.stages;
                    const uint32_t ph = (g / p.stages) & 1;
                    if (!mbar_wait(smem_u32(&ctl->empty[st]), ph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                    const uint32_t full = smem_u32(&ctl->full[st]);
                    mbar_expect_tx(full, stage_bytes);
                    const uint32_t a_st = smem_u32(data + (size_t)st * stage_bytes);
                    const uint32_t b_st = a_st + a_bytes;
                    for (int sl = 0; sl < p.S_slices; ++sl) {
                        const int kap = it * p.S_slices + sl;
                        const int ti = kap / cpt, chunk = kap % cpt;
                        int hc = -(1 << 20), wc = 0, tap = 1 << 20;   // phantom slice: boxes out of range -> zeros
                        if (ti < tt.ntaps) { hc = h0 + tt.dh[ti]; wc = w0 + tt.dw[ti]; tap = tt.wtap[ti]; }
                        tma_load_5d(a_st + sl * kSliceBytes, &mapA, full, chunk * 16, wc, hc, b0, node);
                        if (p.mode == 0) {
                            tma_load_3d(b_st + sl * p.BN * 16, &mapW, full, chunk * 16, tap,
                                        node * p.w_rows_per_node + n0);
                        } else {
                            for (int j = 0; j < p.BN / 16; ++j)
                                tma_load_3d(b_st + j * (p.S_slices * 256) + sl * 256, &mapW, full, n0 + j * 16, tap,
                                            node * p.w_rows_per_node + chunk * 16);
                        }
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = idesc_i8(128, p.BN, 0, p.mode == 0 ? 0 : 1);
            uint32_t g = 0, tcount = 0;
            for (int tile = blockIdx.x; tile < total_tiles && !ctl->abort_flag; tile += gridDim.x, ++tcount) {
                const int acc = tcount & 1;
                const uint32_t aph = (tcount >> 1) & 1;
                if (!mbar_wait(smem_u32(&ctl->tmem_empty[acc]), aph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * p.BN;
                bool ok = true;
                const int iters = p.cls_iters[tile % p.ncls];
                for (int it = 0; it < iters; ++it, ++g) {
                    const int st = g % p.stages;
                    const uint32_t ph = (g / p.stages) & 1;
                    if (!mbar_wait(smem_u32(&ctl->full[st]), ph, &ctl->abort_flag, p.dev_status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_st = smem_u32(data + (size_t)st * stage_bytes);
                    const uint32_t b_st = a_st + a_bytes;
                    for (int j = 0; j < p.S_slices / 2; ++j) {
                        const uint64_t ad = smem_desc(a_st + j * 2 * kSliceBytes, kSliceBytes, 128, 0);
                        const uint64_t bd = (p.mode == 0)
                            ? smem_desc(b_st + j * 2 * p.BN * 16, p.BN * 16, 128, 0)
                            : smem_desc(b_st + j * 512, 128, p.S_slices * 256, 0);
                        mma_i8(d_tmem, ad, bd, idesc, (it | j) != 0);
                    }
                    mma_commit(smem_u32(&ctl->empty[st]));
                }
                if (!ok) break;
                mma_commit(smem_u32(&ctl->tmem_full[acc]));
            }
        }
    } else {
        const int q = warp & 3;                       // TMEM lane quarter of this warp
        const int row = q * 32 + lane;                // tile row = pixel within the tile
        const int pw = row % p.TW, phh = (row / p.TW) % p.TH, pb = row / (p.TW * p.TH);
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < total_tiles && !ctl->abort_flag; tile += gridDim.x, ++tcount) {
            int t = tile;
            const int cls = t % p.ncls; t /= p.ncls;
            const int nt = t % p.tilesN; t /= p.tilesN;
            const int tw = t % p.tilesW; t /= p.tilesW;
            const int th = t % p.tilesH; t /= p.tilesH;
            const int tb = t % p.tilesB; const int node = t / p.tilesB;
            const int n0 = nt * p.BN;
            const int w = (tw * p.TW + pw) * p.out_mul + p.cls_pw[cls];
            const int h = (th * p.TH + phh) * p.out_mul + p.cls_ph[cls];
            const int b = tb * p.TB + pb;
            const bool valid = (w < p.Wout) && (h < p.Hout) && (b < p.B);
            const int acc = tcount & 1;
            const uint32_t aph = (tcount >> 1) & 1;
            if (!mbar_wait(smem_u32(&ctl->tmem_full[acc]), aph, &ctl->abort_flag, p.dev_status)) break;
            tc_fence_after();
            const long long pix = (((long long)node * p.B + b) * p.Hout + h) * p.Wout + w;
            const float sc = p.Y ? __fmul_rn(p.s1[node], p.s2[node]) : 0.f;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * p.BN;
            for (int c = 0; c < p.BN; c += 16) {
                uint32_t v[16];
                tmem_ld_32x16(t_row + c, v);
                tmem_ld_wait();
                if (valid && n0 + c < p.Nc) {
                    const long long o = pix * p.Nc + n0 + c;
                    if (p.Yacc) {
                        int4 *dst = reinterpret_cast<int4 *>(p.Yacc + o);
#pragma unroll
                        for (int k = 0; k < 4; ++k)
                            dst[k] = make_int4((int)v[4 * k], (int)v[4 * k + 1], (int)v[4 * k + 2], (int)v[4 * k + 3]);
                    }
                    if (p.Y) {
                        float f[16];
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            f[k] = __fmul_rn(__int2float_rn((int)v[k]), sc);
                            if (p.bias) f[k] = __fadd_rn(f[k], p.bias[(long long)node * p.bias_stride + n0 + c + k]);
                        }
                        float4 *dst = reinterpret_cast<float4 *>(p.Y + o);
#pragma unroll
                        for (int k = 0; k < 4; ++k) dst[k] = make_float4(f[4 * k], f[4 * k + 1], f[4 * k + 2], f[4 * k + 3]);
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, p.tmem_cols); }
}

// ----------------------------------------------------------------------------------------------
struct WgParams {
    int nodes, B, Ho, Wo, Cin, Cout, R, S, pad, taps, stride;
    int TB, TH, TW, tilesB, tilesH, tilesW;       // pixel tiles = K blocks
    int kblocks, splits, kb_per_split;
    int mgroups, ngroups, mtiles, slicesA, BNc, total_slices;
    int stages, tmem_cols;
    int32_t *acc_out; int32_t *dev_status;
};

__global__ void __launch_bounds__(kThreads, 1)
conv_wgrad_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapE,
                  const WgParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    SharedCtl *ctl = reinterpret_cast<SharedCtl *>(smem);
    unsigned char *data = smem + 1024;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int node = blockIdx.z;
    const int mg = blockIdx.y % p.mgroups, ng = blockIdx.y / p.mgroups;
    const int mu0 = mg * p.mtiles * 8;
    int nA = p.total_slices - mu0; if (nA > p.slicesA) nA = p.slicesA;
    const int n0 = ng * p.BNc, nE = p.BNc / 16;
    const int a_region = p.mtiles * 8 * kSliceBytes;
    const int stage_bytes = a_region + nE * kSliceBytes;
    const int kb0 = blockIdx.x * p.kb_per_split;
    int kb1 = kb0 + p.kb_per_split; if (kb1 > p.kblocks) kb1 = p.kblocks;
    const int cpt = p.Cin / 16;

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.stages; ++i) { mbar_init(smem_u32(&ctl->full[i]), 1); mbar_init(smem_u32(&ctl->empty[i]), 1); }
        mbar_init(smem_u32(&ctl->tmem_full[0]), 1);
        ctl->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&ctl->tmem_base), p.tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = ctl->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&mapX); tma_prefetch_desc(&mapE);
            uint32_t g = 0;
            for (int kb = kb0; kb < kb1; ++kb, ++g) {
                int t = kb;
                const int tw = t % p.tilesW; t /= p.tilesW;
                const int th = t % p.tilesH; const int tb = t / p.tilesH;
                const int w0 = tw * p.TW, h0 = th * p.TH, b0 = tb * p.TB;
                const int st = g % p.stages;
                const uint32_t ph = (g / p.stages) & 1;
                if (!mbar_wait(smem_u32(&ctl->empty[st]), ph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                const uint32_t full = smem_u32(&ctl->full[st]);
                mbar_expect_tx(full, (nA + nE) * kSliceBytes);
                const uint32_t a_st = smem_u32(data + (size_t)st * stage_bytes);
                const uint32_t e_st = a_st + a_region;
                for (int c = 0; c < nE; ++c)
                    tma_load_5d(e_st + c * kSliceBytes, &mapE, full, n0 + c * 16, w0, h0, b0, node);
                for (int i = 0; i < nA; ++i) {
                    const int mu = mu0 + i, tap = mu / cpt, chunk = mu % cpt;
                    const int r = tap / p.S, s = tap % p.S;
                    tma_load_5d(a_st + i * kSliceBytes, &mapX, full, chunk * 16, w0 * p.stride + s - p.pad,
                                h0 * p.stride + r - p.pad, b0, node);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = idesc_i8(128, p.BNc, 1, 1);
            uint32_t g = 0;
            bool ok = true;
            for (int kb = kb0; kb < kb1; ++kb, ++g) {
                const int st = g % p.stages;
                const uint32_t ph = (g / p.stages) & 1;
                if (!mbar_wait(smem_u32(&ctl->full[st]), ph, &ctl->abort_flag, p.dev_status)) { ok = false; break; }
                tc_fence_after();
                const uint32_t a_st = smem_u32(data + (size_t)st * stage_bytes);
                const uint32_t e_st = a_st + a_region;
                for (int t = 0; t < p.mtiles; ++t)
                    for (int kk = 0; kk < 4; ++kk) {
                        const uint64_t ad = smem_desc(a_st + t * 8 * kSliceBytes + kk * 512, 128, kSliceBytes, 0);
                        const uint64_t bd = smem_desc(e_st + kk * 512, 128, kSliceBytes, 0);
                        mma_i8(tmem_base + t * p.BNc, ad, bd, idesc, (g | (uint32_t)kk) != 0);
                    }
                mma_commit(smem_u32(&ctl->empty[st]));
            }
            if (ok) mma_commit(smem_u32(&ctl->tmem_full[0]));
        }
    } else if (kb1 > kb0) {
        const int q = warp & 3;
        const int row = q * 32 + lane;
        if (mbar_wait(smem_u32(&ctl->tmem_full[0]), 0, &ctl->abort_flag, p.dev_status)) {
            tc_fence_after();
            for (int t = 0; t < p.mtiles; ++t) {
                const int i = t * 8 + row / 16;                 // slice within this CTA
                const int mu = mu0 + i;
                const bool valid = (i < nA) && (mu < p.total_slices);
                const int tap = mu / cpt, ci = (mu % cpt) * 16 + (row & 15);
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + t * p.BNc;
                for (int c = 0; c < p.BNc; c += 16) {
                    uint32_t v[16];
                    tmem_ld_32x16(t_row + c, v);
                    tmem_ld_wait();
                    if (valid) {
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            const int co = n0 + c + k;
                            if ((int)v[k] != 0)
                                atomicAdd(p.acc_out + (((long long)node * p.Cout + co) * p.taps + tap) * p.Cin + ci, (int)v[k]);
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, p.tmem_cols); }
}

// ---------------------------------------------------------------------------------------------- host
static int pow2_at_least(int v) { int p = 32; while (p < v) p <<= 1; return p; }

// Pixel tile {TB, TH, TW} with TB*TH*TW = 128 covering a W x H image with least waste.
static void pick_tile(int H, int W, int *TB, int *TH, int *TW) {
    int bw = 1; long best = -1;
    for (int t = 1; t <= 128; t <<= 1) {
        long cover = (long)ceil_div(W, t) * t;
        if (best < 0 || cover <= best) { best = cover; bw = t; }
    }
    int bh = 1; best = -1;
    for (int t = 1; t <= 128 / bw; t <<= 1) {
        long cover = (long)ceil_div(H, t) * t;
        if (best < 0 || cover <= best) { best = cover; bh = t; }
    }
    *TW = bw; *TH = bh; *TB = 128 / (bw * bh);
}

// Activation map: box = one slice {16 channels, TW, TH, TB pixels}.  With estride 2 the
// box samples every second pixel (the traversal stride of the tensor map), which is how
// a stride-2 convolution reads its input.
static bool act_map(CUtensorMap *m, const int8_t *base, int nodes, int B, int H, int W, int C,
                    int TB, int TH, int TW, int estride = 1) {
    uint64_t dims[5] = {(uint64_t)C, (uint64_t)W, (uint64_t)H, (uint64_t)B, (uint64_t)nodes};
    uint64_t strides[4] = {(uint64_t)C, (uint64_t)W * C, (uint64_t)H * W * C, (uint64_t)B * H * W * C};
    uint32_t box[5] = {16, (uint32_t)(TW * estride), (uint32_t)(TH * estride), (uint32_t)TB, 1};
    uint32_t es[5] = {1, (uint32_t)estride, (uint32_t)estride, 1, 1};
    return make_map_u8(m, base, 5, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE, es);
}

static bool weight_map(CUtensorMap *m, const int8_t *base, int nodes, int Cout, int taps, int Cin, int box_rows) {
    uint64_t dims[3] = {(uint64_t)Cin, (uint64_t)taps, (uint64_t)nodes * Cout};
    uint64_t strides[2] = {(uint64_t)Cin, (uint64_t)taps * Cin};
    uint32_t box[3] = {16, 1, (uint32_t)box_rows};
    return make_map_u8(m, base, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE);
}

constexpr int kSmemBudget = 200 * 1024;
constexpr int kMinSmem = 120 * 1024;      // keeps one CTA per SM, so TMEM allocation never waits

bool tc_supported(const lpdt_conv_desc &d) {
    if (d.stride != 1 && d.stride != 2) return false;
    if (d.Cin % 16 || d.Cout % 16) return false;
    if (d.R * d.S > kMaxTaps || d.R > 100 || d.S > 100 || d.pad > 100) return false;
    if (!encode_tiled_fn()) return false;
    return true;
}

static int largest_div16(int C, int cap) {      // largest multiple of 16 dividing C, <= cap
    for (int v = cap - cap % 16; v >= 16; v -= 16) if (C % v == 0) return v;
    return 16;
}

lpdt_status tc_pix(const lpdt_conv_desc &d, int mode, const int8_t *A, const float *s1, const int8_t *Wq,
                   const float *s2, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                   int32_t *dev_status, cudaStream_t st) {
    const int Ho = conv_out(d.H, d.pad, d.R, d.stride), Wo = conv_out(d.W, d.pad, d.S, d.stride);
    PixParams p = {};
    p.mode = mode; p.nodes = d.nodes; p.B = d.B;
    p.Nc = mode == 0 ? d.Cout : d.Cin; p.Kc = mode == 0 ? d.Cin : d.Cout;
    p.out_mul = 1; p.cmul = 1; p.ncls = 1;
    if (mode == 0) {
        // output pixel (oh, ow) reads input (oh*stride + r - pad, ow*stride + s - pad)
        p.Hout = Ho; p.Wout = Wo; p.Hm = Ho; p.Wm = Wo; p.cmul = d.stride;
        TapTable &tt = p.tt[0];
        for (int r = 0; r < d.R; ++r)
            for (int s = 0; s < d.S; ++s) {
                tt.wtap[tt.ntaps] = (signed char)(r * d.S + s);
                tt.dh[tt.ntaps] = (signed char)(r - d.pad); tt.dw[tt.ntaps] = (signed char)(s - d.pad);
                ++tt.ntaps;
            }
    } else {
        // input pixel (ih, iw) = (stride*m + ph, ...) reads error pixel ((ih + pad - r)/stride, ...) for
        // the taps whose offset is divisible by the stride
        p.Hout = d.H; p.Wout = d.W; p.out_mul = d.stride;
        p.Hm = (int)ceil_div(d.H, d.stride); p.Wm = (int)ceil_div(d.W, d.stride);
        p.ncls = d.stride * d.stride;
        for (int c = 0; c < p.ncls; ++c) {
            const int ph = c / d.stride, pw = c % d.stride;
            p.cls_ph[c] = ph; p.cls_pw[c] = pw;
            TapTable &tt = p.tt[c];
            for (int r = 0; r < d.R; ++r) {
                if ((ph + d.pad - r) % d.stride) continue;
                for (int s = 0; s < d.S; ++s) {
                    if ((pw + d.pad - s) % d.stride) continue;
                    tt.wtap[tt.ntaps] = (signed char)(r * d.S + s);
                    // floor division; ph + pad - r may be negative
                    const int nh = ph + d.pad - r, nw = pw + d.pad - s;
                    tt.dh[tt.ntaps] = (signed char)(nh >= 0 ? nh / d.stride : -((-nh) / d.stride));
                    tt.dw[tt.ntaps] = (signed char)(nw >= 0 ? nw / d.stride : -((-nw) / d.stride));
                    ++tt.ntaps;
                }
            }
        }
    }
    pick_tile(p.Hm, p.Wm, &p.TB, &p.TH, &p.TW);
    p.tilesB = (int)ceil_div(d.B, p.TB); p.tilesH = (int)ceil_div(p.Hm, p.TH); p.tilesW = (int)ceil_div(p.Wm, p.TW);
    p.BN = largest_div16(p.Nc, 256);
    p.tilesN = p.Nc / p.BN;
    const int cpt = p.Kc / 16;
    // slices per stage: even, <= 16, stage <= 48 KB, least padded work over the classes
    int S = 2; long best = -1;
    for (int s = 2; s <= 16; s += 2) {
        if (s * (kSliceBytes + p.BN * 16) > 48 * 1024) break;
        long work = 0;
        for (int c = 0; c < p.ncls; ++c) work += ceil_div((long)p.tt[c].ntaps * cpt, s) * s;
        if (best < 0 || work <= best) { best = work; S = s; }
    }
    p.S_slices = S;
    for (int c = 0; c < p.ncls; ++c) {
        p.cls_iters[c] = (int)ceil_div((long)p.tt[c].ntaps * cpt, S);
        if (p.cls_iters[c] < 1) p.cls_iters[c] = 1;      // a class without taps still writes zeros
    }
    const int stage_bytes = S * (kSliceBytes + p.BN * 16);
    p.stages = (kSmemBudget - 1024) / stage_bytes;
    if (p.stages > 8) p.stages = 8;
    if (p.stages < 2) return LPDT_ERR_UNSUPPORTED;
    p.tmem_cols = pow2_at_least(2 * p.BN);
    p.w_rows_per_node = d.Cout;
    p.Y = Y; p.Yacc = Yacc; p.s1 = s1; p.s2 = s2; p.bias = bias; p.bias_stride = bias_stride;
    p.dev_status = dev_status;
    CUtensorMap mA, mW;
    // operand A: activations (fwd: image H x W, Cin, sampled with the conv stride) or errors
    // (bwd-data: image Ho x Wo, Cout, dense)
    if (mode == 0) {
        if (p.TW * d.stride > 256 || p.TH * d.stride > 256) return LPDT_ERR_UNSUPPORTED;
        if (!act_map(&mA, A, d.nodes, d.B, d.H, d.W, p.Kc, p.TB, p.TH, p.TW, d.stride)) return LPDT_ERR_CUDA;
    } else {
        if (!act_map(&mA, A, d.nodes, d.B, Ho, Wo, p.Kc, p.TB, p.TH, p.TW, 1)) return LPDT_ERR_CUDA;
    }
    if (!weight_map(&mW, Wq, d.nodes, d.Cout, d.R * d.S, d.Cin, mode == 0 ? p.BN : 16)) return LPDT_ERR_CUDA;
    size_t smem = 1024 + (size_t)p.stages * stage_bytes;
    if (smem < kMinSmem) smem = kMinSmem;
    static bool attr = false;
    if (!attr) {
        LPDT_CUDA(cudaFuncSetAttribute(conv_pix_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr = true;
    }
    const long long tiles = (long long)p.nodes * p.tilesB * p.tilesH * p.tilesW * p.tilesN * p.ncls;
    const int grid = (int)(tiles < kNumSMs ? tiles : kNumSMs);
    conv_pix_kernel<<<grid, kThreads, smem, st>>>(mA, mW, p);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

lpdt_status tc_wgrad(const lpdt_conv_desc &d, const int8_t *E, const int8_t *A, int32_t *acc_out,
                     int32_t *dev_status, cudaStream_t st) {
    const int Ho = conv_out(d.H, d.pad, d.R, d.stride), Wo = conv_out(d.W, d.pad, d.S, d.stride);
    WgParams p = {};
    p.nodes = d.nodes; p.B = d.B; p.Ho = Ho; p.Wo = Wo; p.Cin = d.Cin; p.Cout = d.Cout;
    p.R = d.R; p.S = d.S; p.pad = d.pad; p.taps = d.R * d.S; p.stride = d.stride;
    pick_tile(Ho, Wo, &p.TB, &p.TH, &p.TW);
    p.tilesB = (int)ceil_div(d.B, p.TB); p.tilesH = (int)ceil_div(Ho, p.TH); p.tilesW = (int)ceil_div(Wo, p.TW);
    p.kblocks = p.tilesB * p.tilesH * p.tilesW;
    p.BNc = largest_div16(d.Cout, 256);
    p.ngroups = d.Cout / p.BNc;
    p.total_slices = p.taps * (d.Cin / 16);
    const int all_tiles = (int)ceil_div(p.total_slices, 8);
    int mt = 512 / p.BNc;                                   // accumulators that fit in TMEM
    int mt_smem = ((96 * 1024) / kSliceBytes - p.BNc / 16) / 8;   // stage <= 96 KB -> at least two stages
    if (mt > mt_smem) mt = mt_smem;
    if (mt > all_tiles) mt = all_tiles;
    if (mt < 1) return LPDT_ERR_UNSUPPORTED;
    p.mtiles = mt;
    p.mgroups = (int)ceil_div(all_tiles, mt);
    p.slicesA = mt * 8;
    const int stage_bytes = (mt * 8 + p.BNc / 16) * kSliceBytes;
    p.stages = (kSmemBudget - 1024) / stage_bytes;
    if (p.stages > 8) p.stages = 8;
    if (p.stages < 2) return LPDT_ERR_UNSUPPORTED;
    p.tmem_cols = pow2_at_least(mt * p.BNc);
    if (p.tmem_cols > 512) return LPDT_ERR_UNSUPPORTED;
    long long ctas_fixed = (long long)d.nodes * p.mgroups * p.ngroups;
    int splits = (int)ceil_div(2 * kNumSMs, ctas_fixed);
    if (splits > p.kblocks) splits = p.kblocks;
    if (splits < 1) splits = 1;
    p.kb_per_split = (int)ceil_div(p.kblocks, splits);
    p.splits = (int)ceil_div(p.kblocks, p.kb_per_split);
    p.acc_out = acc_out; p.dev_status = dev_status;
    CUtensorMap mX, mE;
    if (p.TW * d.stride > 256 || p.TH * d.stride > 256) return LPDT_ERR_UNSUPPORTED;
    if (!act_map(&mX, A, d.nodes, d.B, d.H, d.W, d.Cin, p.TB, p.TH, p.TW, d.stride)) return LPDT_ERR_CUDA;
    if (!act_map(&mE, E, d.nodes, d.B, Ho, Wo, d.Cout, p.TB, p.TH, p.TW)) return LPDT_ERR_CUDA;
    size_t smem = 1024 + (size_t)p.stages * stage_bytes + 16 * 1024;   // slack: descriptors of a partial M tile read past it
    if (smem < kMinSmem) smem = kMinSmem;
    if (smem > 227 * 1024) { p.stages -= 1; smem = 1024 + (size_t)p.stages * stage_bytes + 16 * 1024; }
    if (p.stages < 2 || smem > 227 * 1024) return LPDT_ERR_UNSUPPORTED;
    static bool attr = false;
    if (!attr) {
        LPDT_CUDA(cudaFuncSetAttribute(conv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr = true;
    }
    conv_wgrad_kernel<<<dim3(p.splits, p.mgroups * p.ngroups, d.nodes), kThreads, smem, st>>>(mX, mE, p);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

}  // namespace tc
}  // namespace lpdt
