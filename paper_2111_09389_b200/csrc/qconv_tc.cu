// Tensor-core engine of the quantized contractions: implicit-GEMM convolution
// (stride 1 and 2) and GEMM on tcgen05.mma kind::i8 with TMA-staged operands,
// int32 accumulators in TMEM and a fused dequantize epilogue.
//
// Operand tiles.  Activations stay NHWC int8 in HBM.  A TMA box of
// {RB channel bytes, TW, TH, TB pixels} (TB*TH*TW = 128) lands in shared memory
// as 128 rows of RB bytes, RB = 128, 64, 32 or 16 chosen from the channel count.
// Rows of 32..128 bytes use the matching TMA/UMMA swizzle; rows of 16 bytes are
// the no-swizzle layout (sixteen contiguous 8x16-byte core matrices).  Each box is
// read at the tap's pixel offset; out-of-image pixels are zero-filled by TMA,
// which is exact for symmetric int8.  The same shared-memory image serves
//   - as a K-major operand  (K = (tap, channel): forward and backward-data), and
//   - as an MN-major operand (K = pixels: backward-weight);
// only the descriptor changes.  When C = 16 and the stride is 1, the channel and
// width dimensions are contiguous in memory and are fetched as one 256-byte row
// per 16 pixels instead of sixteen 16-byte rows.
//
// Kernels.  conv_pix_kernel: M = 128 output pixels, N = channels, K = taps x
// channels; each CTA walks a contiguous range of tiles with a double-buffered
// TMEM accumulator, so the epilogue of tile i overlaps the MMAs of tile i+1.
// conv_wgrad_kernel: M = (tap, input channel), N = output channels, K = pixels,
// split over CTAs with exact int32 atomics.  Warp roles: warp 0 issues TMA,
// warp 1 owns TMEM and issues the MMAs, the remaining warps run the epilogue
// (conv_wgrad_kernel: warps 2-5, one TMEM lane quarter each; conv_pix_kernel:
// warps 2-9, two per lane quarter taking alternate column chunks).  The pixel
// kernel's fp32 result leaves through shared memory and bulk tensor stores where
// its layout allows.  Every wait is bounded (tc_common.cuh).
#include <stdlib.h>
#include "qconv_internal.cuh"
#include "tc_common.cuh"

namespace lpdt {
namespace tc {

constexpr int kThreads = 192;
constexpr int kPixThreads = 320;      // pixel kernel: TMA warp, MMA warp, eight epilogue warps (two per TMEM lane quarter)
constexpr int kMaxTaps = 64;

// Row format of an operand tile: RB bytes per row and the UMMA layout code.
__host__ __device__ inline uint32_t layout_code(int RB) { return RB == 128 ? 2u : RB == 64 ? 4u : RB == 32 ? 6u : 0u; }
static int row_bytes_for(int C) { return C % 128 == 0 ? 128 : C % 64 == 0 ? 64 : C % 32 == 0 ? 32 : 16; }
static CUtensorMapSwizzle swizzle_for(int RB) {
    return RB == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : RB == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
         : RB == 32 ? CU_TENSOR_MAP_SWIZZLE_32B : CU_TENSOR_MAP_SWIZZLE_NONE;
}

// A tile belongs to one "class" of M-space pixels.  Stride-1 problems have one
// class holding every filter tap.  The stride-2 backward-data problem splits the
// input pixels by the parity of (ih, iw): each parity class sees its own subset of
// taps and is a stride-1 problem on the error image.
struct TapTable {
    int ntaps;
    signed char wtap[kMaxTaps];               // tap index in the weight tensor (r*S + s)
    signed char dh[kMaxTaps], dw[kMaxTaps];   // operand-A pixel offset of the tap
};

struct PixParams {
    int mode;                 // 0 forward, 1 backward-data
    int uns;                  // operands are unsigned 8-bit codes
    int nodes, B, Hm, Wm;     // M-space grid of one class
    int Hout, Wout;           // full output image; output pixel = out_mul*m + class parity
    int out_mul, cmul;        // cmul scales tile origins into operand-A coordinates (forward stride)
    int ncls, cls_ph[4], cls_pw[4], cls_iters[4];
    TapTable tt[4];
    int Nc, Kc;               // N channels, K channels per tap
    int RBa, RBn;             // row bytes of operand A (K side) and, backward-data, of the N side
    int merged;               // operand A fetched through the merged (channel, width) map
    int raster;               // 1: CTAs take tiles round-robin in a blocked M x N order (long-K tiles, L2 reuse)
    int TB, TH, TW, tilesB, tilesH, tilesW, tilesN, BN;
    int U, stages, tmem_cols; // K units (one A box each) per stage
    int w_rows_per_node;      // Cout: rows of the weight map per node
    float *Y; int32_t *Yacc;
    const float *s1, *s2, *bias; long long bias_stride;
    const float *addend;      // nullable: fp32 tensor of the result's shape, added to the dequantized result
    int32_t *dev_status;
    // fp32 result through shared memory and bulk tensor stores: every epilogue warp stages its 32 pixels x 32
    // channels (128-byte rows, 128-byte swizzle) and stores them as one box {32 channels, bw, bh, bb pixels}
    int tma_out, out_off;     // out_off: byte offset of the staging area in shared memory (1024-byte aligned)
    int bw, bh;               // the warp's sub-box of the pixel tile: bw x bh x 32/(bw*bh) pixels
    // Forward product on affine (zero-point) operands, corrected in the epilogue (null asum: plain product):
    //   sum (qa - zA)(qw - zW) = acc - zW * ra - zA * rw + cnt * zA * zW   over the taps inside the image,
    // ra = the per-pixel channel sums of the input (asum [nodes][B][H][W]) over those taps, rw = the weights'
    // channel sums over them, from a prefix table over the filter taps (wpre [nodes][R+1][S+1][Cout]; the taps
    // inside the image form a rectangle of the filter), cnt = taps inside x Cin.  All modulo 2^32.
    const int32_t *asum, *wpre, *zA, *zW;
    int aH, aW, aR, aS, apad, astride, aCin;
};

// Zero-point terms of one output pixel: what does not depend on the output channel (fixed) and the corners of
// the pixel's tap rectangle in the prefix table.
struct AffinePixel { unsigned fixed, za; int c11, c01, c10, c00; bool interior; };
__device__ __forceinline__ AffinePixel affine_pixel(const PixParams &p, int node, int b, int oh, int ow) {
    int r_lo = p.apad - oh * p.astride; if (r_lo < 0) r_lo = 0;
    int r_hi = p.aH + p.apad - oh * p.astride; if (r_hi > p.aR) r_hi = p.aR;
    int s_lo = p.apad - ow * p.astride; if (s_lo < 0) s_lo = 0;
    int s_hi = p.aW + p.apad - ow * p.astride; if (s_hi > p.aS) s_hi = p.aS;
    if (r_hi < r_lo) r_hi = r_lo;
    if (s_hi < s_lo) s_hi = s_lo;
    const long long nb = (long long)node * p.B + b;
    unsigned ra = 0;
    for (int r = r_lo; r < r_hi; ++r)
        for (int s = s_lo; s < s_hi; ++s)
            ra += (unsigned)__ldg(p.asum + (nb * p.aH + oh * p.astride + r - p.apad) * p.aW + ow * p.astride + s - p.apad);
    AffinePixel a;
    const unsigned za = (unsigned)p.zA[node], zw = (unsigned)p.zW[node];
    a.za = za;
    a.fixed = (unsigned)((r_hi - r_lo) * (s_hi - s_lo) * p.aCin) * za * zw - zw * ra;
    const int PS = p.aS + 1;
    a.c11 = (r_hi * PS + s_hi) * p.Nc; a.c01 = (r_lo * PS + s_hi) * p.Nc;
    a.c10 = (r_hi * PS + s_lo) * p.Nc; a.c00 = (r_lo * PS + s_lo) * p.Nc;
    a.interior = r_lo == 0 && s_lo == 0;          // the three other corners are zero
    return a;
}
// acc[k] += fixed - za * rw[channel c0 + k], k < NV (NV a multiple of 4, c0 a multiple of 4)
template <int NV>
__device__ __forceinline__ void affine_apply(const PixParams &p, const AffinePixel &a, int node, int c0, uint32_t (&v)[NV]) {
    const int32_t *t = p.wpre + (long long)node * (p.aR + 1) * (p.aS + 1) * p.Nc + c0;
#pragma unroll
    for (int k = 0; k < NV; k += 4) {
        const int4 q11 = __ldg(reinterpret_cast<const int4 *>(t + a.c11 + k));
        unsigned rw[4] = {(unsigned)q11.x, (unsigned)q11.y, (unsigned)q11.z, (unsigned)q11.w};
        if (!a.interior) {
            const int4 q01 = __ldg(reinterpret_cast<const int4 *>(t + a.c01 + k));
            const int4 q10 = __ldg(reinterpret_cast<const int4 *>(t + a.c10 + k));
            const int4 q00 = __ldg(reinterpret_cast<const int4 *>(t + a.c00 + k));
            rw[0] += (unsigned)q00.x - (unsigned)q01.x - (unsigned)q10.x; rw[1] += (unsigned)q00.y - (unsigned)q01.y - (unsigned)q10.y;
            rw[2] += (unsigned)q00.z - (unsigned)q01.z - (unsigned)q10.z; rw[3] += (unsigned)q00.w - (unsigned)q01.w - (unsigned)q10.w;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) v[k + j] = v[k + j] + a.fixed - a.za * rw[j];
    }
}

struct SharedCtl {
    unsigned long long full[8], empty[8], tmem_full[2], tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};

struct TileCoord { int cls, tw, th, tb, nt, node; };
// tile order: node, N tile, batch tile, row tile, column tile, class (fastest).  A CTA walks
// consecutive tiles, so the coordinate is decoded once and then advanced like an odometer
// (the single-thread roles are instruction-bound: no divisions in their loops).
__device__ __forceinline__ TileCoord decode_tile(const PixParams &p, int tile) {
    TileCoord c; int t = tile;
    c.cls = t % p.ncls; t /= p.ncls;
    c.tw = t % p.tilesW; t /= p.tilesW;
    c.th = t % p.tilesH; t /= p.tilesH;
    c.tb = t % p.tilesB; t /= p.tilesB;
    c.nt = t % p.tilesN; c.node = t / p.tilesN;
    return c;
}
__device__ __forceinline__ void next_tile(const PixParams &p, TileCoord &c) {
    if (++c.cls < p.ncls) return; c.cls = 0;
    if (++c.tw < p.tilesW) return; c.tw = 0;
    if (++c.th < p.tilesH) return; c.th = 0;
    if (++c.tb < p.tilesB) return; c.tb = 0;
    if (++c.nt < p.tilesN) return; c.nt = 0;
    ++c.node;
}

// Blocked order for long-K tiles: groups of kRasterM M tiles sweep all N tiles, so the tiles in flight
// at any moment (consecutive indices, one per CTA) share a few operand panels that stay in L2.
constexpr int kRasterM = 16;
__device__ __forceinline__ TileCoord decode_raster(const PixParams &p, int tile) {
    const int mtiles = p.nodes * p.tilesB * p.tilesH * p.tilesW;
    const int per_group = kRasterM * p.tilesN;
    const int mg = tile / per_group, rem = tile - mg * per_group;
    int gsize = mtiles - mg * kRasterM; if (gsize > kRasterM) gsize = kRasterM;
    TileCoord c; c.cls = 0;
    c.nt = rem / gsize;
    int m = mg * kRasterM + (rem - c.nt * gsize);
    c.tw = m % p.tilesW; m /= p.tilesW;
    c.th = m % p.tilesH; m /= p.tilesH;
    c.tb = m % p.tilesB; c.node = m / p.tilesB;
    return c;
}

// MINB = 2: the register budget of two resident CTAs per SM, for layers whose K loop is a few stages long: a
// CTA's fill and drain (first operand boxes, the last tile's epilogue) then overlap its neighbour's main loop.
template <int MINB>
__global__ void __launch_bounds__(kPixThreads, MINB)
conv_pix_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapW,
                const __grid_constant__ CUtensorMap mapY, const PixParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    SharedCtl *ctl = reinterpret_cast<SharedCtl *>(smem);
    unsigned char *data = smem + 1024;
    const int a_unit = 128 * p.RBa;                        // bytes of one A box
    const int b_unit = p.BN * p.RBa;                       // weight bytes that go with it
    const int a_bytes = p.U * a_unit;
    const int stage_bytes = p.U * (a_unit + b_unit);
    // warp index (and below the TMEM base) go through a shuffle so that the compiler knows they are
    // warp-uniform and keeps the single-issuer role loops on the uniform datapath
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const long long total_tiles = (long long)p.nodes * p.tilesN * p.tilesB * p.tilesH * p.tilesW * p.ncls;
    const int tile_lo = p.raster ? (int)blockIdx.x : (int)(total_tiles * blockIdx.x / gridDim.x);
    const int tile_hi = p.raster ? (int)total_tiles : (int)(total_tiles * (blockIdx.x + 1) / gridDim.x);
    const int tile_step = p.raster ? (int)gridDim.x : 1;

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.stages; ++i) { mbar_init(smem_u32(&ctl->full[i]), 1); mbar_init(smem_u32(&ctl->empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&ctl->tmem_full[i]), 1); mbar_init(smem_u32(&ctl->tmem_empty[i]), 8); }
        ctl->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&ctl->tmem_base), p.tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_enter();          // nothing above touches global memory
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, ctl->tmem_base, 0);
    const int cpt = p.Kc / p.RBa;          // A boxes per tap

    if (warp == 0) {
        {
            if (elect_one()) { tma_prefetch_desc(&mapA); tma_prefetch_desc(&mapW); }
            uint32_t g = 0;     // running stage counter
            int st = 0; uint32_t ph = 0;
            TileCoord c = decode_tile(p, p.raster ? 0 : tile_lo);
            const int nj = p.BN / p.RBn, bj_stride = p.U * p.RBa * p.RBn, bu_stride = p.RBa * p.RBn;
            for (int tile = tile_lo; tile < tile_hi && !ctl->abort_flag; tile += tile_step) {
                if (p.raster) c = decode_raster(p, tile); else if (tile != tile_lo) next_tile(p, c);
                const int n0 = c.nt * p.BN, w0 = c.tw * p.TW * p.cmul, h0 = c.th * p.TH * p.cmul, b0 = c.tb * p.TB;
                const int wrow = c.node * p.w_rows_per_node;
                const TapTable &tt = p.tt[c.cls];
                int ti = 0, chunk = 0;                      // running (tap, channel chunk) of the next unit
                for (int it = 0; it < p.cls_iters[c.cls]; ++it, ++g) {
                    if (!mbar_wait(smem_u32(&ctl->empty[st]), ph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                    const uint32_t full = smem_u32(&ctl->full[st]);
                    const bool leader = elect_one();        // the whole warp walks the loop, one lane issues
                    if (leader) mbar_expect_tx(full, stage_bytes);
                    uint32_t a_dst = smem_u32(data + (size_t)st * stage_bytes);
                    uint32_t b_dst = a_dst + a_bytes;
                    for (int u = 0; u < p.U; ++u) {
                        int hc = -(1 << 20), wc = 0, tap = 1 << 20;   // phantom unit: boxes out of range -> zeros
                        if (ti < tt.ntaps) { hc = h0 + tt.dh[ti]; wc = w0 + tt.dw[ti]; tap = tt.wtap[ti]; }
                        if (leader) {
                            if (p.merged) tma_load_4d(a_dst, &mapA, full, wc * 16, hc, b0, c.node);
                            else tma_load_5d(a_dst, &mapA, full, chunk * p.RBa, wc, hc, b0, c.node);
                            if (p.mode == 0) {
                                tma_load_3d(b_dst, &mapW, full, chunk * p.RBa, tap, wrow + n0);
                            } else {
                                // N side in chunks of RBn bytes; this unit's RBa weight rows go at row u*RBa of each chunk
                                for (int j = 0; j < nj; ++j)
                                    tma_load_3d(b_dst + j * bj_stride, &mapW, full, n0 + j * p.RBn, tap,
                                                wrow + chunk * p.RBa);
                            }
                        }
                        b_dst += (p.mode == 0) ? b_unit : bu_stride;
                        a_dst += a_unit;
                        if (++chunk == cpt) { chunk = 0; ++ti; }
                    }
                    __syncwarp();
                    if (++st == p.stages) { st = 0; ph ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        {
            const uint32_t idesc = idesc_i8(128, p.BN, 0, p.mode == 0 ? 0 : 1, p.uns);
            // Descriptor templates (start address 0); the loop only adds address increments.
            const uint64_t a_tpl = (p.RBa == 16) ? smem_desc(0, a_unit, 128, 0)
                                                 : smem_desc(0, 16, 8 * p.RBa, layout_code(p.RBa));
            uint64_t b_tpl;
            if (p.mode == 0) b_tpl = (p.RBa == 16) ? smem_desc(0, b_unit, 128, 0) : smem_desc(0, 16, 8 * p.RBa, layout_code(p.RBa));
            else b_tpl = (p.RBn == 16) ? smem_desc(0, 128, p.U * p.RBa * 16, 0)
                                       : smem_desc(0, p.U * p.RBa * p.RBn, 8 * p.RBn, layout_code(p.RBn));
            // per-MMA (32 K bytes) and per-unit address steps, in 16-byte units
            const int n_units = (p.RBa == 16) ? p.U / 2 : p.U;
            const int steps = (p.RBa == 16) ? 1 : p.RBa / 32;
            const uint32_t a_step = 2, a_unit_step = (p.RBa == 16) ? (2 * a_unit) >> 4 : (a_unit - p.RBa) >> 4;
            uint32_t b_step, b_unit_step;
            if (p.mode == 0) { b_step = 2; b_unit_step = (p.RBa == 16) ? (2 * b_unit) >> 4 : (b_unit - p.RBa) >> 4; }
            else { b_step = (32 * p.RBn) >> 4; b_unit_step = (p.RBa == 16) ? b_step : 0; }
            uint32_t g = 0, tcount = 0;
            int st = 0; uint32_t ph = 0;
            int cls = tile_lo % p.ncls;
            for (int tile = tile_lo; tile < tile_hi && !ctl->abort_flag; tile += tile_step, ++tcount) {
                const int acc = tcount & 1;
                const uint32_t aph = (tcount >> 1) & 1;
                if (!mbar_wait(smem_u32(&ctl->tmem_empty[acc]), aph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * p.BN;
                bool ok = true;
                const int iters = p.cls_iters[cls];
                if (++cls == p.ncls) cls = 0;
                uint32_t accum = 0;
                for (int it = 0; it < iters; ++it, ++g) {
                    if (!mbar_wait(smem_u32(&ctl->full[st]), ph, &ctl->abort_flag, p.dev_status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_st = smem_u32(data + (size_t)st * stage_bytes);
                    if (elect_one()) {
                        uint32_t a_lo = a_st >> 4, b_lo = (a_st + a_bytes) >> 4, af = accum;
                        for (int u = 0; u < n_units; ++u) {
                            for (int k = 0; k < steps; ++k) {
                                mma_i8(d_tmem, a_tpl | (a_lo & 0x3FFFu), b_tpl | (b_lo & 0x3FFFu), idesc, af);
                                af = 1;
                                a_lo += a_step; b_lo += b_step;
                            }
                            if (p.RBa == 16) { a_lo += a_unit_step - a_step; b_lo += b_unit_step - b_step; }
                            else { a_lo += a_unit_step; b_lo += b_unit_step; }
                        }
                        mma_commit(smem_u32(&ctl->empty[st]));
                        if (it == iters - 1) mma_commit(smem_u32(&ctl->tmem_full[acc]));
                    }
                    __syncwarp();
                    accum = 1;
                    if (++st == p.stages) { st = 0; ph ^= 1; }
                }
                if (!ok) break;
            }
        }
    } else {
        const int q = warp & 3;                       // TMEM lane quarter of this warp
        const int row = q * 32 + lane;                // tile row = pixel within the tile
        const int pw = row % p.TW, phh = (row / p.TW) % p.TH, pb = row / (p.TW * p.TH);
        uint32_t tcount = 0;
        TileCoord c = decode_tile(p, p.raster ? 0 : tile_lo);
        int sc_node = -1; float sc = 0.f;
        // Two warps share a TMEM lane quarter and take alternate column chunks of its 32 pixels.
        const int half = (warp - 2) >> 2;
        // bulk-store path: this warp's 4 KB staging buffer and the origin of its 32 pixels inside the tile
        unsigned char *buf = smem + p.out_off + (warp - 2) * 4096;
        const int r0 = q * 32;
        const int box_w0 = r0 % p.TW, box_h0 = (r0 / p.TW) % p.TH, box_b0 = r0 / (p.TW * p.TH);
        if (p.tma_out && lane == 0) tma_prefetch_desc(&mapY);
        for (int tile = tile_lo; tile < tile_hi && !ctl->abort_flag; tile += tile_step, ++tcount) {
            if (p.raster) c = decode_raster(p, tile); else if (tile != tile_lo) next_tile(p, c);
            const int n0 = c.nt * p.BN;
            const int w = (c.tw * p.TW + pw) * p.out_mul + p.cls_pw[c.cls];
            const int h = (c.th * p.TH + phh) * p.out_mul + p.cls_ph[c.cls];
            const int b = c.tb * p.TB + pb;
            const bool valid = (w < p.Wout) && (h < p.Hout) && (b < p.B);
            if (p.Y && c.node != sc_node) { sc_node = c.node; sc = __fmul_rn(p.s1[c.node], p.s2[c.node]); }
            const int acc = tcount & 1;
            const uint32_t aph = (tcount >> 1) & 1;
            if (!mbar_wait(smem_u32(&ctl->tmem_full[acc]), aph, &ctl->abort_flag, p.dev_status)) break;
            tc_fence_after();
            const long long pix = (((long long)c.node * p.B + b) * p.Hout + h) * p.Wout + w;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * p.BN;
            AffinePixel aff = {};
            if (p.asum && valid) aff = affine_pixel(p, c.node, b, h, w);
            if (p.tma_out) {
                // 32 channels at a time: accumulators -> fp32 -> this warp's staging buffer (one 128-byte row per
                // lane, 16-byte pieces XOR-swizzled by the row so that the lanes spread over all banks, which is
                // also the layout the store's box expects) -> one bulk tensor store.  Box parts outside the
                // image are not written.  The next chunk's accumulators are fetched while this one is converted,
                // and the buffer is rewritten only after the previous store has read it.
                const uint32_t sw = (uint32_t)(lane & 7);
                uint32_t v[32];
                int cc = half * 32;
                bool have = cc < p.BN;
                if (have) tmem_ld_32x32(t_row + cc, v);
                while (have) {
                    tmem_ld_wait();
                    if (p.asum && valid) affine_apply<32>(p, aff, c.node, n0 + cc, v);
                    float f[32];
#pragma unroll
                    for (int k = 0; k < 32; ++k) f[k] = __fmul_rn(__int2float_rn((int)v[k]), sc);
                    const int ncc = cc + 64;
                    const bool more = ncc < p.BN;
                    if (more) tmem_ld_32x32(t_row + ncc, v);
                    if (p.bias) {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            f[k] = __fadd_rn(f[k], p.bias[(long long)c.node * p.bias_stride + n0 + cc + k]);
                    }
                    if (p.addend && valid) {
                        const float4 *ad = reinterpret_cast<const float4 *>(p.addend + pix * p.Nc + n0 + cc);
#pragma unroll
                        for (int k = 0; k < 8; ++k) {
                            const float4 a4 = ad[k];
                            f[4 * k] = __fadd_rn(f[4 * k], a4.x); f[4 * k + 1] = __fadd_rn(f[4 * k + 1], a4.y);
                            f[4 * k + 2] = __fadd_rn(f[4 * k + 2], a4.z); f[4 * k + 3] = __fadd_rn(f[4 * k + 3], a4.w);
                        }
                    }
                    if (lane == 0) tma_store_wait_read<0>();
                    __syncwarp();
                    float4 *grow = reinterpret_cast<float4 *>(buf + lane * 128);
#pragma unroll
                    for (int k = 0; k < 8; ++k)
                        grow[(uint32_t)k ^ sw] = make_float4(f[4 * k], f[4 * k + 1], f[4 * k + 2], f[4 * k + 3]);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_5d(&mapY, smem_u32(buf), n0 + cc, c.tw * p.TW + box_w0, c.th * p.TH + box_h0,
                                     c.tb * p.TB + box_b0, c.node);
                        tma_store_commit();
                    }
                    cc = ncc; have = more;
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
                continue;
            }
            for (int cc = half * 16; cc < p.BN; cc += 32) {
                uint32_t v[16];
                tmem_ld_32x16(t_row + cc, v);
                tmem_ld_wait();
                if (valid) {
                    const long long o = pix * p.Nc + n0 + cc;
                    if (p.asum) affine_apply<16>(p, aff, c.node, n0 + cc, v);
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
                            if (p.bias) f[k] = __fadd_rn(f[k], p.bias[(long long)c.node * p.bias_stride + n0 + cc + k]);
                        }
                        if (p.addend) {
                            const float4 *ad = reinterpret_cast<const float4 *>(p.addend + o);
#pragma unroll
                            for (int k = 0; k < 4; ++k) {
                                const float4 a4 = ad[k];
                                f[4 * k] = __fadd_rn(f[4 * k], a4.x); f[4 * k + 1] = __fadd_rn(f[4 * k + 1], a4.y);
                                f[4 * k + 2] = __fadd_rn(f[4 * k + 2], a4.z); f[4 * k + 3] = __fadd_rn(f[4 * k + 3], a4.w);
                            }
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
        if (p.tma_out && lane == 0) tma_store_wait_all();     // staged tiles read and written out before the CTA ends
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
    int RBx, RBe, merged;                         // row bytes of the input tiles and of the error tiles
    int halo, PW, PH, halo_bytes;                 // 16-channel halo mode: one input box per pixel tile (see below)
    int mgroups, ngroups, mtiles, BNc, total_units;
    int stages, tmem_cols;
    int cin_real;                                 // channels of the caller's weight layout (< Cin when the input was zero-padded)
    int32_t *acc_out;                             // int32 sums [nodes][Cout][taps][cin_real] (nullable if 1 split)
    float *dW; long long dw_stride;               // fp32 result, written here only if 1 split (nullable)
    const float *s1, *s2;                         // per-node scales of the two operands
    int32_t *dev_status;
    int uns;                                      // operands are unsigned 8-bit codes
};

__global__ void __launch_bounds__(kThreads, 1)
conv_wgrad_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapE,
                  const WgParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    SharedCtl *ctl = reinterpret_cast<SharedCtl *>(smem);
    unsigned char *data = smem + 1024;
    // warp index (and below the TMEM base) go through a shuffle so that the compiler knows they are
    // warp-uniform and keeps the single-issuer role loops on the uniform datapath
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int node = blockIdx.z;
    const int mg = blockIdx.y % p.mgroups, ng = blockIdx.y / p.mgroups;
    const int G = 128 / p.RBx;                    // input boxes stacked in one 128-lane M tile
    const int x_unit = 128 * p.RBx, e_unit = 128 * p.RBe;
    const int mu0 = mg * p.mtiles * G;
    int nX = p.total_units - mu0; if (nX > p.mtiles * G) nX = p.mtiles * G;
    const int n0 = ng * p.BNc, nE = p.BNc / p.RBe;
    const int x_region = p.halo ? p.halo_bytes : p.mtiles * 16384;
    const int stage_bytes = x_region + 128 * p.BNc;
    const int kb0 = blockIdx.x * p.kb_per_split;
    int kb1 = kb0 + p.kb_per_split; if (kb1 > p.kblocks) kb1 = p.kblocks;
    const int cpt = p.Cin / p.RBx;

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
    pdl_enter();          // nothing above touches global memory
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, ctl->tmem_base, 0);

    if (warp == 0) {
        {
            if (elect_one()) { tma_prefetch_desc(&mapX); tma_prefetch_desc(&mapE); }
            int st = 0; uint32_t ph = 0;
            int tw = kb0 % p.tilesW, th = (kb0 / p.tilesW) % p.tilesH, tb = kb0 / (p.tilesW * p.tilesH);
            const int tap0 = mu0 / cpt, chunk0 = mu0 % cpt, r0 = tap0 / p.S, s0 = tap0 % p.S;
            for (int kb = kb0; kb < kb1; ++kb) {
                const int w0 = tw * p.TW, h0 = th * p.TH, b0 = tb * p.TB;
                if (!mbar_wait(smem_u32(&ctl->empty[st]), ph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                const uint32_t full = smem_u32(&ctl->full[st]);
                const bool leader = elect_one();
                if (leader) mbar_expect_tx(full, (p.halo ? p.PW * p.PH * 16 : nX * x_unit) + nE * e_unit);
                uint32_t x_dst = smem_u32(data + (size_t)st * stage_bytes);
                uint32_t e_dst = x_dst + x_region;
                for (int c = 0; c < nE; ++c, e_dst += e_unit)
                    if (leader) tma_load_5d(e_dst, &mapE, full, n0 + c * p.RBe, w0, h0, b0, node);
                // halo mode: the 8 x 16 pixel tile plus its filter halo in one box; taps are descriptor offsets
                if (p.halo && leader) tma_load_4d(x_dst, &mapX, full, (w0 - p.pad) * 16, h0 - p.pad, b0, node);
                int chunk = chunk0, r = r0, s = s0;
                for (int i = 0; i < (p.halo ? 0 : nX); ++i, x_dst += x_unit) {
                    const int wc = w0 * p.stride + s - p.pad, hc = h0 * p.stride + r - p.pad;
                    if (leader) {
                        if (p.merged) tma_load_4d(x_dst, &mapX, full, wc * 16, hc, b0, node);
                        else tma_load_5d(x_dst, &mapX, full, chunk * p.RBx, wc, hc, b0, node);
                    }
                    if (++chunk == cpt) { chunk = 0; if (++s == p.S) { s = 0; ++r; } }
                }
                __syncwarp();
                if (++tw == p.tilesW) { tw = 0; if (++th == p.tilesH) { th = 0; ++tb; } }
                if (++st == p.stages) { st = 0; ph ^= 1; }
            }
        }
    } else if (warp == 1) {
        {
            const uint32_t idesc = idesc_i8(128, p.BNc, 1, 1, p.uns);
            // halo mode: M tile r stacks the S taps of filter row r, one pixel (16 bytes) apart; 8-pixel
            // K groups are one halo row apart
            const uint64_t a_tpl = p.halo ? smem_desc(0, p.PW * 16, 16, 0)
                                 : (p.RBx == 16) ? smem_desc(0, 128, x_unit, 0)
                                                 : smem_desc(0, x_unit, 8 * p.RBx, layout_code(p.RBx));
            const uint64_t b_tpl = (p.RBe == 16) ? smem_desc(0, 128, e_unit, 0)
                                                 : smem_desc(0, e_unit, 8 * p.RBe, layout_code(p.RBe));
            const uint32_t a_step = p.halo ? (uint32_t)(4 * p.PW) : (uint32_t)((32 * p.RBx) >> 4);   // 32 pixel rows per MMA
            const uint32_t b_step = (32 * p.RBe) >> 4;
            const uint32_t a_tile_step = p.halo ? (uint32_t)p.PW : (uint32_t)(16384 >> 4);
            uint32_t accum = 0;
            int st = 0; uint32_t ph = 0;
            for (int kb = kb0; kb < kb1; ++kb) {
                if (!mbar_wait(smem_u32(&ctl->full[st]), ph, &ctl->abort_flag, p.dev_status)) break;
                tc_fence_after();
                const uint32_t x_st = smem_u32(data + (size_t)st * stage_bytes);
                const uint32_t e_lo0 = (x_st + x_region) >> 4;
                if (elect_one()) {
                    uint32_t a_tile = x_st >> 4, d_tmem = tmem_base;
                    for (int t = 0; t < p.mtiles; ++t) {
                        uint32_t a_lo = a_tile, b_lo = e_lo0;
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            mma_i8(d_tmem, a_tpl | (a_lo & 0x3FFFu), b_tpl | (b_lo & 0x3FFFu), idesc, accum | (uint32_t)kk);
                            a_lo += a_step; b_lo += b_step;
                        }
                        a_tile += a_tile_step; d_tmem += p.BNc;
                    }
                    mma_commit(smem_u32(&ctl->empty[st]));
                    if (kb == kb1 - 1) mma_commit(smem_u32(&ctl->tmem_full[0]));
                }
                __syncwarp();
                accum = 1;
                if (++st == p.stages) { st = 0; ph ^= 1; }
            }
        }
    } else if (kb1 > kb0) {
        // Epilogue.  One split: raw sums and/or the dequantized fp32 result go straight to their
        // destinations.  Several splits: partial sums are added with exact int32 atomics into zeroed
        // storage and the launcher converts them afterwards.
        const int q = warp & 3;
        const int row = q * 32 + lane;
        if (mbar_wait(smem_u32(&ctl->tmem_full[0]), 0, &ctl->abort_flag, p.dev_status)) {
            tc_fence_after();
            const float sc = (p.dW && p.splits == 1) ? __fmul_rn(p.s1[node], p.s2[node]) : 0.f;
            const long long cstride = (long long)p.taps * p.cin_real;
            for (int t = 0; t < p.mtiles; ++t) {
                int tap, ci; bool valid;
                if (p.halo) {                                       // lane = (s, ci) of filter row t
                    tap = t * p.S + (row >> 4); ci = row & 15; valid = (row >> 4) < p.S;
                } else {
                    const int i = t * G + row / p.RBx;             // input box within this CTA
                    const int mu = mu0 + i;
                    valid = (i < nX) && (mu < p.total_units);
                    tap = mu / cpt; ci = (mu % cpt) * p.RBx + row % p.RBx;
                }
                valid = valid && (ci < p.cin_real);
                const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + t * p.BNc;
                for (int c = 0; c < p.BNc; c += 16) {
                    uint32_t v[16];
                    tmem_ld_32x16(t_row + c, v);
                    tmem_ld_wait();
                    if (!valid) continue;
                    const long long o = ((long long)(n0 + c) * p.taps + tap) * p.cin_real + ci;
                    int32_t *acc = p.acc_out + (long long)node * p.Cout * cstride + o;
                    if (p.splits > 1) {
#pragma unroll
                        for (int k = 0; k < 16; ++k)
                            if ((int)v[k] != 0) atomicAdd(acc + k * cstride, (int)v[k]);
                    } else {
                        if (p.acc_out) {
#pragma unroll
                            for (int k = 0; k < 16; ++k) acc[k * cstride] = (int)v[k];
                        }
                        if (p.dW) {
                            float *dst = p.dW + (long long)node * p.dw_stride + o;
#pragma unroll
                            for (int k = 0; k < 16; ++k) dst[k * cstride] = __fmul_rn(__int2float_rn((int)v[k]), sc);
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
static void pick_tile(int H, int W, int max_tw, int *TB, int *TH, int *TW) {
    int bw = 1; long best = -1;
    for (int t = 1; t <= max_tw; t <<= 1) {
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

// Activation map: box = {RB channel bytes, TW, TH, TB pixels, 1 node}.  With estride 2 the
// box samples every second pixel (the traversal stride of the tensor map), which is how
// a stride-2 convolution reads its input.
static bool act_map(CUtensorMap *m, const int8_t *base, int nodes, int B, int H, int W, int C, int RB,
                    int TB, int TH, int TW, int estride = 1) {
    uint64_t dims[5] = {(uint64_t)C, (uint64_t)W, (uint64_t)H, (uint64_t)B, (uint64_t)nodes};
    uint64_t strides[4] = {(uint64_t)C, (uint64_t)W * C, (uint64_t)H * W * C, (uint64_t)B * H * W * C};
    uint32_t box[5] = {(uint32_t)RB, (uint32_t)(TW * estride), (uint32_t)(TH * estride), (uint32_t)TB, 1};
    uint32_t es[5] = {1, (uint32_t)estride, (uint32_t)estride, 1, 1};
    return make_map_u8(m, base, 5, dims, strides, box, swizzle_for(RB), es);
}
// C = 16, stride 1: (channel, width) is one contiguous row of 16*W bytes; a box row is TW pixels.
static bool act_map_merged(CUtensorMap *m, const int8_t *base, int nodes, int B, int H, int W,
                           int TB, int TH, int TW) {
    uint64_t dims[4] = {(uint64_t)W * 16, (uint64_t)H, (uint64_t)B, (uint64_t)nodes};
    uint64_t strides[3] = {(uint64_t)W * 16, (uint64_t)H * W * 16, (uint64_t)B * H * W * 16};
    uint32_t box[4] = {(uint32_t)TW * 16, (uint32_t)TH, (uint32_t)TB, 1};
    return make_map_u8(m, base, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE);
}

static bool weight_map(CUtensorMap *m, const int8_t *base, int nodes, int Cout, int taps, int Cin, int box_inner,
                       int box_rows) {
    uint64_t dims[3] = {(uint64_t)Cin, (uint64_t)taps, (uint64_t)nodes * Cout};
    uint64_t strides[2] = {(uint64_t)Cin, (uint64_t)taps * Cin};
    uint32_t box[3] = {(uint32_t)box_inner, 1, (uint32_t)box_rows};
    return make_map_u8(m, base, 3, dims, strides, box, swizzle_for(box_inner));
}

constexpr int kSmemBudget = 200 * 1024;
constexpr int kMinSmem = 120 * 1024;      // keeps one CTA per SM, so TMEM allocation never waits
constexpr int kMinSmemTwo = 78 * 1024;    // two-CTAs-per-SM launches: keeps a third one out
// LPDT_PIX_TWO=0: one CTA per SM for every shape (A/B timing, parity tests)
static bool pix_two_enabled() {
    static int on = -1;
    if (on < 0) { const char *e = getenv("LPDT_PIX_TWO"); on = (e && e[0] == '0') ? 0 : 1; }
    return on == 1;
}

bool tc_supported(const lpdt_conv_desc &d) {
    if (d.stride != 1 && d.stride != 2) return false;
    if (d.Cin % 16 || d.Cout % 16) return false;
    if (d.R * d.S > kMaxTaps || d.R > 100 || d.S > 100 || d.pad > 100) return false;
    if (!encode_tiled_fn()) return false;
    return true;
}

// LPDT_PIX_DIRECT_STORE=1 keeps the pixel kernel's per-lane global stores (A/B timing and parity tests).
static bool pix_tma_out_enabled() {
    static int off = -1;
    if (off < 0) { const char *e = getenv("LPDT_PIX_DIRECT_STORE"); off = (e && e[0] == '1') ? 1 : 0; }
    return off == 0;
}

static int largest_div(int C, int cap, int unit) {      // largest multiple of unit dividing C, <= cap
    for (int v = cap - cap % unit; v >= unit; v -= unit) if (C % v == 0) return v;
    return unit;
}

lpdt_status tc_pix(const lpdt_conv_desc &d, int mode, const int8_t *A, const float *s1, const int8_t *Wq,
                   const float *s2, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                   int32_t *dev_status, cudaStream_t st, bool uns, const float *addend, const AffineArgs *aff) {
    const int Ho = conv_out(d.H, d.pad, d.R, d.stride), Wo = conv_out(d.W, d.pad, d.S, d.stride);
    PixParams p = {};
    p.addend = addend;
    if (aff) {
        if (mode != 0 || d.Cout % 4) return LPDT_ERR_UNSUPPORTED;
        p.asum = aff->asum; p.wpre = aff->wpre; p.zA = aff->zA; p.zW = aff->zW;
        p.aH = d.H; p.aW = d.W; p.aR = d.R; p.aS = d.S; p.apad = d.pad; p.astride = d.stride; p.aCin = d.Cin;
    }
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
                    tt.dh[tt.ntaps] = (signed char)((ph + d.pad - r) / d.stride);   // exact: divisible
                    tt.dw[tt.ntaps] = (signed char)((pw + d.pad - s) / d.stride);
                    ++tt.ntaps;
                }
            }
        }
    }
    p.RBa = row_bytes_for(p.Kc);
    p.RBn = row_bytes_for(p.Nc);
    const int estride = mode == 0 ? d.stride : 1;
    p.merged = (p.Kc == 16 && estride == 1) ? 1 : 0;
    pick_tile(p.Hm, p.Wm, p.merged ? 16 : 128, &p.TB, &p.TH, &p.TW);
    if (p.TW * estride > 256 || p.TH * estride > 256) return LPDT_ERR_UNSUPPORTED;
    p.tilesB = (int)ceil_div(d.B, p.TB); p.tilesH = (int)ceil_div(p.Hm, p.TH); p.tilesW = (int)ceil_div(p.Wm, p.TW);
    p.BN = largest_div(p.Nc, 256, mode == 0 ? 16 : p.RBn);
    {   // few tiles (small maps, small batches, small GEMMs): narrower N tiles while the doubled count still fits
        // one wave of SMs.  Measured: 32 -> 64 -> 128 tiles gains 10-80 %; past one wave the narrower tile's
        // extra shared-memory traffic per MMA loses 10-25 %.
        const long long mtiles = (long long)p.nodes * p.tilesB * p.tilesH * p.tilesW * p.ncls;
        const int unit = mode == 0 ? 16 : p.RBn;
        while (p.BN >= 128 && p.BN % 2 == 0 && (p.BN / 2) % unit == 0 && 2 * mtiles * (p.Nc / p.BN) <= kNumSMs) p.BN /= 2;
    }
    p.tilesN = p.Nc / p.BN;
    const int cpt = p.Kc / p.RBa;
    const int unit_bytes = 128 * p.RBa + p.BN * p.RBa;
    // K units per stage: stage <= 48 KB, at most 16 units, an even count for 16-byte rows (one MMA
    // consumes two of them); the least padded work over the classes wins, ties go to the larger stage
    int U = 0; long best = -1;
    const int ustep = p.RBa == 16 ? 2 : 1;
    for (int u = ustep; u <= 16; u += ustep) {
        if (u * unit_bytes > 48 * 1024 && U) break;
        long work = 0;
        for (int c = 0; c < p.ncls; ++c) {
            long n = (long)p.tt[c].ntaps * cpt; if (n < 1) n = 1;
            work += ceil_div(n, u) * u;
        }
        if (best < 0 || work <= best) { best = work; U = u; }
    }
    p.U = U;
    for (int c = 0; c < p.ncls; ++c) {
        p.cls_iters[c] = (int)ceil_div((long)p.tt[c].ntaps * cpt, U);
        if (p.cls_iters[c] < 1) p.cls_iters[c] = 1;      // a class without taps still writes zeros
    }
    // long K loops (GEMM-like): blocked round-robin tile order; short ones: contiguous ranges
    p.raster = (p.ncls == 1 && p.cls_iters[0] >= 8) ? 1 : 0;
    const int stage_bytes = U * unit_bytes;
    // fp32 result through shared memory and bulk tensor stores (not with raw accumulators, not for the strided
    // pixel classes of a stride-2 backward-data pass): 8 warps x 4 KB of staging after the ring
    p.tma_out = (Y && !Yacc && aligned(Y, 16) && p.ncls == 1 && p.out_mul == 1 && p.BN % 32 == 0 &&
                 pix_tma_out_enabled()) ? 1 : 0;
    p.bw = p.TW < 32 ? p.TW : 32;
    p.bh = p.TH < 32 / p.bw ? p.TH : 32 / p.bw;
    const int out_bytes = p.tma_out ? 32 * 1024 + 1024 : 0;        // 8 warps x 4 KB + slack to reach a 1024-byte boundary
    p.stages = ((p.tma_out ? 227 * 1024 - out_bytes : kSmemBudget) - 1024) / stage_bytes;
    if (p.stages > 8) p.stages = 8;
    if (p.stages < 2) return LPDT_ERR_UNSUPPORTED;
    p.tmem_cols = pow2_at_least(2 * p.BN);
    const long long tiles = (long long)p.nodes * p.tilesB * p.tilesH * p.tilesW * p.tilesN * p.ncls;
    if (tiles > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    // Two CTAs per SM for short K loops (at most four stages per tile) over more than one tile per SM: such
    // a CTA spends most of its time filling and draining, which a neighbour on the same SM hides.  Needs two
    // stages and the staging buffers inside half of the shared memory and both accumulator pairs in TMEM.
    bool two = false;
    {
        int longest = 0;
        for (int c = 0; c < p.ncls; ++c) longest = p.cls_iters[c] > longest ? p.cls_iters[c] : longest;
        const int stages2 = (113 * 1024 - out_bytes - 1024) / stage_bytes;
        two = pix_two_enabled() && longest <= 4 && tiles > kNumSMs && stages2 >= 2 && 2 * p.tmem_cols <= 512;
        if (two) p.stages = stages2 > 8 ? 8 : stages2;
    }
    p.w_rows_per_node = d.Cout;
    p.Y = Y; p.Yacc = Yacc; p.s1 = s1; p.s2 = s2; p.bias = bias; p.bias_stride = bias_stride;
    p.dev_status = dev_status; p.uns = uns ? 1 : 0;
    CUtensorMap mA, mW;
    // operand A: activations (fwd: image H x W, Cin, sampled with the conv stride) or errors
    // (bwd-data: image Ho x Wo, Cout, dense)
    const int Ha = mode == 0 ? d.H : Ho, Wa = mode == 0 ? d.W : Wo;
    if (p.merged) { if (!act_map_merged(&mA, A, d.nodes, d.B, Ha, Wa, p.TB, p.TH, p.TW)) return LPDT_ERR_CUDA; }
    else if (!act_map(&mA, A, d.nodes, d.B, Ha, Wa, p.Kc, p.RBa, p.TB, p.TH, p.TW, estride)) return LPDT_ERR_CUDA;
    if (mode == 0) { if (!weight_map(&mW, Wq, d.nodes, d.Cout, d.R * d.S, d.Cin, p.RBa, p.BN)) return LPDT_ERR_CUDA; }
    else if (!weight_map(&mW, Wq, d.nodes, d.Cout, d.R * d.S, d.Cin, p.RBn, p.RBa)) return LPDT_ERR_CUDA;
    size_t smem = 1024 + (size_t)p.stages * stage_bytes;
    CUtensorMap mY = CUtensorMap{};
    if (p.tma_out) {
        p.out_off = (int)align_up(smem, 1024);
        smem = (size_t)p.out_off + 32 * 1024;
        uint64_t dims[5] = {(uint64_t)p.Nc, (uint64_t)p.Wout, (uint64_t)p.Hout, (uint64_t)d.B, (uint64_t)d.nodes};
        uint64_t strides[4] = {(uint64_t)p.Nc * 4, (uint64_t)p.Wout * p.Nc * 4, (uint64_t)p.Hout * p.Wout * p.Nc * 4,
                               (uint64_t)d.B * p.Hout * p.Wout * p.Nc * 4};
        uint32_t box[5] = {32, (uint32_t)p.bw, (uint32_t)p.bh, (uint32_t)(32 / (p.bw * p.bh)), 1};
        if (!make_map(&mY, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, Y, 5, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B))
            return LPDT_ERR_CUDA;
    }
    if (smem < (two ? kMinSmemTwo : kMinSmem)) smem = two ? kMinSmemTwo : kMinSmem;
    if (smem > (two ? (size_t)113 * 1024 : (size_t)227 * 1024)) return LPDT_ERR_UNSUPPORTED;
    static PerDeviceOnce attr;
    int dev;
    if (attr.pending(&dev)) {
        LPDT_CUDA(cudaFuncSetAttribute(conv_pix_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        LPDT_CUDA(cudaFuncSetAttribute(conv_pix_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, 113 * 1024));
        attr.mark(dev);
    }
    const int slots = two ? 2 * kNumSMs : kNumSMs;
    const int grid = (int)(tiles < slots ? tiles : slots);
    g_last_kernel = "lpdt::tc::conv_pix_kernel";
    if (two) launch_k(conv_pix_kernel<2>, grid, kPixThreads, smem, st, mA, mW, mY, p);
    else launch_k(conv_pix_kernel<1>, grid, kPixThreads, smem, st, mA, mW, mY, p);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

// acc_user: the caller's raw-sum array or null; acc_ws: scratch of the same shape [nodes][Cout][taps][cin_real]
// (the caller's weight layout); dW: fp32 result or null.  With one split the kernel writes both outputs
// itself; with several it accumulates into zeroed int32 storage and a conversion launch follows.
lpdt_status tc_wgrad(const lpdt_conv_desc &d, int cin_real, const int8_t *E, const float *sE, const int8_t *A,
                     const float *sA, int32_t *acc_user, int32_t *acc_ws, float *dW, int64_t dw_stride,
                     int32_t *dev_status, cudaStream_t st, bool uns) {
    const int Ho = conv_out(d.H, d.pad, d.R, d.stride), Wo = conv_out(d.W, d.pad, d.S, d.stride);
    WgParams p = {};
    p.nodes = d.nodes; p.B = d.B; p.Ho = Ho; p.Wo = Wo; p.Cin = d.Cin; p.Cout = d.Cout;
    p.R = d.R; p.S = d.S; p.pad = d.pad; p.taps = d.R * d.S; p.stride = d.stride;
    p.RBx = row_bytes_for(d.Cin); p.RBe = row_bytes_for(d.Cout);
    p.merged = (d.Cin == 16 && d.stride == 1) ? 1 : 0;
    p.BNc = largest_div(d.Cout, 256, p.RBe);
    p.halo = (p.merged && d.S <= 8 && d.R * p.BNc <= 512 && d.R <= 16) ? 1 : 0;
    if (p.halo) { p.TW = 8; p.TH = 16; p.TB = 1; p.PW = 8 + d.S - 1; p.PH = 16 + d.R - 1; p.halo_bytes = (int)align_up((size_t)p.PW * p.PH * 16 + 256, 1024); }
    else pick_tile(Ho, Wo, p.merged ? 16 : 128, &p.TB, &p.TH, &p.TW);
    if (p.TW * d.stride > 256 || p.TH * d.stride > 256) return LPDT_ERR_UNSUPPORTED;
    p.tilesB = (int)ceil_div(d.B, p.TB); p.tilesH = (int)ceil_div(Ho, p.TH); p.tilesW = (int)ceil_div(Wo, p.TW);
    p.kblocks = p.tilesB * p.tilesH * p.tilesW;
    const int G = 128 / p.RBx;
    p.total_units = p.taps * (d.Cin / p.RBx);
    const int all_tiles = (int)ceil_div(p.total_units, G);
    // Short pixel loops (GEMM-like shapes with few rows): rather narrower N groups, so that the output tiles alone
    // give the SMs work, than a split of a loop of a few blocks whose partial sums meet in atomics.
    // (Measured on the GEMM sweep: up to 64 output tiles this is 2.3-3.4 times faster; from 128 tiles on the split
    // wins.)
    const bool short_k = !p.halo && p.kblocks <= 16 && (long long)d.nodes * all_tiles * (d.Cout / p.BNc) <= 64;
    if (short_k)
        while (p.BNc >= 2 * p.RBe && p.BNc >= 256 && (long long)d.nodes * all_tiles * (d.Cout / p.BNc) < kNumSMs) p.BNc /= 2;
    p.ngroups = d.Cout / p.BNc;
    int mt = 512 / p.BNc;                                        // accumulators that fit in TMEM
    const int mt_smem = (96 * 1024 - 128 * p.BNc) / 16384;       // stage <= 96 KB -> at least two stages
    if (mt > mt_smem) mt = mt_smem;
    if (mt > all_tiles) mt = all_tiles;
    if (mt < 1) return LPDT_ERR_UNSUPPORTED;
    // Few nodes with small layers: rather more CTAs with fewer M tiles each (the error tile is re-read
    // from L2) than a deep split of the pixel loop, whose partial sums meet in atomics.
    while (mt > 1 && (long long)d.nodes * ceil_div(all_tiles, mt) * p.ngroups < kNumSMs) --mt;
    p.mtiles = mt;
    p.mgroups = (int)ceil_div(all_tiles, mt);
    if (p.halo) { p.mtiles = d.R; p.mgroups = 1; }
    const int stage_bytes = (p.halo ? p.halo_bytes : p.mtiles * 16384) + 128 * p.BNc;
    p.tmem_cols = pow2_at_least(p.mtiles * p.BNc);
    if (p.tmem_cols > 512) return LPDT_ERR_UNSUPPORTED;
    // CTAs per SM: as many (up to four) as leave each at least four stages and fit TMEM; the shared-memory
    // request keeps any further CTA off the SM, so a TMEM allocation never waits
    int per_sm = 4;
    for (;; --per_sm) {
        p.stages = ((224 * 1024) / per_sm - 2048 - 1024) / stage_bytes;
        if (p.stages > 8) p.stages = 8;
        if (per_sm == 1 || (p.stages >= 4 && per_sm * p.tmem_cols <= 512)) break;
    }
    if (p.stages < 2) return LPDT_ERR_UNSUPPORTED;
    const long long ctas_fixed = (long long)d.nodes * p.mgroups * p.ngroups;
    const long long slots = (long long)kNumSMs * per_sm;         // one wave of co-resident CTAs
    int splits = ctas_fixed >= slots ? 1 : (int)(slots / ctas_fixed);
    if (short_k) splits = 1;
    if (splits > p.kblocks) splits = p.kblocks;
    if (splits < 1) splits = 1;
    p.kb_per_split = (int)ceil_div(p.kblocks, splits);
    p.splits = (int)ceil_div(p.kblocks, p.kb_per_split);
    p.cin_real = cin_real; p.dW = dW; p.dw_stride = dw_stride; p.s1 = sE; p.s2 = sA;
    p.acc_out = p.splits == 1 ? acc_user : (acc_user ? acc_user : acc_ws);
    p.dev_status = dev_status; p.uns = uns ? 1 : 0;
    CUtensorMap mX, mE;
    if (p.halo) {
        uint64_t dims[4] = {(uint64_t)d.W * 16, (uint64_t)d.H, (uint64_t)d.B, (uint64_t)d.nodes};
        uint64_t strides[3] = {(uint64_t)d.W * 16, (uint64_t)d.H * d.W * 16, (uint64_t)d.B * d.H * d.W * 16};
        uint32_t box[4] = {(uint32_t)p.PW * 16, (uint32_t)p.PH, 1, 1};
        if (!make_map_u8(&mX, A, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return LPDT_ERR_CUDA;
    } else if (p.merged) { if (!act_map_merged(&mX, A, d.nodes, d.B, d.H, d.W, p.TB, p.TH, p.TW)) return LPDT_ERR_CUDA; }
    else if (!act_map(&mX, A, d.nodes, d.B, d.H, d.W, d.Cin, p.RBx, p.TB, p.TH, p.TW, d.stride)) return LPDT_ERR_CUDA;
    if (!act_map(&mE, E, d.nodes, d.B, Ho, Wo, d.Cout, p.RBe, p.TB, p.TH, p.TW)) return LPDT_ERR_CUDA;
    size_t smem = 1024 + (size_t)p.stages * stage_bytes;
    if (smem < (size_t)(228 * 1024) / (per_sm + 1)) smem = (size_t)(228 * 1024) / (per_sm + 1);
    if (smem > 227 * 1024) return LPDT_ERR_UNSUPPORTED;
    static PerDeviceOnce attr;
    int dev;
    if (attr.pending(&dev)) {
        LPDT_CUDA(cudaFuncSetAttribute(conv_wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr.mark(dev);
    }
    if (d.nodes > 65535 || p.mgroups * p.ngroups > 65535) return LPDT_ERR_UNSUPPORTED;
    const int64_t per_node = (int64_t)d.Cout * p.taps * cin_real;
    if (p.splits > 1) {
        if (!p.acc_out) return LPDT_ERR_WORKSPACE;
        LPDT_CUDA(cudaMemsetAsync(p.acc_out, 0, (size_t)d.nodes * per_node * sizeof(int32_t), st));
    }
    g_last_kernel = "lpdt::tc::conv_wgrad_kernel";
    launch_k(conv_wgrad_kernel, dim3(p.splits, p.mgroups * p.ngroups, d.nodes), kThreads, smem, st, mX, mE, p);
    LPDT_LAUNCH_CHECK();
    if (p.splits > 1 && dW) return dequant_acc_launch(p.acc_out, d.nodes, per_node, sE, sA, dW, dw_stride, st);
    return LPDT_OK;
}

}  // namespace tc
}  // namespace lpdt
