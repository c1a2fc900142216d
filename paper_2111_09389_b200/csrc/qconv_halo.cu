// Halo-tile variant of the pixel-M convolution kernel for narrow operands at
// stride 1 (K channels = 16, 32, 64, 96 or 128): forward by Cin, backward-data by
// Cout.
//
// A 16-channel chunk of a pixel is exactly one 16-byte row of the no-swizzle
// core-matrix layout, and a filter tap is a shift by whole rows.  So instead of
// one TMA box per tap, one box per tile fetches the 8 x 16 pixel tile together
// with its halo ((8+S-1) x (16+R-1) pixels, out-of-image pixels zero-filled),
// and each tap is reached through the matrix descriptor alone: start address =
// the tap's offset inside the halo, stride between 8-row groups = the halo row
// pitch, and the leading-dimension offset = the distance to the second tap of the
// pair that shares a K = 32 MMA (an odd last tap is paired with a block of zeros).
// With more than 16 channels the box carries the 16-byte chunks as its outermost
// dimension (one halo image per chunk) and an MMA pairs two chunks of the same tap.
// The node's weights are loaded into shared memory once per node, not per tile.
// Per tile this is 1 TMA request and ceil(taps*chunks/2) MMAs.
#include <stdlib.h>
#include "qconv_internal.cuh"
#include "tc_common.cuh"

namespace lpdt {
namespace tc {

constexpr int kHaloThreads = 192;
constexpr int kHaloMaxTaps = 64;
constexpr int kHaloMaxMma = 72;
constexpr int kTileW = 8, kTileH = 16;
constexpr int kZeroBytes = 4096;          // >= 15 halo rows of at most 256 bytes + one 8-row group

struct HaloParams {
    int mode;                  // 0 forward, 1 backward-data
    int uns;                   // operands are unsigned 8-bit codes
    int nodes, B, Hm, Wm;      // output image of this pass
    int N;                     // output channels of this pass
    int ntaps, cpt, nslices;   // taps, 16-channel chunks per tap, K slices = taps * chunks (order: tap, chunk)
    signed char wtap[kHaloMaxTaps];       // tap index in the weight tensor of the i-th tap in halo order
    int n_mma;                            // one MMA per pair of K slices
    unsigned short a_off16[kHaloMaxMma];  // first slice of the pair: offset inside the stage, in 16-byte rows
    unsigned short a_lbo16[kHaloMaxMma];  // distance to the second slice (0xFFFF: pair with the zero block)
    int org_h, org_w;          // halo origin relative to the tile origin (smallest tap offsets)
    int PH, PW;                // halo rows / pixels per row
    int tilesH, tilesW;
    int stages, halo_bytes, wres_bytes, tmem_cols;
    int nacc_log2;             // log2 of the number of TMEM accumulators (2, 4 or 8 tiles in flight)
    int tma_out;               // fp32 result leaves through shared memory and bulk tensor stores
    int out_inner;             // channels per store box: 32 (128-byte swizzled rows) or 16 (64-byte)
    int w_rows_per_node;
    float *Y; int32_t *Yacc;
    const float *s1, *s2, *bias; long long bias_stride;
    const float *addend;       // nullable: fp32 tensor of the result's shape, added to the dequantized result
    int32_t *dev_status;
};

struct HaloCtl {
    unsigned long long full[8], empty[8], tmem_full[8], tmem_empty[8], wfull;
    uint32_t tmem_base;
    volatile int abort_flag;
};

struct HaloTile { int tw, th, b, node; };
__device__ __forceinline__ HaloTile halo_decode(const HaloParams &p, int tile) {
    HaloTile c; int t = tile;
    c.tw = t % p.tilesW; t /= p.tilesW;
    c.th = t % p.tilesH; t /= p.tilesH;
    c.b = t % p.B; c.node = t / p.B;
    return c;
}
__device__ __forceinline__ void halo_next(const HaloParams &p, HaloTile &c) {
    if (++c.tw < p.tilesW) return; c.tw = 0;
    if (++c.th < p.tilesH) return; c.th = 0;
    if (++c.b < p.B) return; c.b = 0;
    ++c.node;
}

__global__ void __launch_bounds__(kHaloThreads, 1)
conv_halo16_kernel(const __grid_constant__ CUtensorMap mapA, const __grid_constant__ CUtensorMap mapW,
                   const __grid_constant__ CUtensorMap mapY, const HaloParams p) {
    extern __shared__ __align__(1024) unsigned char smem[];
    HaloCtl *ctl = reinterpret_cast<HaloCtl *>(smem);
    unsigned char *wres = smem + 1024;
    unsigned char *stage0 = wres + p.wres_bytes;
    unsigned char *zeros = stage0 + (size_t)p.stages * p.halo_bytes;     // above every tile: offsets to it are positive
    // two result tiles of 128 x N fp32 (tma_out), on a swizzle-atom boundary
    unsigned char *out_tiles = smem + (((size_t)(zeros - smem) + kZeroBytes + 1023) & ~(size_t)1023);
    // warp index and TMEM base are broadcast through a shuffle so that the compiler knows they are
    // warp-uniform and keeps the role loops on the uniform datapath
    const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const long long total_tiles = (long long)p.nodes * p.B * p.tilesH * p.tilesW;
    const int tile_lo = (int)(total_tiles * blockIdx.x / gridDim.x);
    const int tile_hi = (int)(total_tiles * (blockIdx.x + 1) / gridDim.x);

    for (int i = threadIdx.x; i < kZeroBytes / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(zeros)[i] = 0u;
    for (int i = threadIdx.x; i < p.wres_bytes / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(wres)[i] = 0u;
    if (threadIdx.x == 0) {
        for (int i = 0; i < p.stages; ++i) { mbar_init(smem_u32(&ctl->full[i]), 1); mbar_init(smem_u32(&ctl->empty[i]), 1); }
        for (int i = 0; i < 8; ++i) { mbar_init(smem_u32(&ctl->tmem_full[i]), 1); mbar_init(smem_u32(&ctl->tmem_empty[i]), 4); }
        mbar_init(smem_u32(&ctl->wfull), 1);
        ctl->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(&ctl->tmem_base), p.tmem_cols); tmem_relinquish(); }
    // the zero fills above are generic-proxy writes that the tensor core (async proxy) will read
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    pdl_enter();          // nothing above touches global memory
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, ctl->tmem_base, 0);
    const int slot_bytes = p.mode == 0 ? p.N * 16 : 256;      // one K slice of weights (backward: per 16-column chunk)
    const int nchunk = p.N / 16;

    if (warp == 0) {
        {
            if (elect_one()) { tma_prefetch_desc(&mapA); tma_prefetch_desc(&mapW); }
            int st = 0; uint32_t ph = 0;
            int cur_node = -1;
            HaloTile c = halo_decode(p, tile_lo);
            for (int tile = tile_lo; tile < tile_hi && !ctl->abort_flag; ++tile, halo_next(p, c)) {
                if (c.node != cur_node) {
                    // drain: every stage issued so far must have been consumed before the weights change
                    int s2 = st; uint32_t ph2 = ph; bool ok = true;
                    for (int i = 0; i < p.stages && ok; ++i) {
                        ok = mbar_wait(smem_u32(&ctl->empty[s2]), ph2 ^ 1, &ctl->abort_flag, p.dev_status);
                        if (++s2 == p.stages) { s2 = 0; ph2 ^= 1; }
                    }
                    if (!ok) break;
                    cur_node = c.node;
                    const uint32_t wfull = smem_u32(&ctl->wfull);
                    const int wrow = c.node * p.w_rows_per_node;
                    if (elect_one()) {
                        mbar_expect_tx(wfull, p.nslices * p.N * 16);
                        int kap = 0;
                        for (int i = 0; i < p.ntaps; ++i)
                            for (int c2 = 0; c2 < p.cpt; ++c2, ++kap) {
                                if (p.mode == 0) {      // N rows of 16 K bytes
                                    tma_load_3d(smem_u32(wres) + kap * slot_bytes, &mapW, wfull, c2 * 16, p.wtap[i], wrow);
                                } else {                // 16 K rows (output channels of the layer) of 16 N bytes
                                    for (int j = 0; j < nchunk; ++j)
                                        tma_load_3d(smem_u32(wres) + (j * (p.nslices + 1) + kap) * 256, &mapW, wfull,
                                                    j * 16, p.wtap[i], wrow + c2 * 16);
                                }
                            }
                    }
                    __syncwarp();
                }
                if (!mbar_wait(smem_u32(&ctl->empty[st]), ph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                const uint32_t full = smem_u32(&ctl->full[st]);
                if (elect_one()) {
                    mbar_expect_tx(full, p.PH * p.PW * 16 * p.cpt);
                    if (p.cpt == 1)
                        tma_load_4d(smem_u32(stage0 + (size_t)st * p.halo_bytes), &mapA, full,
                                    (c.tw * kTileW + p.org_w) * 16, c.th * kTileH + p.org_h, c.b, c.node);
                    else
                        tma_load_5d(smem_u32(stage0 + (size_t)st * p.halo_bytes), &mapA, full, 0,
                                    c.tw * kTileW + p.org_w, c.th * kTileH + p.org_h, c.node * p.B + c.b, 0);
                }
                __syncwarp();
                if (++st == p.stages) { st = 0; ph ^= 1; }
            }
        }
    } else if (warp == 1) {
        {
            const uint32_t idesc = idesc_i8(128, p.N, 0, p.mode == 0 ? 0 : 1, p.uns);
            const uint32_t sbo_a = p.PW * 16;                       // next 8-pixel row group = next halo row
            const uint64_t a_fixed = ((uint64_t)((sbo_a >> 4) & 0x3FFFu) << 32) | ((uint64_t)1 << 46);
            const uint64_t b_tpl = (p.mode == 0) ? smem_desc(0, p.N * 16, 128, 0)
                                                 : smem_desc(0, 128, (p.nslices + 1) * 256, 0);
            const uint32_t w_lo0 = smem_u32(wres) >> 4;
            const uint32_t b_pair_step = (2 * slot_bytes) >> 4;
            const uint32_t zero_lo = smem_u32(zeros) >> 4;
            int st = 0; uint32_t ph = 0, tcount = 0, wph = 0;
            int cur_node = -1;
            HaloTile c = halo_decode(p, tile_lo);
            for (int tile = tile_lo; tile < tile_hi && !ctl->abort_flag; ++tile, ++tcount, halo_next(p, c)) {
                if (c.node != cur_node) {
                    if (!mbar_wait(smem_u32(&ctl->wfull), wph, &ctl->abort_flag, p.dev_status)) break;
                    wph ^= 1; cur_node = c.node;
                }
                const int acc = tcount & ((1u << p.nacc_log2) - 1u);
                const uint32_t aph = (tcount >> p.nacc_log2) & 1;
                if (!mbar_wait(smem_u32(&ctl->tmem_empty[acc]), aph ^ 1, &ctl->abort_flag, p.dev_status)) break;
                if (!mbar_wait(smem_u32(&ctl->full[st]), ph, &ctl->abort_flag, p.dev_status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * p.N;
                const uint32_t halo_lo = smem_u32(stage0 + (size_t)st * p.halo_bytes) >> 4;
                if (elect_one()) {
                    uint32_t b_lo = w_lo0;
                    for (int i = 0; i < p.n_mma; ++i) {
                        const uint32_t s0 = halo_lo + p.a_off16[i];
                        const uint32_t lbo = p.a_lbo16[i] != 0xFFFFu ? (uint32_t)p.a_lbo16[i] : (zero_lo - s0);
                        const uint64_t ad = a_fixed | (uint64_t)(s0 & 0x3FFFu) | ((uint64_t)(lbo & 0x3FFFu) << 16);
                        mma_i8(d_tmem, ad, b_tpl | (b_lo & 0x3FFFu), idesc, (uint32_t)i);
                        b_lo += b_pair_step;
                    }
                    mma_commit(smem_u32(&ctl->empty[st]));
                    mma_commit(smem_u32(&ctl->tmem_full[acc]));
                }
                __syncwarp();
                if (++st == p.stages) { st = 0; ph ^= 1; }
            }
        }
    } else {
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const int pw = row % kTileW, phh = row / kTileW;
        uint32_t tcount = 0;
        HaloTile c = halo_decode(p, tile_lo);
        int sc_node = -1; float sc = 0.f;
        if (p.tma_out && lane == 0) tma_prefetch_desc(&mapY);
        for (int tile = tile_lo; tile < tile_hi && !ctl->abort_flag; ++tile, ++tcount, halo_next(p, c)) {
            const int w = c.tw * kTileW + pw, h = c.th * kTileH + phh;
            const bool valid = (w < p.Wm) && (h < p.Hm);
            if (p.Y && c.node != sc_node) { sc_node = c.node; sc = __fmul_rn(p.s1[c.node], p.s2[c.node]); }
            const int acc = tcount & ((1u << p.nacc_log2) - 1u);
            const uint32_t aph = (tcount >> p.nacc_log2) & 1;
            if (!mbar_wait(smem_u32(&ctl->tmem_full[acc]), aph, &ctl->abort_flag, p.dev_status)) break;
            tc_fence_after();
            const long long pix = (((long long)c.node * p.B + c.b) * p.Hm + h) * p.Wm + w;
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + acc * p.N;
            if (p.tma_out) {
                // Result rows -> shared memory (pixel-major, the layout of the store's box) -> bulk tensor stores.
                // Every epilogue warp stores its own 32 pixels (4 rows of the tile) and tracks its own stores, so
                // the four warps never wait for one another; parts of a box outside the image are not written.
                // Two buffers per warp: the store issued two tiles ago must have finished reading this one.
                const int ob = tcount & 1u;
                unsigned char *ot = out_tiles + (size_t)ob * 128 * p.N * 4;
                if (lane == 0) tma_store_wait_read<1>();
                __syncwarp();
                const int inner = p.out_inner;
                const uint32_t sw = inner == 32 ? (uint32_t)(row & 7) : (uint32_t)((row >> 1) & 3);   // the box's swizzle
                for (int cc = 0; cc < p.N; cc += 16) {
                    uint32_t v[16];
                    tmem_ld_32x16(t_row + cc, v);
                    tmem_ld_wait();
                    float f[16];
#pragma unroll
                    for (int k = 0; k < 16; ++k) {
                        f[k] = __fmul_rn(__int2float_rn((int)v[k]), sc);
                        if (p.bias) f[k] = __fadd_rn(f[k], p.bias[(long long)c.node * p.bias_stride + cc + k]);
                    }
                    if (p.addend && valid) {
                        const float4 *ad = reinterpret_cast<const float4 *>(p.addend + pix * p.N + cc);
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const float4 a4 = ad[k];
                            f[4 * k] = __fadd_rn(f[4 * k], a4.x); f[4 * k + 1] = __fadd_rn(f[4 * k + 1], a4.y);
                            f[4 * k + 2] = __fadd_rn(f[4 * k + 2], a4.z); f[4 * k + 3] = __fadd_rn(f[4 * k + 3], a4.w);
                        }
                    }
                    const int g = cc / inner, k0 = (cc % inner) >> 2;
                    float4 *grow = reinterpret_cast<float4 *>(ot + ((size_t)g * 128 + row) * inner * 4);
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        grow[(uint32_t)(k0 + k) ^ sw] = make_float4(f[4 * k], f[4 * k + 1], f[4 * k + 2], f[4 * k + 3]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&ctl->tmem_empty[acc]));
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    for (int g = 0; g * inner < p.N; ++g)
                        tma_store_5d(&mapY, smem_u32(ot + ((size_t)g * 128 + q * 32) * inner * 4), g * inner,
                                     c.tw * kTileW, c.th * kTileH + q * (32 / kTileW), c.b, c.node);
                    tma_store_commit();
                }
                continue;
            }
            for (int cc = 0; cc < p.N; cc += 16) {
                uint32_t v[16];
                tmem_ld_32x16(t_row + cc, v);
                tmem_ld_wait();
                if (valid) {
                    const long long o = pix * p.N + cc;
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
                            if (p.bias) f[k] = __fadd_rn(f[k], p.bias[(long long)c.node * p.bias_stride + cc + k]);
                            if (p.addend) f[k] = __fadd_rn(f[k], p.addend[o + k]);
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
        if (p.tma_out && lane == 0) tma_store_wait_all();    // this warp's rows in shared memory have been read and written out
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, p.tmem_cols); }
}

// LPDT_FORCE_HALO=1 takes the halo kernel wherever it is valid (used by the parity tests).
static bool halo_forced() {
    static int forced = -1;
    if (forced < 0) { const char *e = getenv("LPDT_FORCE_HALO"); forced = (e && e[0] == '1') ? 1 : 0; }
    return forced == 1;
}

static int halo_pow2(int v) { int p = 32; while (p < v) p <<= 1; return p; }

bool halo_supported(const lpdt_conv_desc &d, int mode) {
    if (d.stride != 1) return false;
    const int Kc = mode == 0 ? d.Cin : d.Cout, N = mode == 0 ? d.Cout : d.Cin;
    if (Kc % 16 || Kc > 128 || (Kc > 16 && Kc % 32) || N % 16 || N > 256) return false;
    if (d.S > 9 || d.R > 64 || d.R * d.S > kHaloMaxTaps) return false;
    // measured: with several chunks the 16-byte TMA rows only pay off for up to 64 channels on maps at
    // least one tile (16 rows) high; elsewhere the general kernel is as fast or faster
    const int Hm = mode == 0 ? conv_out(d.H, d.pad, d.R, 1) : d.H;
    if (Kc > 16 && (Kc > 64 || Hm < 16) && !halo_forced()) return false;
    const int nslices = d.R * d.S * (Kc / 16);
    if ((nslices + 1) / 2 > kHaloMaxMma) return false;
    if ((nslices + 1) * N * 16 > 72 * 1024) return false;
    if ((8 + d.S - 1) * (16 + d.R - 1) >= 0x3FFF) return false;
    if (d.pad > 100) return false;
    return encode_tiled_fn() != nullptr;
}

lpdt_status tc_pix_halo(const lpdt_conv_desc &d, int mode, const int8_t *A, const float *s1, const int8_t *Wq,
                        const float *s2, const float *bias, int64_t bias_stride, float *Y, int32_t *Yacc,
                        int32_t *dev_status, cudaStream_t st, bool uns, const float *addend) {
    const int Ho = conv_out(d.H, d.pad, d.R, 1), Wo = conv_out(d.W, d.pad, d.S, 1);
    HaloParams p = {};
    p.addend = addend;
    p.mode = mode; p.uns = uns ? 1 : 0; p.nodes = d.nodes; p.B = d.B;
    p.N = mode == 0 ? d.Cout : d.Cin;
    p.Hm = mode == 0 ? Ho : d.H; p.Wm = mode == 0 ? Wo : d.W;
    const int Ha = mode == 0 ? d.H : Ho, Wa = mode == 0 ? d.W : Wo;     // image of operand A
    p.PH = kTileH + d.R - 1; p.PW = kTileW + d.S - 1;
    // tap (r, s) reads operand pixel (m + dh, m + dw): dh = r - pad forward, pad - r backward
    p.org_h = mode == 0 ? -d.pad : d.pad - (d.R - 1);
    p.org_w = mode == 0 ? -d.pad : d.pad - (d.S - 1);
    p.ntaps = d.R * d.S;
    const int Kc = mode == 0 ? d.Cin : d.Cout;
    p.cpt = Kc / 16; p.nslices = p.ntaps * p.cpt;
    const int chunk16 = p.PH * p.PW;                    // one chunk's halo image, in 16-byte rows
    unsigned short off16[kHaloMaxTaps];
    for (int i = 0; i < p.ntaps; ++i) {
        // ascending halo offset: forward walks (r, s) up, backward walks them down
        const int a = i / d.S, b = i % d.S;
        const int r = mode == 0 ? a : d.R - 1 - a, s = mode == 0 ? b : d.S - 1 - b;
        off16[i] = (unsigned short)(a * p.PW + b);
        p.wtap[i] = (signed char)(r * d.S + s);
    }
    p.n_mma = (p.nslices + 1) / 2;
    for (int m = 0; m < p.n_mma; ++m) {
        const int k0 = 2 * m, k1 = 2 * m + 1;            // K slices (tap, chunk) of this MMA
        const int o0 = (k0 % p.cpt) * chunk16 + off16[k0 / p.cpt];
        p.a_off16[m] = (unsigned short)o0;
        if (k1 < p.nslices) p.a_lbo16[m] = (unsigned short)((k1 % p.cpt) * chunk16 + off16[k1 / p.cpt] - o0);
        else p.a_lbo16[m] = 0xFFFFu;
    }
    p.tilesH = (int)ceil_div(p.Hm, kTileH); p.tilesW = (int)ceil_div(p.Wm, kTileW);
    p.halo_bytes = (int)align_up((size_t)p.PH * p.PW * 16 * p.cpt, 128);
    p.wres_bytes = (int)align_up((size_t)(p.nslices + 1) * p.N * 16, 128);
    if (15 * p.PW * 16 + 128 > kZeroBytes) return LPDT_ERR_UNSUPPORTED;
    // CTAs per SM: these tiles are short dependent chains (one TMA box, a few MMAs, a 128 x N epilogue), so
    // several resident CTAs hide each other's latencies.  As many as leave every CTA at least four stages
    // and fit TMEM (512 columns per SM): shared memory is sized so that no further CTA becomes resident and
    // a TMEM allocation never has to wait.
    // TMEM accumulators: as many tiles in flight between the MMA warp and the epilogue warps as 128 columns
    // hold (8 at N = 16, 4 at N = 32, 2 from N = 64 on), so that the MMA warp does not wait for the epilogue's
    // round trip on these short tiles
    p.nacc_log2 = p.N <= 16 ? 3 : p.N <= 32 ? 2 : 1;
    p.tmem_cols = halo_pow2((1 << p.nacc_log2) * p.N);
    // fp32 result through shared memory and bulk tensor stores (not when the raw accumulators are asked for)
    p.tma_out = (Y && !Yacc && aligned(Y, 16)) ? 1 : 0;
    p.out_inner = p.N % 32 == 0 ? 32 : 16;
    const int out_bytes = p.tma_out ? 2 * 128 * p.N * 4 + 1024 : 0;          // + slack to reach a 1024-byte boundary
    int per_sm = 4, stages = 0;
    for (;; --per_sm) {
        const int budget = (224 * 1024) / per_sm - 2048;
        stages = (budget - 1024 - p.wres_bytes - kZeroBytes - out_bytes) / p.halo_bytes;
        if (stages > 8) stages = 8;
        if (per_sm == 1 || (stages >= 4 && per_sm * p.tmem_cols <= 512)) break;
    }
    if (stages < 2) return LPDT_ERR_UNSUPPORTED;
    p.stages = stages;
    p.w_rows_per_node = d.Cout;
    p.Y = Y; p.Yacc = Yacc; p.s1 = s1; p.s2 = s2; p.bias = bias; p.bias_stride = bias_stride;
    p.dev_status = dev_status;
    CUtensorMap mA, mW, mY;
    if (p.tma_out) {
        if (!make_map_out_f32(&mY, Y, d.nodes, d.B, p.Hm, p.Wm, p.N, p.out_inner, 32 / kTileW, kTileW)) return LPDT_ERR_CUDA;
    } else {
        mY = CUtensorMap{};
    }
    if (p.cpt > 1) {   // 16-byte chunk rows; the chunk index is the outermost box dimension
        uint64_t dims[5] = {16, (uint64_t)Wa, (uint64_t)Ha, (uint64_t)d.nodes * d.B, (uint64_t)p.cpt};
        uint64_t strides[4] = {(uint64_t)Kc, (uint64_t)Wa * Kc, (uint64_t)Ha * Wa * Kc, 16};
        uint32_t box[5] = {16, (uint32_t)p.PW, (uint32_t)p.PH, 1, (uint32_t)p.cpt};
        if (!make_map_u8(&mA, A, 5, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return LPDT_ERR_UNSUPPORTED;
    } else {   // operand A with (channel, width) merged into one contiguous row of 16*Wa bytes
        uint64_t dims[4] = {(uint64_t)Wa * 16, (uint64_t)Ha, (uint64_t)d.B, (uint64_t)d.nodes};
        uint64_t strides[3] = {(uint64_t)Wa * 16, (uint64_t)Ha * Wa * 16, (uint64_t)d.B * Ha * Wa * 16};
        uint32_t box[4] = {(uint32_t)p.PW * 16, (uint32_t)p.PH, 1, 1};
        if (!make_map_u8(&mA, A, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return LPDT_ERR_CUDA;
    }
    {   // weights [nodes*Cout][taps][Cin]: forward box = N rows of one tap, backward = 16 rows x 16 columns
        uint64_t dims[3] = {(uint64_t)d.Cin, (uint64_t)p.ntaps, (uint64_t)d.nodes * d.Cout};
        uint64_t strides[2] = {(uint64_t)d.Cin, (uint64_t)p.ntaps * d.Cin};
        uint32_t box[3] = {16, 1, (uint32_t)(mode == 0 ? p.N : 16)};
        if (!make_map_u8(&mW, Wq, 3, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE)) return LPDT_ERR_CUDA;
    }
    size_t smem = 1024 + (size_t)p.wres_bytes + (size_t)p.stages * p.halo_bytes + kZeroBytes + out_bytes;
    const size_t smem_floor = (size_t)(228 * 1024) / (per_sm + 1);     // keeps the (per_sm + 1)-th CTA out
    if (smem < smem_floor) smem = smem_floor;
    static PerDeviceOnce attr;
    int dev;
    if (attr.pending(&dev)) {
        LPDT_CUDA(cudaFuncSetAttribute(conv_halo16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
        attr.mark(dev);
    }
    const long long tiles = (long long)p.nodes * p.B * p.tilesH * p.tilesW;
    if (tiles > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    const int grid = (int)(tiles < (long long)kNumSMs * per_sm ? tiles : (long long)kNumSMs * per_sm);
    g_last_kernel = "lpdt::tc::conv_halo16_kernel";
    launch_k(conv_halo16_kernel, grid, kHaloThreads, smem, st, mA, mW, mY, p);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

}  // namespace tc
}  // namespace lpdt
