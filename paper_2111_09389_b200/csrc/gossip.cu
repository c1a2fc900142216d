// Gossip step of CHOCO-SGD (Algorithm 3) for all simulated nodes at once:
// exact top-k selection of x_half - x_hat per (node, segment) by radix select
// on the magnitude bits, then one fused streaming pass that updates the public
// copies and mixes.  The mix pass is HBM-bound: per parameter and node it reads
// x_half and x_hat and writes x_hat and x (16 bytes); the neighbours' updated
// x_hat values are exchanged through shared memory, never re-read from HBM.
#include "common.cuh"

namespace lpdt {

constexpr int kMaxSeg = 128;
constexpr int kMaxNodes = 64;

struct SegTable {
    int32_t n_seg;
    int32_t plus;            // 0: keys are |x_half - state| (CHOCO public copy); 1: |x_half + state| (Deep-Squeeze error buffer)
    int64_t off[kMaxSeg + 1];
    int64_t k[kMaxSeg];
};

struct SelectOut {       // per (node, segment)
    uint32_t thr;        // magnitude bits of the k-th largest |delta|
    uint32_t dense;      // 1: keep everything
    int64_t cut;         // ties (== thr) are kept only below this index
};

template <int V> struct VecIO;
template <> struct VecIO<4> {
    static __device__ __forceinline__ void ld(const float *p, float (&o)[4]) {
        float4 t = *reinterpret_cast<const float4 *>(p); o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
    }
    static __device__ __forceinline__ void st(float *p, const float (&o)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(o[0], o[1], o[2], o[3]);
    }
};
template <> struct VecIO<2> {
    static __device__ __forceinline__ void ld(const float *p, float (&o)[2]) {
        float2 t = *reinterpret_cast<const float2 *>(p); o[0] = t.x; o[1] = t.y;
    }
    static __device__ __forceinline__ void st(float *p, const float (&o)[2]) {
        *reinterpret_cast<float2 *>(p) = make_float2(o[0], o[1]);
    }
};
template <> struct VecIO<1> {
    static __device__ __forceinline__ void ld(const float *p, float (&o)[1]) { o[0] = *p; }
    static __device__ __forceinline__ void st(float *p, const float (&o)[1]) { *p = o[0]; }
};

__device__ __forceinline__ uint32_t mag_bits(float xh, float state, int plus) {
    return __float_as_uint(plus ? __fadd_rn(xh, state) : __fsub_rn(xh, state)) & 0x7fffffffu;
}

// Index just past the need-th key equal to thr in [lo, hi), walking in index order (whole CTA;
// every thread returns the same value; -1 if there are fewer than need such keys).
__device__ long long ordered_cut(const float *__restrict__ xh, const float *__restrict__ xq, int64_t lo, int64_t hi,
                                 uint32_t thr, long long need, int plus) {
    __shared__ long long s_run, s_cut;
    __shared__ int warp_cnt[32];
    __syncthreads();
    if (threadIdx.x == 0) { s_run = 0; s_cut = -1; }
    __syncthreads();
    for (int64_t base = lo; base < hi; base += blockDim.x) {
        const int64_t e = base + threadIdx.x;
        const int flag = (e < hi) && (mag_bits(xh[e], xq[e], plus) == thr);
        const int cnt = __syncthreads_count(flag);
        const long long run = s_run;
        if (run + cnt >= need) {
            // the cut lies in this stretch: rank the flags with a ballot scan
            const unsigned bal = __ballot_sync(0xffffffffu, flag);
            const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
            if (lane == 0) warp_cnt[warp] = __popc(bal);
            __syncthreads();
            int before = 0;
            for (int w = 0; w < warp; ++w) before += warp_cnt[w];
            const int rank = before + __popc(bal & ((1u << lane) - 1u));   // ties before me in the stretch
            if (flag && run + rank + 1 == need) s_cut = e + 1;
            __syncthreads();
            break;
        }
        __syncthreads();
        if (threadIdx.x == 0) s_run = run + cnt;
        __syncthreads();
    }
    __syncthreads();
    return s_cut;
}

// A segment takes the multi-CTA path when it is long and the selection is not trivial.
constexpr int64_t kBigMin = 32768;     // shortest segment split over several CTAs
constexpr int kChunk = 16384;          // elements per CTA on that path
__device__ __host__ __forceinline__ bool is_big(int64_t len, int64_t k) { return len >= kBigMin && k > 0 && k < len; }

// Block-wide radix select over n 32-bit keys given by key(e), e in [0, n), 8 bits per pass, most
// significant first.  The keys agree on their bits above `free_bits` (prefix0 holds them), so only the
// low free_bits are scanned; with SKIP_ZERO, keys equal to 0 are left out.  Returns in every thread the
// need-th largest key (need at least 1 and at most the number of keys scanned), how many keys equal to
// it are among the need largest (*need_out) and how many keys equal it in all (*eq_out).
template <bool SKIP_ZERO, typename KeyFn>
__device__ uint32_t radix_select(int64_t n, KeyFn key, long long need, int free_bits, uint32_t prefix0,
                                 long long *need_out, long long *eq_out) {
    __shared__ unsigned int hist[256];
    __shared__ uint32_t s_prefix, s_mask;
    __shared__ long long s_need;      // how many more keys to take inside the current prefix
    __shared__ long long s_eq;        // population of the chosen bucket
    __syncthreads();
    if (threadIdx.x == 0) {
        s_mask = free_bits >= 32 ? 0u : ~((1u << free_bits) - 1u);
        s_prefix = prefix0 & s_mask;
        s_need = need;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31;
    for (int top = free_bits; top > 0;) {
        const int w = top >= 8 ? 8 : top, shift = top - w;
        const uint32_t dmask = (1u << w) - 1u;
        for (int i = threadIdx.x; i < 256; i += blockDim.x) hist[i] = 0;
        __syncthreads();
        const uint32_t prefix = s_prefix, mask = s_mask;
        // eight independent loads per thread.  Consecutive hits of a thread that fall into the same bin are
        // counted in a register and added once: in the first passes one or two bins (the common exponents)
        // take nearly every key, and per-key atomics would queue up on those few shared-memory words.
        uint32_t run_bin = 0; unsigned run_cnt = 0;
        for (int64_t base = 0; base < n; base += 8 * (int64_t)blockDim.x) {
            uint32_t k[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int64_t eu = base + u * (int64_t)blockDim.x + threadIdx.x;
                k[u] = eu < n ? key(eu) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int64_t eu = base + u * (int64_t)blockDim.x + threadIdx.x;
                const bool hit = eu < n && !(SKIP_ZERO && k[u] == 0u) && (k[u] & mask) == prefix;
                if (!hit) continue;
                const uint32_t bin = (k[u] >> shift) & dmask;
                if (run_cnt && bin == run_bin) { ++run_cnt; continue; }
                if (run_cnt) atomicAdd(&hist[run_bin], run_cnt);
                run_bin = bin; run_cnt = 1;
            }
        }
        if (run_cnt) atomicAdd(&hist[run_bin], run_cnt);
        __syncthreads();
        if (threadIdx.x < 32) {
            // bucket of the need-th largest key: lane l owns bins [8l, 8l+8); suffix sums across lanes by shuffles
            long long mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine += hist[lane * 8 + j];
            long long incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const long long v = __shfl_down_sync(0xffffffffu, incl, o);
                if (lane + o < 32) incl += v;
            }
            const long long above = incl - mine, nd0 = s_need;
            if (above < nd0 && nd0 <= above + mine) {
                long long nd = nd0 - above;
                int bsel = lane * 8 + 7;
                for (; bsel > lane * 8; --bsel) {
                    if ((long long)hist[bsel] >= nd) break;
                    nd -= hist[bsel];
                }
                s_need = nd;                     // 1 <= nd <= hist[bsel]
                s_eq = hist[bsel];
                s_prefix = prefix | ((uint32_t)bsel << shift);
                s_mask = mask | (dmask << shift);
            }
        }
        __syncthreads();
        top = shift;
    }
    *need_out = s_need; *eq_out = s_eq;
    return s_prefix;
}

// One CTA selects over a whole segment: the k-th largest magnitude by radix select, then an ordered
// pass that places the tie cut.  The path of short segments, and of long ones whose candidates did
// not fit (below).
__device__ void select_whole_segment(const float *__restrict__ xh, const float *__restrict__ xq, int64_t lo, int64_t hi,
                                     int64_t k, int plus, SelectOut *o) {
    long long need, eq;
    const uint32_t thr = radix_select<false>(hi - lo, [&](int64_t e) { return mag_bits(xh[lo + e], xq[lo + e], plus); },
                                             (long long)k, 32, 0u, &need, &eq);
    if (eq == need) {        // every tie is taken
        if (threadIdx.x == 0) { o->thr = thr; o->dense = 0; o->cut = hi; }
        return;
    }
    const long long cut = ordered_cut(xh, xq, lo, hi, thr, need, plus);
    if (threadIdx.x == 0) { o->thr = thr; o->dense = 0; o->cut = cut; }
}

// ---- long segments: a sampled threshold, one streaming pass, a selection over the candidates ----
// Sample (big_sample_kernel): 1/64 of the segment, read as runs of eight consecutive parameters, goes into
// a histogram of the top 12 magnitude bits (exponent and four mantissa bits: buckets 1/16 of an octave
// wide); the CTA that finishes last walks it from the top and picks a bucket that, by the sample, has
// comfortably more than k keys at or above it.  Collect (big_collect_kernel): the one pass over the
// segment copies every key at or above that bucket, with its position, into a candidate list and counts
// them exactly.  Select (one CTA per segment): if the exact count reached k, the k largest keys are all
// in the list, and the threshold and the tie cut are found there (1-2 % of the data).  The sample only
// steers: when the count falls short of k, or the candidates outgrow the list (1/8 of the segment: near-
// constant magnitudes), the exact whole-segment path takes over, so the result never depends on the sample.
struct BigList {
    int32_t n;
    int32_t id[kMaxSeg];               // segment index
    int32_t chunk_base[kMaxSeg + 1];   // prefix sums of the chunk counts
    int64_t cand_base[kMaxSeg + 1];    // prefix sums of the candidate capacities
};
constexpr int kTopBins = 4096;
// zeroed per call.  h0: histogram of the sample; h1: exact histogram of the collected keys (same 12 bits);
// cand_count: keys at or above the chosen bucket
struct BigCtl { uint32_t h0[kTopBins], h1[kTopBins]; uint32_t ticket, cand_count, sampled, pad; };
struct BigState { uint32_t prefix; uint32_t sampled; };    // lowest magnitude bits of the chosen bucket; keys sampled
struct __align__(8) Cand { uint32_t key, pos; };    // magnitude bits, position inside the segment

__device__ __host__ __forceinline__ int64_t cand_capacity(int64_t len) { return len / 8 + 4096; }

// Walk a histogram from its top bin: the bucket holding the need-th largest key, the keys still
// needed inside it and its population.  Whole CTA (its thread count divides nbins); same result in every thread.
// The histogram was filled by other CTAs' atomics: read it from L2.
__device__ void pick_bucket(const uint32_t *hist, int nbins, long long need, int *bucket,
                            long long *need_out, long long *eq_out) {
    __shared__ long long wtot[32];
    __shared__ long long res[3];
    const int t = threadIdx.x, lane = t & 31, warp = t >> 5, nwarps = blockDim.x >> 5, per = nbins / blockDim.x;
    long long mine = 0;
    for (int b = 0; b < per; ++b) mine += __ldcg(hist + t * per + b);
    // suffix sums over the 256 slices: inside the warp by shuffles, across warps through shared memory
    long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const long long v = __shfl_down_sync(0xffffffffu, incl, o);
        if (lane + o < 32) incl += v;
    }
    __syncthreads();
    if (lane == 0) wtot[warp] = incl;
    __syncthreads();
    long long above = incl - mine;
    for (int w = warp + 1; w < nwarps; ++w) above += wtot[w];
    if (above < need && need <= above + mine) {
        long long n = need - above;
        int b = t * per + per - 1;
        for (; b > t * per; --b) {
            const long long hb = __ldcg(hist + b);
            if (hb >= n) break;
            n -= hb;
        }
        res[0] = b; res[1] = n; res[2] = __ldcg(hist + b);
    }
    __syncthreads();
    *bucket = (int)res[0]; *need_out = res[1]; *eq_out = res[2];
}

constexpr int kTopShift = 19;          // the histogram keys on magnitude bits 30..19
__device__ __forceinline__ int64_t ceil_div_dev(int64_t a, int64_t b) { return (a + b - 1) / b; }

constexpr int kSampleRun = 8;                 // consecutive parameters per sampled run
constexpr int kSampleEvery = 64;              // one run per kSampleRun * kSampleEvery parameters
constexpr int64_t kSampleChunk = 1 << 17;     // parameters per CTA of the sample launch: eight runs per group of eight threads

__global__ void __launch_bounds__(256)
big_sample_kernel(const float *__restrict__ x_half, const float *__restrict__ x_hat, int64_t d, SegTable seg,
                  BigList big, BigCtl *__restrict__ ctl, BigState *__restrict__ state) {
    pdl_enter();
    const int bi = blockIdx.y, node = blockIdx.z, s = big.id[bi], plus = seg.plus;
    const int64_t lo = seg.off[s], hi = seg.off[s + 1];
    const int64_t c0 = lo + (int64_t)blockIdx.x * kSampleChunk;
    if (c0 >= hi) return;
    const int64_t c1 = (c0 + kSampleChunk < hi) ? c0 + kSampleChunk : hi;
    BigCtl *h = ctl + (int64_t)node * big.n + bi;
    const float *xh = x_half + (int64_t)node * d, *xq = x_hat + (int64_t)node * d;
    __shared__ unsigned int sh[kTopBins];
    __shared__ unsigned int s_ticket, s_taken;
    for (int i = threadIdx.x; i < kTopBins; i += blockDim.x) sh[i] = 0;
    if (threadIdx.x == 0) s_taken = 0;
    __syncthreads();
    // thread t of a group of eight reads parameter t of a run: 32 contiguous bytes per run and array
    const int64_t span = (int64_t)kSampleRun * kSampleEvery;
    unsigned taken = 0;
    const int64_t r0 = c0 + (int64_t)(threadIdx.x / kSampleRun) * span + (threadIdx.x % kSampleRun);
    const int64_t rstep = (int64_t)(blockDim.x / kSampleRun) * span;
    constexpr int kU = (int)(kSampleChunk / ((256 / kSampleRun) * kSampleRun * kSampleEvery));     // runs per thread group
    float va[kU], vb[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) {                   // every load of the thread in flight at once
        const int64_t e = r0 + u * rstep;
        if (e < c1) { va[u] = xh[e]; vb[u] = xq[e]; }
    }
#pragma unroll
    for (int u = 0; u < kU; ++u)
        if (r0 + u * rstep < c1) { atomicAdd(&sh[mag_bits(va[u], vb[u], plus) >> kTopShift], 1u); ++taken; }
    atomicAdd(&s_taken, taken);
    __syncthreads();
    for (int i = threadIdx.x; i < kTopBins; i += blockDim.x)
        if (sh[i]) atomicAdd(&h->h0[i], sh[i]);
    if (threadIdx.x == 0) atomicAdd(&h->sampled, s_taken);
    // last CTA of this (node, segment): every chunk's counts have landed
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_ticket = atomicAdd(&h->ticket, 1u);
    __syncthreads();
    const unsigned nchunks = (unsigned)ceil_div_dev(hi - lo, kSampleChunk);
    if (s_ticket != nchunks - 1) return;
    __threadfence();
    // keys the sample must show at or above the bucket: the sampled share of k, a tenth more, and four
    // standard deviations of the sampled count
    const double m = (double)__ldcg(&h->sampled), f = m / (double)(hi - lo), fk = f * (double)seg.k[s];
    long long target = (long long)(1.10 * fk + 4.0 * sqrt(fk) + 8.0);
    int b = 0; long long need, eq;
    if (target <= (long long)m) pick_bucket(h->h0, kTopBins, target, &b, &need, &eq);
    if (threadIdx.x == 0) {
        BigState nx;
        nx.prefix = (uint32_t)b << kTopShift;
        nx.sampled = (uint32_t)m;
        state[(int64_t)node * big.n + bi] = nx;
    }
}

// Copy every key at or above the chosen bucket, with its position, into the (node, segment)'s candidate
// list, and count them all (the count keeps running past the list's capacity; writes stop there).
// Matches are staged in shared memory and flushed with one reservation per CTA; the order inside the
// list is arbitrary (the selection over it does not depend on it).
constexpr int kStage = 2048;
__global__ void __launch_bounds__(256)
big_collect_kernel(const float *__restrict__ x_half, const float *__restrict__ x_hat, int64_t d, SegTable seg,
                   BigList big, BigCtl *__restrict__ ctl, const BigState *__restrict__ state,
                   Cand *__restrict__ cands, int64_t cand_per_node, unsigned int *__restrict__ amax_bits,
                   int chunk /*elements per CTA*/) {
    pdl_enter();
    const int bi = blockIdx.y, node = blockIdx.z, s = big.id[bi], plus = seg.plus;
    const int64_t lo = seg.off[s], hi = seg.off[s + 1];
    const int64_t c0 = lo + (int64_t)blockIdx.x * chunk;
    if (c0 >= hi) return;
    const int64_t c1 = (c0 + chunk < hi) ? c0 + chunk : hi;
    const BigState stt = state[(int64_t)node * big.n + bi];
    const unsigned cap = (unsigned)cand_capacity(hi - lo);
    BigCtl *h = ctl + (int64_t)node * big.n + bi;
    Cand *list = cands + (int64_t)node * cand_per_node + big.cand_base[bi];
    const float *xh = x_half + (int64_t)node * d, *xq = x_hat + (int64_t)node * d;
    const uint32_t bucket = stt.prefix >> kTopShift;
    __shared__ Cand stage[kStage];
    __shared__ unsigned int sh1[kTopBins];       // this CTA's share of the exact histogram of the collected keys
    __shared__ unsigned int s_cnt, s_base;
    for (int i = threadIdx.x; i < kTopBins; i += blockDim.x) sh1[i] = 0;
    if (threadIdx.x == 0) s_cnt = 0;
    __syncthreads();
    uint32_t kmax = 0;          // largest magnitude of the chunk: the range of the segment's 8-bit message
    auto consider = [&](float a, float b, int64_t eu) {
        const uint32_t key = mag_bits(a, b, plus);
        kmax = key > kmax ? key : kmax;
        if ((key >> kTopShift) >= bucket) {
            atomicAdd(&sh1[key >> kTopShift], 1u);
            Cand c; c.key = key; c.pos = (uint32_t)(eu - lo);
            const unsigned slot = atomicAdd(&s_cnt, 1u);
            if (slot < kStage) stage[slot] = c;
            else {                                             // a dense stretch: straight to the list
                const unsigned at = atomicAdd(&h->cand_count, 1u);
                if (at < cap) list[at] = c;
            }
        }
    };
    // 16-byte loads, four pairs in flight per thread, where both rows sit on 16-byte boundaries; scalar loads
    // for the ragged ends (or the whole chunk)
    int64_t v0 = c0, v1 = c0;
    if ((((uintptr_t)(xh + c0) ^ (uintptr_t)(xq + c0)) & 15) == 0) {
        v0 = c0 + (int64_t)(((16 - ((uintptr_t)(xh + c0) & 15)) & 15) >> 2);
        if (v0 > c1) v0 = c1;
        v1 = v0 + ((c1 - v0) & ~(int64_t)3);
    }
    for (int64_t e = c0 + threadIdx.x; e < v0; e += blockDim.x) consider(xh[e], xq[e], e);
    {
        const float4 *h4 = reinterpret_cast<const float4 *>(xh + v0), *q4 = reinterpret_cast<const float4 *>(xq + v0);
        const int64_t n4 = (v1 - v0) >> 2;
        for (int64_t i = threadIdx.x; i < n4; i += 4 * (int64_t)blockDim.x) {
            float4 a[4], b[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t iu = i + u * (int64_t)blockDim.x;
                if (iu < n4) { a[u] = __ldg(h4 + iu); b[u] = __ldg(q4 + iu); }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int64_t iu = i + u * (int64_t)blockDim.x;
                if (iu < n4) {
                    const int64_t e = v0 + 4 * iu;
                    consider(a[u].x, b[u].x, e); consider(a[u].y, b[u].y, e + 1);
                    consider(a[u].z, b[u].z, e + 2); consider(a[u].w, b[u].w, e + 3);
                }
            }
        }
    }
    for (int64_t e = v1 + threadIdx.x; e < c1; e += blockDim.x) consider(xh[e], xq[e], e);
    __syncthreads();
    if (amax_bits) {            // the same value the range pass of the 8-bit messages would find
        for (int o = 16; o > 0; o >>= 1) { const uint32_t t = __shfl_xor_sync(0xffffffffu, kmax, o); kmax = t > kmax ? t : kmax; }
        if ((threadIdx.x & 31) == 0 && kmax) atomicMax(amax_bits + (int64_t)node * seg.n_seg + s, kmax);
    }
    for (int i = bucket + threadIdx.x; i < kTopBins; i += blockDim.x)
        if (sh1[i]) atomicAdd(&h->h1[i], sh1[i]);
    const unsigned n = s_cnt < kStage ? s_cnt : kStage;
    if (n == 0) return;
    if (threadIdx.x == 0) s_base = atomicAdd(&h->cand_count, n);
    __syncthreads();
    for (unsigned i = threadIdx.x; i < n; i += blockDim.x)
        if (s_base + i < cap) list[s_base + i] = stage[i];
}

// Threshold and tie cut of a long segment from its candidate list (one CTA).  The list holds every key
// at or above a bucket and at least k of them, so its k-th largest is the segment's k-th largest; if only
// some of the keys equal to it are taken, those at the lowest positions are: the cut follows the
// need-th smallest position among them.
__device__ void select_from_candidates(const Cand *__restrict__ list, int64_t n_cand, int64_t k, const uint32_t *h1,
                                       int64_t lo, int64_t hi, SelectOut *o, uint32_t *s_keys, int key_cap) {
    // the collect pass left the exact histogram of the candidates' top 12 bits: the bucket of the k-th largest
    // key comes from it without a scan, and only the 19 bits below are searched
    int b1; long long need1, eq1;
    pick_bucket(h1, kTopBins, (long long)k, &b1, &need1, &eq1);
    long long need, eq;
    uint32_t thr;
    if (eq1 <= (long long)key_cap) {
        // The bucket's keys (their exact number is known) fit the shared-memory buffer: one pass over the list
        // copies them there, and the radix passes run over shared memory instead of re-reading the list.
        __shared__ unsigned int s_n;
        if (threadIdx.x == 0) s_n = 0;
        __syncthreads();
        const unsigned long long *l64 = reinterpret_cast<const unsigned long long *>(list);
        for (int64_t base = 0; base < n_cand; base += 8 * (int64_t)blockDim.x) {
            unsigned long long c[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int64_t eu = base + u * (int64_t)blockDim.x + threadIdx.x;
                c[u] = eu < n_cand ? __ldg(l64 + eu) : 0ull;       // {key, pos}: the key is the low word
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int64_t eu = base + u * (int64_t)blockDim.x + threadIdx.x;
                const uint32_t key = (uint32_t)c[u];
                if (eu < n_cand && (int)(key >> kTopShift) == b1) {
                    const unsigned slot = atomicAdd(&s_n, 1u);
                    if (slot < (unsigned)key_cap) s_keys[slot] = key;
                }
            }
        }
        __syncthreads();
        const int64_t n_in = s_n < (unsigned)key_cap ? s_n : key_cap;      // equals eq1
        thr = radix_select<false>(n_in, [&](int64_t e) { return s_keys[e]; }, need1, kTopShift,
                                  (uint32_t)b1 << kTopShift, &need, &eq);
    } else {
        thr = radix_select<false>(n_cand, [&](int64_t e) { return list[e].key; }, need1, kTopShift,
                                  (uint32_t)b1 << kTopShift, &need, &eq);
    }
    if (eq == need) {
        if (threadIdx.x == 0) { o->thr = thr; o->dense = 0; o->cut = hi; }
        return;
    }
    long long n2, e2;      // ties keyed by descending position (never 0); the other candidates are skipped
    const uint32_t inv = radix_select<true>(n_cand,
                                            [&](int64_t e) { return list[e].key == thr ? 0xFFFFFFFFu - list[e].pos : 0u; },
                                            need, 32, 0u, &n2, &e2);
    if (threadIdx.x == 0) { o->thr = thr; o->dense = 0; o->cut = lo + (int64_t)(0xFFFFFFFFu - inv) + 1; }
}

// Row i of the mixing matrix as a compact list of its non-zero entries (j ascending), built once
// per call by one extra CTA of the select launch.  Layout in the workspace: cnt[nodes] (int32),
// then idx[nodes][nodes] (int32), then val[nodes][nodes] (fp32).
__device__ void build_rows(const float *__restrict__ Wmix, int nodes, int32_t *__restrict__ tab) {
    int32_t *cnt = tab, *idx = tab + nodes;
    float *val = reinterpret_cast<float *>(tab + nodes + nodes * nodes);
    for (int i = threadIdx.x; i < nodes; i += blockDim.x) {
        int c = 0;
        for (int j = 0; j < nodes; ++j) {
            const float w = Wmix[i * nodes + j];
            if (w != 0.f) { idx[i * nodes + c] = j; val[i * nodes + c] = w; ++c; }
        }
        cnt[i] = c;
    }
}

// 8-bit messages: max |x_half - x_hat| per (node, segment), as float bits through atomicMax (zeroed by
// the launcher).  Block = one chunk of one node's parameters; a chunk may straddle segments.
__global__ void __launch_bounds__(256)
delta_amax_kernel(const float *__restrict__ x_half, const float *__restrict__ x_hat, int64_t d, SegTable seg,
                  unsigned int *__restrict__ amax_bits) {
    pdl_enter();
    const int node = blockIdx.y, plus = seg.plus;
    const int64_t c0 = (int64_t)blockIdx.x * kChunk, c1 = (c0 + kChunk < d) ? c0 + kChunk : d;
    const float *xh = x_half + (int64_t)node * d, *xq = x_hat + (int64_t)node * d;
    int a = 0, b = seg.n_seg;
    while (b - a > 1) { const int m = (a + b) >> 1; if (seg.off[m] <= c0) a = m; else b = m; }
    __shared__ unsigned int s_m[8];
    for (int s = a; s < seg.n_seg && seg.off[s] < c1; ++s) {
        const int64_t lo = seg.off[s] > c0 ? seg.off[s] : c0, hi = seg.off[s + 1] < c1 ? seg.off[s + 1] : c1;
        unsigned int m = 0;
        // 16-byte loads, four pairs in flight per thread, over the part of the span where both rows sit on
        // 16-byte boundaries; scalar loads for the ragged ends (or the whole span)
        int64_t v0 = lo, v1 = lo;
        if ((((uintptr_t)(xh + lo) ^ (uintptr_t)(xq + lo)) & 15) == 0) {
            v0 = lo + (int64_t)(((16 - ((uintptr_t)(xh + lo) & 15)) & 15) >> 2);
            if (v0 > hi) v0 = hi;
            v1 = v0 + ((hi - v0) & ~(int64_t)3);
        }
        for (int64_t e = lo + threadIdx.x; e < v0; e += blockDim.x) {
            const unsigned int key = mag_bits(xh[e], xq[e], plus);
            m = key > m ? key : m;
        }
        {
            const float4 *h4 = reinterpret_cast<const float4 *>(xh + v0), *q4 = reinterpret_cast<const float4 *>(xq + v0);
            const int64_t n4 = (v1 - v0) >> 2;
            for (int64_t i = threadIdx.x; i < n4; i += 4 * (int64_t)blockDim.x) {
                float4 a[4], b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int64_t iu = i + u * (int64_t)blockDim.x;
                    if (iu < n4) { a[u] = __ldg(h4 + iu); b[u] = __ldg(q4 + iu); }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (i + u * (int64_t)blockDim.x < n4) {
                        unsigned int k0 = mag_bits(a[u].x, b[u].x, plus), k1 = mag_bits(a[u].y, b[u].y, plus);
                        unsigned int k2 = mag_bits(a[u].z, b[u].z, plus), k3 = mag_bits(a[u].w, b[u].w, plus);
                        k0 = k0 > k1 ? k0 : k1; k2 = k2 > k3 ? k2 : k3; k0 = k0 > k2 ? k0 : k2;
                        m = k0 > m ? k0 : m;
                    }
                }
            }
        }
        for (int64_t e = v1 + threadIdx.x; e < hi; e += blockDim.x) {
            const unsigned int key = mag_bits(xh[e], xq[e], plus);
            m = key > m ? key : m;
        }
        for (int o = 16; o > 0; o >>= 1) { const unsigned int t = __shfl_xor_sync(0xffffffffu, m, o); m = t > m ? t : m; }
        if ((threadIdx.x & 31) == 0) s_m[threadIdx.x >> 5] = m;
        __syncthreads();
        if (threadIdx.x == 0) {
            for (int w = 1; w < 8; ++w) m = s_m[w] > m ? s_m[w] : m;
            if (m) atomicMax(amax_bits + (int64_t)node * seg.n_seg + s, m);
        }
        __syncthreads();
    }
}

// The step of the symmetric 8-bit quantizer for each (node, segment) message and its reciprocal:
// scale = amax/127, inv = 127/amax (1 and 1 when nothing is sent or everything is zero).
__device__ void message_scales(const unsigned int *__restrict__ amax_bits, const SegTable &seg, int nodes,
                               float *__restrict__ scale, float *__restrict__ inv) {
    for (int i = threadIdx.x; i < nodes * seg.n_seg; i += blockDim.x) {
        const float amax = seg.k[i % seg.n_seg] > 0 ? __uint_as_float(amax_bits[i]) : 0.f;
        const bool live = amax > 0.f;
        scale[i] = live ? __fdiv_rn(amax, 127.f) : 1.f;
        inv[i] = live ? __fdiv_rn(127.f, amax) : 1.f;
    }
}

__global__ void __launch_bounds__(1024)
select_and_rows_kernel(const float *__restrict__ x_half, const float *__restrict__ x_hat, int64_t d,
                       SegTable seg, SelectOut *__restrict__ out, const float *__restrict__ Wmix, int nodes,
                       int32_t *__restrict__ tab, const unsigned int *__restrict__ amax_bits,
                       float *__restrict__ msg_scale, float *__restrict__ msg_inv, BigList big,
                       const BigCtl *__restrict__ ctl, const Cand *__restrict__ cands, int64_t cand_per_node,
                       int key_cap /*keys the dynamic shared memory holds*/) {
    pdl_enter();
    if ((int)blockIdx.y == nodes) {
        if (blockIdx.x == 0) {
            build_rows(Wmix, nodes, tab);
            if (amax_bits) message_scales(amax_bits, seg, nodes, msg_scale, msg_inv);
        }
        return;
    }
    const int s = blockIdx.x, node = blockIdx.y;
    const int64_t lo = seg.off[s], hi = seg.off[s + 1], len = hi - lo, k = seg.k[s];
    SelectOut *o = out + (int64_t)node * seg.n_seg + s;
    if (k >= len) {          // keep everything
        if (threadIdx.x == 0) { o->thr = 0; o->dense = 1; o->cut = hi; }
        return;
    }
    if (k <= 0) {            // keep nothing: threshold above every finite key, no ties
        if (threadIdx.x == 0) { o->thr = 0xffffffffu; o->dense = 0; o->cut = lo; }
        return;
    }
    const float *xh = x_half + (int64_t)node * d, *xq = x_hat + (int64_t)node * d;
    if (is_big(len, k)) {
        int bi = 0;
        while (big.id[bi] != s) ++bi;            // every long segment is in the list
        // exact count of the keys at or above the sampled bucket: with at least k of them, all in the list,
        // the k largest are among the candidates; otherwise the whole-segment path below decides
        const int64_t n_cand = (int64_t)ctl[(int64_t)node * big.n + bi].cand_count;
        if (n_cand >= k && n_cand <= cand_capacity(len)) {
            extern __shared__ __align__(16) uint32_t s_sel_keys[];
            select_from_candidates(cands + (int64_t)node * cand_per_node + big.cand_base[bi], n_cand, k,
                                   ctl[(int64_t)node * big.n + bi].h1, lo, hi, o, s_sel_keys, key_cap);
            return;
        }
    }
    select_whole_segment(xh, xq, lo, hi, k, seg.plus, o);
}

// Fused public-copy update + mixing.  A block owns TE*V consecutive parameters of all nodes; a thread
// owns V consecutive ones (16-byte accesses when V = 4).  Phase 1 streams x_half and x_hat of every
// node, writes the updated public copy and parks it in shared memory; phase 2 mixes each node with
// its neighbours' copies from shared memory (x_half is read again: an L1/L2 hit).
// DS: Deep-Squeeze form (supplementary Algorithm 2): the state array is the error buffer, the message is the
// compressed x_half + state, the buffer keeps what was not sent and the mix runs over the messages themselves.
template <int V, bool Q8, bool DS>
__global__ void __launch_bounds__(256)
gossip_mix_kernel(int nodes, int64_t d, const float *__restrict__ x_half, float *__restrict__ x_hat,
                  float *__restrict__ x_out, float gamma, SegTable seg, const SelectOut *__restrict__ sel,
                  const int32_t *__restrict__ tab, const float *__restrict__ msg_scale,
                  const float *__restrict__ msg_inv) {
    pdl_enter();
    extern __shared__ __align__(16) float sm[];
    const int TE = blockDim.x;
    int32_t *s_cnt = reinterpret_cast<int32_t *>(sm);            // [nodes]
    int32_t *s_idx = s_cnt + nodes;                              // [nodes][nodes]
    float *s_val = reinterpret_cast<float *>(s_idx + nodes * nodes);
    const int tab_words = nodes + 2 * nodes * nodes;
    float *s_hat = sm + ((tab_words + 3) & ~3);                  // [nodes][TE][V], 16-byte aligned
    for (int i = threadIdx.x; i < tab_words; i += TE) s_cnt[i] = tab[i];
    __syncthreads();       // the only block-wide wait: the parked copies below are read back by the thread that wrote them
    const int64_t e0 = ((int64_t)blockIdx.x * TE + threadIdx.x) * V;
    const bool live = e0 < d;                                    // d % V == 0: a thread is all in or all out
    int s0 = 0;
    bool one_seg = true;
    if (live) {   // segment of the first parameter (segments tile [0,d))
        int a = 0, b = seg.n_seg;
        while (b - a > 1) { int m = (a + b) >> 1; if (seg.off[m] <= e0) a = m; else b = m; }
        s0 = a;
        one_seg = seg.off[s0 + 1] >= e0 + V;
    }
    constexpr int kU = V == 4 ? 8 : 4;                           // nodes per batch of independent loads (as measured)
    for (int ib = 0; ib < nodes; ib += kU) {
        float xh[kU][V], xq[kU][V];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            if (live && ib + u < nodes) {
                VecIO<V>::ld(x_half + (int64_t)(ib + u) * d + e0, xh[u]);
                VecIO<V>::ld(x_hat + (int64_t)(ib + u) * d + e0, xq[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int i = ib + u;
            if (i >= nodes) break;
            float hn[V], st_new[V];
#pragma unroll
            for (int k = 0; k < V; ++k) hn[k] = 0.f;
            if (live) {
                SelectOut so = sel[(int64_t)i * seg.n_seg + s0];
                bool changed = DS;         // the public copy changes only where an entry is sent (top-k: 1 in 100)
                float q_scale = 1.f, q_inv = 1.f;
                if (Q8) { q_scale = msg_scale[(int64_t)i * seg.n_seg + s0]; q_inv = msg_inv[(int64_t)i * seg.n_seg + s0]; }
#pragma unroll
                for (int k = 0; k < V; ++k) {
                    if (!one_seg && k > 0) {
                        int sk = s0;
                        while (seg.off[sk + 1] <= e0 + k) ++sk;
                        so = sel[(int64_t)i * seg.n_seg + sk];
                        if (Q8) { q_scale = msg_scale[(int64_t)i * seg.n_seg + sk]; q_inv = msg_inv[(int64_t)i * seg.n_seg + sk]; }
                    }
                    const float delta = DS ? __fadd_rn(xh[u][k], xq[u][k]) : __fsub_rn(xh[u][k], xq[u][k]);
                    const uint32_t key = __float_as_uint(delta) & 0x7fffffffu;
                    const bool keep = so.dense || key > so.thr || (key == so.thr && e0 + k < so.cut);
                    changed |= keep;
                    float msg = delta;
                    if (Q8) {      // the message is the 8-bit code times the step; the state absorbs exactly that
                        const float code = fminf(fmaxf(rintf(__fmul_rn(delta, q_inv)), -127.f), 127.f);
                        msg = __fmul_rn(code, q_scale);
                    }
                    if (DS) {      // park the message, keep the remainder in the error buffer
                        hn[k] = keep ? msg : 0.f;
                        st_new[k] = __fsub_rn(delta, hn[k]);
                    } else {       // public copy + message; that sum is also what the neighbours mix
                        hn[k] = keep ? __fadd_rn(xq[u][k], msg) : xq[u][k];
                        st_new[k] = hn[k];
                    }
                }
                if (changed) VecIO<V>::st(x_hat + (int64_t)i * d + e0, st_new);      // unchanged values are not rewritten
            }
            VecIO<V>::st(s_hat + ((size_t)i * TE + threadIdx.x) * V, hn);
        }
    }
    if (!live) return;
    for (int ib = 0; ib < nodes; ib += kU) {
        float xh[kU][V];
#pragma unroll
        for (int u = 0; u < kU; ++u)
            if (ib + u < nodes) VecIO<V>::ld(x_half + (int64_t)(ib + u) * d + e0, xh[u]);
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int i = ib + u;
            if (i >= nodes) break;
            float hi_[V], acc[V], o[V];
            VecIO<V>::ld(s_hat + ((size_t)i * TE + threadIdx.x) * V, hi_);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] = 0.f;
            const int c = s_cnt[i];
            for (int m = 0; m < c; ++m) {                        // neighbours in ascending j
                const int j = s_idx[i * nodes + m];
                const float w = s_val[i * nodes + m];
                float hj[V];
                VecIO<V>::ld(s_hat + ((size_t)j * TE + threadIdx.x) * V, hj);
#pragma unroll
                for (int k = 0; k < V; ++k)
                    acc[k] = DS ? __fadd_rn(acc[k], __fmul_rn(w, hj[k]))                         // sum_j W_ij c_j
                                : __fadd_rn(acc[k], __fmul_rn(w, __fsub_rn(hj[k], hi_[k])));      // sum_j W_ij (xhat_j - xhat_i)
            }
            if (DS) {
#pragma unroll
                for (int k = 0; k < V; ++k) acc[k] = __fsub_rn(acc[k], hi_[k]);                   // - I_ij c_j
            }
#pragma unroll
            for (int k = 0; k < V; ++k) o[k] = __fadd_rn(xh[u][k], __fmul_rn(gamma, acc[k]));
            VecIO<V>::st(x_out + (int64_t)i * d + e0, o);
        }
    }
}

// Push-sum bias weights and de-biased model (supplementary Algorithms 4 and 5: second half of the gossip
// update, then the de-biasing step).  Grid (chunks, nodes); every CTA recomputes its node's new bias
// weight (one row of W times u: at most 64 multiply-adds, j ascending, by one thread) and then streams
// z = x / u_new over its chunk (4 B read + 4 B write per parameter).
template <int V>
__global__ void __launch_bounds__(256)
pushsum_debias_kernel(int nodes, int64_t d, const float *__restrict__ x, const float *__restrict__ u,
                      const float *__restrict__ Wmix, float eta, float *__restrict__ u_new, float *__restrict__ z) {
    pdl_enter();
    const int node = blockIdx.y;
    __shared__ float s_u;
    if (threadIdx.x == 0) {
        float acc = 0.f;
        for (int j = 0; j < nodes; ++j) acc = __fadd_rn(acc, __fmul_rn(Wmix[node * nodes + j], u[j]));
        acc = __fsub_rn(acc, u[node]);
        const float un = __fadd_rn(u[node], __fmul_rn(eta, acc));
        s_u = un;
        if (blockIdx.x == 0) u_new[node] = un;
    }
    __syncthreads();
    const float un = s_u;
    const float *xr = x + (int64_t)node * d;
    float *zr = z + (int64_t)node * d;
    constexpr int kU = 4;                                        // independent loads per thread
    const int64_t per_block = (int64_t)blockDim.x * V * kU;
    const int64_t b0 = (int64_t)blockIdx.x * per_block;
    float v[kU][V];
#pragma unroll
    for (int q = 0; q < kU; ++q) {
        const int64_t e = b0 + ((int64_t)q * blockDim.x + threadIdx.x) * V;
        if (e < d) VecIO<V>::ld(xr + e, v[q]);
    }
#pragma unroll
    for (int q = 0; q < kU; ++q) {
        const int64_t e = b0 + ((int64_t)q * blockDim.x + threadIdx.x) * V;
        if (e < d) {
#pragma unroll
            for (int k = 0; k < V; ++k) v[q][k] = __fdiv_rn(v[q][k], un);
            VecIO<V>::st(zr + e, v[q]);
        }
    }
}


// SGD half-step fused into the uncompressed gossip step (Algorithm 1 "update the model" followed by Algorithm 3
// with every entry kept): x_half = x - lr*g is computed where the mix needs it, so the parameters and gradients
// are read once and the separate update pass (12 B per parameter) disappears.  Same operation order as
// lpdt_sgd_update followed by lpdt_gossip_mix with dense segments: x_hat <- x_hat + (x_half - x_hat), then the mix
// over the updated copies.  Every CTA builds the compact rows of W itself (nodes^2 values).
template <int V>
__global__ void __launch_bounds__(256)
sgd_dense_mix_kernel(int nodes, int64_t d, const float *__restrict__ x, const float *__restrict__ g, float lr,
                     float *x_half, float *__restrict__ x_hat, float *__restrict__ x_out,
                     const float *__restrict__ Wmix, float gamma) {
    pdl_enter();
    extern __shared__ __align__(16) float sm[];
    const int TE = blockDim.x;
    int32_t *s_cnt = reinterpret_cast<int32_t *>(sm);            // [nodes]
    int32_t *s_idx = s_cnt + nodes;                              // [nodes][nodes]
    float *s_val = reinterpret_cast<float *>(s_idx + nodes * nodes);
    const int tab_words = nodes + 2 * nodes * nodes;
    float *s_hat = sm + ((tab_words + 3) & ~3);                  // [nodes][TE][V]
    for (int i = threadIdx.x; i < nodes; i += TE) {
        int c = 0;
        for (int j = 0; j < nodes; ++j) {
            const float w = Wmix[i * nodes + j];
            if (w != 0.f) { s_idx[i * nodes + c] = j; s_val[i * nodes + c] = w; ++c; }
        }
        s_cnt[i] = c;
    }
    __syncthreads();
    const int64_t e0 = ((int64_t)blockIdx.x * TE + threadIdx.x) * V;
    if (e0 >= d) return;                                         // d % V == 0: a thread is all in or all out
    constexpr int kU = 4;
    for (int ib = 0; ib < nodes; ib += kU) {
        float xv[kU][V], gv[kU][V], xq[kU][V];
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            if (ib + u < nodes) {
                VecIO<V>::ld(x + (int64_t)(ib + u) * d + e0, xv[u]);
                VecIO<V>::ld(g + (int64_t)(ib + u) * d + e0, gv[u]);
                VecIO<V>::ld(x_hat + (int64_t)(ib + u) * d + e0, xq[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int i = ib + u;
            if (i >= nodes) break;
            float xh[V], hn[V];
#pragma unroll
            for (int k = 0; k < V; ++k) {
                xh[k] = __fsub_rn(xv[u][k], __fmul_rn(lr, gv[u][k]));
                hn[k] = __fadd_rn(xq[u][k], __fsub_rn(xh[k], xq[u][k]));
            }
            VecIO<V>::st(x_half + (int64_t)i * d + e0, xh);
            VecIO<V>::st(x_hat + (int64_t)i * d + e0, hn);
            VecIO<V>::st(s_hat + ((size_t)i * TE + threadIdx.x) * V, hn);
        }
    }
    for (int ib = 0; ib < nodes; ib += kU) {
        float xh[kU][V];
#pragma unroll
        for (int u = 0; u < kU; ++u)           // written above by this thread (plain pointer: no read-only path)
            if (ib + u < nodes) VecIO<V>::ld(x_half + (int64_t)(ib + u) * d + e0, xh[u]);
#pragma unroll
        for (int u = 0; u < kU; ++u) {
            const int i = ib + u;
            if (i >= nodes) break;
            float hi_[V], acc[V], o[V];
            VecIO<V>::ld(s_hat + ((size_t)i * TE + threadIdx.x) * V, hi_);
#pragma unroll
            for (int k = 0; k < V; ++k) acc[k] = 0.f;
            const int c = s_cnt[i];
            for (int m = 0; m < c; ++m) {                        // neighbours in ascending j
                const int j = s_idx[i * nodes + m];
                const float w = s_val[i * nodes + m];
                float hj[V];
                VecIO<V>::ld(s_hat + ((size_t)j * TE + threadIdx.x) * V, hj);
#pragma unroll
                for (int k = 0; k < V; ++k) acc[k] = __fadd_rn(acc[k], __fmul_rn(w, __fsub_rn(hj[k], hi_[k])));
            }
#pragma unroll
            for (int k = 0; k < V; ++k) o[k] = __fadd_rn(xh[u][k], __fmul_rn(gamma, acc[k]));
            VecIO<V>::st(x_out + (int64_t)i * d + e0, o);
        }
    }
}

}  // namespace lpdt

using namespace lpdt;

static size_t select_bytes(int32_t nodes, int32_t n_segments) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)(n_segments > 0 ? n_segments : 1) * sizeof(SelectOut), 256);
}
static size_t rows_bytes(int32_t nodes) {
    const size_t nn = (size_t)(nodes > 0 ? nodes : 1);
    return align_up((nn + 2 * nn * nn) * sizeof(int32_t), 256);
}
// the most long segments any segmentation of d parameters into n_segments can have
static int64_t max_big(int64_t d, int32_t n_segments) {
    int64_t m = d / kBigMin;
    return m < n_segments ? m : n_segments;
}
// candidate entries per node that any segmentation can need: sum over long segments of cand_capacity(len)
static int64_t max_cands(int64_t d, int32_t n_segments) { return d / 8 + 4096 * max_big(d, n_segments); }
static size_t big_ctl_bytes(int32_t nodes, int64_t d, int32_t n_segments) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)max_big(d, n_segments) * (sizeof(BigCtl) + sizeof(BigState)), 256);
}
static size_t cand_bytes(int32_t nodes, int64_t d, int32_t n_segments) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)max_cands(d, n_segments) * sizeof(Cand), 256);
}
// range words and reciprocal steps of the 8-bit messages, one per (node, segment) each (last in the workspace)
static size_t q8_bytes(int32_t nodes, int32_t n_segments) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)(n_segments > 0 ? n_segments : 1) * sizeof(float), 256);
}

extern "C" size_t lpdt_gossip_mix_workspace_size(int32_t nodes, int64_t d, int32_t n_segments) {
    if (d < 0) d = 0;
    if (n_segments < 1) n_segments = 1;
    return select_bytes(nodes, n_segments) + rows_bytes(nodes) + big_ctl_bytes(nodes, d, n_segments) +
           cand_bytes(nodes, d, n_segments) + 2 * q8_bytes(nodes, n_segments);
}

static lpdt_status gossip_impl(int32_t nodes, int64_t d, const float *x_half, float *x_hat,
                               float *x_out, const float *Wmix, float gamma, int32_t n_segments,
                               const int64_t *seg_offsets, const int64_t *seg_k, float *msg_scale, bool q8, bool ds,
                               void *ws, size_t ws_bytes, int32_t *dev_status, void *stream) {
    (void)dev_status;
    LPDT_CHECK_ARG(nodes >= 0 && d >= 0 && n_segments >= 1);
    if (nodes == 0 || d == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x_half && x_hat && x_out && Wmix && seg_offsets && seg_k && (!q8 || msg_scale));
    LPDT_CHECK_ARG(x_hat != x_half && x_hat != x_out);
    if (nodes > kMaxNodes || n_segments > kMaxSeg) return LPDT_ERR_UNSUPPORTED;
    LPDT_CHECK_ARG(seg_offsets[0] == 0 && seg_offsets[n_segments] == d);
    SegTable seg;
    seg.n_seg = n_segments;
    seg.plus = ds ? 1 : 0;
    for (int s = 0; s < n_segments; ++s) {
        LPDT_CHECK_ARG(seg_offsets[s + 1] > seg_offsets[s] && seg_k[s] >= 0);
        seg.off[s] = seg_offsets[s];
        seg.k[s] = seg_k[s];
    }
    seg.off[n_segments] = d;
    if (!ws || ws_bytes < lpdt_gossip_mix_workspace_size(nodes, d, n_segments) || !aligned(ws, 8))
        return LPDT_ERR_WORKSPACE;
    cudaStream_t st = as_stream(stream);
    SelectOut *sel = (SelectOut *)ws;
    int32_t *tab = (int32_t *)((char *)ws + select_bytes(nodes, n_segments));
    BigList big;
    big.n = 0; big.chunk_base[0] = 0; big.cand_base[0] = 0;
    int64_t most_chunks = 0, longest = 0;
    for (int s = 0; s < n_segments; ++s) {
        const int64_t len = seg.off[s + 1] - seg.off[s];
        if (!is_big(len, seg.k[s])) continue;
        if (len > 0xFFFFFFFFll) return LPDT_ERR_UNSUPPORTED;      // candidate positions are 32-bit
        const int64_t nc = ceil_div(len, (int64_t)kChunk);
        big.id[big.n] = s;
        big.chunk_base[big.n + 1] = big.chunk_base[big.n] + (int32_t)nc;
        big.cand_base[big.n + 1] = big.cand_base[big.n] + cand_capacity(len);
        if (nc > most_chunks) most_chunks = nc;
        if (len > longest) longest = len;
        ++big.n;
    }
    char *big_region = (char *)tab + rows_bytes(nodes);
    BigCtl *ctl = (BigCtl *)big_region;
    BigState *state = (BigState *)(ctl + (size_t)nodes * big.n);
    Cand *cands = (Cand *)(big_region + big_ctl_bytes(nodes, d, n_segments));
    const int64_t cand_per_node = big.cand_base[big.n];
    // 8-bit messages: ranges of the differences (the kept entries are the largest of their segment).  The collect
    // pass of a long compressed segment sees every difference anyway and records the range itself; the separate
    // range pass runs only when some segment does not go through it.
    unsigned int *amax_bits = nullptr;
    float *msg_inv = nullptr;
    if (q8) {
        amax_bits = (unsigned int *)((char *)ws + lpdt_gossip_mix_workspace_size(nodes, d, n_segments) - 2 * q8_bytes(nodes, n_segments));
        msg_inv = (float *)((char *)amax_bits + q8_bytes(nodes, n_segments));
        if (nodes > 65535) return LPDT_ERR_UNSUPPORTED;
        LPDT_CUDA(cudaMemsetAsync(amax_bits, 0, (size_t)nodes * n_segments * sizeof(unsigned int), st));
    }
    if (big.n > 0) {
        if (most_chunks > 0x7fffffff || nodes > 65535) return LPDT_ERR_UNSUPPORTED;
        LPDT_CUDA(cudaMemsetAsync(ctl, 0, (size_t)nodes * big.n * sizeof(BigCtl), st));
        // elements per CTA of the collect pass: every CTA clears and flushes a 4096-bin histogram, so chunks are as
        // long as still leaves several CTAs per SM (16 K ... 64 K elements)
        int chunk = kChunk;
        while (chunk < 65536 && ceil_div(longest, (int64_t)chunk * 2) * big.n * nodes >= 4 * (int64_t)kNumSMs) chunk *= 2;
        const dim3 g((unsigned)ceil_div(longest, (int64_t)chunk), big.n, nodes);
        const int64_t sample_ctas = ceil_div(longest, kSampleChunk);
        if (sample_ctas > 65535) return LPDT_ERR_UNSUPPORTED;
        launch_k(big_sample_kernel, dim3((unsigned)sample_ctas, big.n, nodes), 256, 0, st, x_half, x_hat, d, seg, big, ctl, state);
        LPDT_LAUNCH_CHECK();
        launch_k(big_collect_kernel, g, 256, 0, st, x_half, x_hat, d, seg, big, ctl, state, cands, cand_per_node, amax_bits, chunk);
        LPDT_LAUNCH_CHECK();
    }
    if (q8 && big.n < n_segments) {
        launch_k(delta_amax_kernel, dim3((unsigned)ceil_div(d, (int64_t)kChunk), nodes), 256, 0, st, x_half, x_hat, d, seg, amax_bits);
        LPDT_LAUNCH_CHECK();
    }
    // Shared-memory buffer for the keys of the threshold's bucket of a long segment (1/16 of an octave of
    // magnitudes: well under 1/64 of the segment unless the magnitudes are nearly constant; when they do not
    // fit, the selection reads the candidate list again for every radix pass instead).
    int key_cap = 0;
    if (big.n > 0) {
        int64_t want = longest / 64;
        key_cap = (int)(want < 1024 ? 1024 : want > 40960 ? 40960 : want);
        static PerDeviceOnce attr;
        int dev;
        if (attr.pending(&dev)) {
            LPDT_CUDA(cudaFuncSetAttribute(select_and_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 40960 * 4));
            attr.mark(dev);
        }
    }
    launch_k(select_and_rows_kernel, dim3(n_segments, nodes + 1), 1024, (size_t)key_cap * sizeof(uint32_t), st, x_half, x_hat, d,
             seg, sel, Wmix, nodes, tab, amax_bits, msg_scale, msg_inv, big, ctl, cands, cand_per_node, key_cap);
    LPDT_LAUNCH_CHECK();
    // parameters per thread: 16-byte accesses need every node's row on a 16-byte boundary (d a multiple of 4);
    // the networks' parameter counts are even but not multiples of 4, which still allows 8-byte accesses
    const bool v4 = d % 4 == 0 && aligned(x_half, 16) && aligned(x_hat, 16) && aligned(x_out, 16);
    const bool v2 = !v4 && d % 2 == 0 && aligned(x_half, 8) && aligned(x_hat, 8) && aligned(x_out, 8);
    const int V = v4 ? 4 : v2 ? 2 : 1;
    const int vi = v4 ? 2 : v2 ? 1 : 0;
    // threads per block: as many as keep the parked public copies within 64 KB of shared memory
    int TE = (int)((64 * 1024) / ((size_t)nodes * V * sizeof(float))) / 32 * 32;
    if (TE > 128) TE = 128;
    if (TE < 32) TE = 32;
    const size_t tab_words = ((size_t)nodes + 2 * (size_t)nodes * nodes + 3) & ~(size_t)3;
    const size_t smem = tab_words * sizeof(int32_t) + (size_t)nodes * TE * V * sizeof(float);
    using MixFn = void (*)(int, int64_t, const float *, float *, float *, float, SegTable, const SelectOut *,
                           const int32_t *, const float *, const float *);
    static const MixFn fns[12] = {
        gossip_mix_kernel<1, false, false>, gossip_mix_kernel<2, false, false>, gossip_mix_kernel<4, false, false>,
        gossip_mix_kernel<1, true, false>,  gossip_mix_kernel<2, true, false>,  gossip_mix_kernel<4, true, false>,
        gossip_mix_kernel<1, false, true>,  gossip_mix_kernel<2, false, true>,  gossip_mix_kernel<4, false, true>,
        gossip_mix_kernel<1, true, true>,   gossip_mix_kernel<2, true, true>,   gossip_mix_kernel<4, true, true>};
    static PerDeviceOnce attr_set;
    int dev;
    if (attr_set.pending(&dev)) {
        for (int i = 0; i < 12; ++i)
            LPDT_CUDA(cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024));
        attr_set.mark(dev);
    }
    const unsigned blocks = (unsigned)ceil_div(d, (int64_t)TE * V);
    launch_k(fns[(ds ? 6 : 0) + (q8 ? 3 : 0) + vi], blocks, TE, smem, st, nodes, d, x_half, x_hat, x_out, gamma, seg, sel, tab,
                                                                            q8 ? msg_scale : nullptr, msg_inv);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_gossip_mix(int32_t nodes, int64_t d, const float *x_half, float *x_hat,
                                       float *x_out, const float *Wmix, float gamma, int32_t n_segments,
                                       const int64_t *seg_offsets, const int64_t *seg_k, void *ws,
                                       size_t ws_bytes, int32_t *dev_status, void *stream) {
    return gossip_impl(nodes, d, x_half, x_hat, x_out, Wmix, gamma, n_segments, seg_offsets, seg_k, nullptr, false, false,
                       ws, ws_bytes, dev_status, stream);
}

extern "C" lpdt_status lpdt_gossip_mix_q8(int32_t nodes, int64_t d, const float *x_half, float *x_hat,
                                          float *x_out, const float *Wmix, float gamma, int32_t n_segments,
                                          const int64_t *seg_offsets, const int64_t *seg_k, float *msg_scale,
                                          void *ws, size_t ws_bytes, int32_t *dev_status, void *stream) {
    return gossip_impl(nodes, d, x_half, x_hat, x_out, Wmix, gamma, n_segments, seg_offsets, seg_k, msg_scale, true, false,
                       ws, ws_bytes, dev_status, stream);
}

extern "C" lpdt_status lpdt_deepsqueeze_mix(int32_t nodes, int64_t d, const float *x_half, float *delta,
                                            float *x_out, const float *Wmix, float eta, int32_t n_segments,
                                            const int64_t *seg_offsets, const int64_t *seg_k, int32_t message_bits,
                                            float *msg_scale, void *ws, size_t ws_bytes, int32_t *dev_status,
                                            void *stream) {
    LPDT_CHECK_ARG(message_bits == 32 || message_bits == 8);
    return gossip_impl(nodes, d, x_half, delta, x_out, Wmix, eta, n_segments, seg_offsets, seg_k, msg_scale,
                       message_bits == 8, true, ws, ws_bytes, dev_status, stream);
}

extern "C" lpdt_status lpdt_pushsum_debias(int32_t nodes, int64_t d, const float *x, const float *u, const float *Wmix,
                                           float eta, float *u_new, float *z, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && d >= 0);
    if (nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(u && Wmix && u_new && u_new != u && (d == 0 || (x && z)));
    if (nodes > kMaxNodes) return LPDT_ERR_UNSUPPORTED;
    cudaStream_t st = as_stream(stream);
    const bool v4 = d % 4 == 0 && aligned(x, 16) && aligned(z, 16);
    const int64_t per_block = 256 * 4 * (v4 ? 4 : 1);
    int64_t chunks = ceil_div(d, per_block);
    if (chunks < 1) chunks = 1;                                  // d = 0: the bias weights alone
    if (chunks > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    const dim3 g((unsigned)chunks, nodes);
    if (v4) launch_k(pushsum_debias_kernel<4>, g, 256, 0, st, nodes, d, x, u, Wmix, eta, u_new, z);
    else launch_k(pushsum_debias_kernel<1>, g, 256, 0, st, nodes, d, x, u, Wmix, eta, u_new, z);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_sgd_gossip_mix(int32_t nodes, int64_t d, const float *x, const float *g, float lr,
                                           float *x_half, float *x_hat, float *x_out, const float *Wmix, float gamma,
                                           void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && d >= 0);
    if (nodes == 0 || d == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && g && x_half && x_hat && x_out && Wmix);
    LPDT_CHECK_ARG(x_half != x && x_half != g && x_hat != x_half && x_out != x_half && x_out != x_hat && x_out != x &&
                   x_out != g && x_hat != x && x_hat != g);
    if (nodes > kMaxNodes) return LPDT_ERR_UNSUPPORTED;
    const float *in[2] = {x, g};
    float *io[3] = {x_half, x_hat, x_out};
    bool a16 = d % 4 == 0, a8 = d % 2 == 0;
    for (int i = 0; i < 2; ++i) { a16 = a16 && aligned(in[i], 16); a8 = a8 && aligned(in[i], 8); }
    for (int i = 0; i < 3; ++i) { a16 = a16 && aligned(io[i], 16); a8 = a8 && aligned(io[i], 8); }
    const int V = a16 ? 4 : a8 ? 2 : 1;
    int TE = (int)((64 * 1024) / ((size_t)nodes * V * sizeof(float))) / 32 * 32;
    if (TE > 128) TE = 128;
    if (TE < 32) TE = 32;
    const size_t tab_words = ((size_t)nodes + 2 * (size_t)nodes * nodes + 3) & ~(size_t)3;
    const size_t smem = tab_words * sizeof(int32_t) + (size_t)nodes * TE * V * sizeof(float);
    using Fn = void (*)(int, int64_t, const float *, const float *, float, float *, float *, float *, const float *, float);
    static const Fn fns[3] = {sgd_dense_mix_kernel<1>, sgd_dense_mix_kernel<2>, sgd_dense_mix_kernel<4>};
    static PerDeviceOnce attr_set;
    int dev;
    if (attr_set.pending(&dev)) {
        for (int i = 0; i < 3; ++i)
            LPDT_CUDA(cudaFuncSetAttribute(fns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, 128 * 1024));
        attr_set.mark(dev);
    }
    const int64_t blocks = ceil_div(d, (int64_t)TE * V);
    if (blocks > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    launch_k(fns[V == 4 ? 2 : V == 2 ? 1 : 0], (unsigned)blocks, TE, smem, as_stream(stream), nodes, d, x, g, lr, x_half,
             x_hat, x_out, Wmix, gamma);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
