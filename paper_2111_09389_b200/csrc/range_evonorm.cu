// Range-EvoNorm (Eq. "ren") forward and backward.
//
// One CTA per (node, sample); the forward kernel can split a sample over a cluster
// of up to 8 CTAs.  Every thread owns a fixed vector-column of V channels and walks
// the pixels, so global accesses are fully coalesced 16-byte loads and the thread's
// channel parameters and group live in registers.
// Forward: pass 1 finds the per-group extrema; a warp-shuffle reduction with a
// (value, lowest index) comparator merges the threads of a group, the CTAs of a
// cluster exchange their group extrema through distributed shared memory; pass 2
// re-reads the sample and writes the output.  The second read is an L2 hit as long
// as the samples in flight fit the L2: with large samples the cluster split keeps
// that footprint small (fewer samples in flight, each finished sooner).  Backward is a single pass: the local term of dx is written while the
// group sum S and the per-channel gradient sums accumulate, and S is applied
// afterwards at the two extremum positions of each group.  Both kernels are
// HBM-bound: forward moves 4 B in + 4 B out per element, backward 8 B in + 4 B out.
#include <math.h>
#include <stdlib.h>
#include <map>
#include <mutex>
#include <tuple>
#include <cooperative_groups.h>
#include "common.cuh"

namespace lpdt {

struct Ext { float v; int idx; };

__device__ __forceinline__ Ext ext_max(Ext a, Ext b) {
    return (b.v > a.v || (b.v == a.v && b.idx < a.idx)) ? b : a;
}
__device__ __forceinline__ Ext ext_min(Ext a, Ext b) {
    return (b.v < a.v || (b.v == a.v && b.idx < a.idx)) ? b : a;
}
__device__ __forceinline__ Ext shfl_ext(Ext e, int o) {
    Ext r; r.v = __shfl_xor_sync(0xffffffffu, e.v, o); r.idx = __shfl_xor_sync(0xffffffffu, e.idx, o);
    return r;
}

template <int V> struct VecLoad;
template <> struct VecLoad<4> {
    static __device__ __forceinline__ void ld(const float *p, float (&o)[4]) {
        float4 t = *reinterpret_cast<const float4 *>(p); o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
    }
    static __device__ __forceinline__ void st(float *p, const float (&o)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(o[0], o[1], o[2], o[3]);
    }
};
template <> struct VecLoad<1> {
    static __device__ __forceinline__ void ld(const float *p, float (&o)[1]) { o[0] = *p; }
    static __device__ __forceinline__ void st(float *p, const float (&o)[1]) { *p = o[0]; }
};

// hard sigmoid and the normalised product, each operation rounded on its own
// (u + 3)/6 correctly rounded without the division unit: q = a*y with y = RN(1/6), the
// exact residual r = a - 6q by FMA, and one correction step q + r*y (Markstein's
// division by a constant); identical to the IEEE quotient for every finite a here.
__device__ __forceinline__ float hsig(float u) {
    const float a = __fadd_rn(u, 3.f);
    const float y = 0x1.555556p-3f;
    const float q = __fmul_rn(a, y);
    const float r = __fmaf_rn(-6.f, q, a);
    float h = __fmaf_rn(r, y, q);
    return fminf(fmaxf(h, 0.f), 1.f);
}

// Reduce per-thread extrema to per-group extrema.  s_mn/s_mx hold one entry per
// thread; members of group g are the threads whose column lies in the group.
template <int V>
__device__ void reduce_groups(Ext mn, Ext mx, Ext *s_mn, Ext *s_mx, Ext *g_mn, Ext *g_mx,
                              int CV, int cpg, int groups) {
    const int T = blockDim.x, t = threadIdx.x;
    s_mn[t] = mn; s_mx[t] = mx;
    __syncthreads();
    const int lane = t & 31, warp = t >> 5, nw = T >> 5;
    const int cols = cpg / V, rows = T / CV, members = cols * rows;
    for (int g = warp; g < groups; g += nw) {
        Ext a; a.v = INFINITY; a.idx = 0x7fffffff;
        Ext b; b.v = -INFINITY; b.idx = 0x7fffffff;
        for (int m = lane; m < members; m += 32) {
            int th = (m / cols) * CV + g * cols + (m % cols);
            a = ext_min(a, s_mn[th]); b = ext_max(b, s_mx[th]);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) { a = ext_min(a, shfl_ext(a, o)); b = ext_max(b, shfl_ext(b, o)); }
        if (lane == 0) { g_mn[g] = a; g_mx[g] = b; }
    }
    __syncthreads();
}

template <int V, bool RES>
__global__ void __launch_bounds__(512, 2)
ren_fwd_kernel(int HW, int C, int groups, float eps, float Cst,
               const float *__restrict__ x, const float *__restrict__ v,
               const float *__restrict__ gamma, const float *__restrict__ beta, int64_t pstride,
               int B, float *__restrict__ y, float *__restrict__ gmin, float *__restrict__ gmax,
               int32_t *__restrict__ argmin, int32_t *__restrict__ argmax, float *__restrict__ amax_out,
               const float *__restrict__ res, int R /*CTAs per sample (cluster size)*/, int ppc /*pixels per CTA*/) {
    namespace cg = cooperative_groups;
    pdl_enter();
    extern __shared__ unsigned char smem_raw[];
    const int T = blockDim.x, t = threadIdx.x;
    Ext *s_mn = reinterpret_cast<Ext *>(smem_raw);
    Ext *s_mx = s_mn + T;
    Ext *g_mn = s_mx + T;                 // the sample's group extrema
    Ext *g_mx = g_mn + groups;
    Ext *part_mn = g_mx + groups;         // this CTA's group extrema, read by the whole cluster (R > 1)
    Ext *part_mx = part_mn + groups;
    const int CV = C / V, cpg = C / groups;
    const int col = t % CV, row0 = t / CV, rstep = T / CV;
    const int c0 = col * V, grp = c0 / cpg;
    const int rank = (int)(blockIdx.x % R);
    const int64_t sample = blockIdx.x / R;     // node*B + b
    const int p_lo = rank * ppc;
    const int p_end = (p_lo + ppc < HW) ? p_lo + ppc : HW;     // this CTA's pixels: [p_lo, p_end)
    const int node = (int)(sample / B);
    const float *xs = x + sample * (int64_t)HW * C;
    float *ys = y + sample * (int64_t)HW * C;

    Ext mn, mx; mn.v = INFINITY; mn.idx = 0x7fffffff; mx.v = -INFINITY; mx.idx = 0x7fffffff;
    // kU independent 16-byte loads per thread are issued before any of them is used: the kernel
    // is bound by the bytes in flight, not by arithmetic
    constexpr int kU = 8;
    int p = p_lo + row0;
    for (; p + (kU - 1) * rstep < p_end; p += kU * rstep) {
        float xv[kU][V];
#pragma unroll
        for (int j = 0; j < kU; ++j) VecLoad<V>::ld(xs + (int64_t)(p + j * rstep) * C + c0, xv[j]);
#pragma unroll
        for (int j = 0; j < kU; ++j) {
#pragma unroll
            for (int k = 0; k < V; ++k) {
                int idx = (p + j * rstep) * C + c0 + k;
                if (xv[j][k] > mx.v) { mx.v = xv[j][k]; mx.idx = idx; }
                if (xv[j][k] < mn.v) { mn.v = xv[j][k]; mn.idx = idx; }
            }
        }
    }
    for (; p < p_end; p += rstep) {
        float xv[V];
        VecLoad<V>::ld(xs + (int64_t)p * C + c0, xv);
#pragma unroll
        for (int k = 0; k < V; ++k) {
            int idx = p * C + c0 + k;
            if (xv[k] > mx.v) { mx.v = xv[k]; mx.idx = idx; }
            if (xv[k] < mn.v) { mn.v = xv[k]; mn.idx = idx; }
        }
    }
    if (R == 1) {
        reduce_groups<V>(mn, mx, s_mn, s_mx, g_mn, g_mx, CV, cpg, groups);
    } else {
        reduce_groups<V>(mn, mx, s_mn, s_mx, part_mn, part_mx, CV, cpg, groups);
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();                        // every CTA's part_* is complete and visible
        if (t < groups) {
            Ext a = part_mn[t], b = part_mx[t];
            for (int r = 1; r < R; ++r) {      // equal values: the lowest index wins, in any order
                const int other = (rank + r) % R;
                a = ext_min(a, *cluster.map_shared_rank(part_mn + t, other));
                b = ext_max(b, *cluster.map_shared_rank(part_mx + t, other));
            }
            g_mn[t] = a; g_mx[t] = b;
        }
        __syncthreads();
        cluster.barrier_arrive();              // done reading the others' shared memory; waited for before exit
    }
    if (t < groups && rank == 0) {
        int64_t sg = sample * groups + t;
        gmin[sg] = g_mn[t].v; gmax[sg] = g_mx[t].v; argmin[sg] = g_mn[t].idx; argmax[sg] = g_mx[t].idx;
    }
    const float rng = __fsub_rn(g_mx[grp].v, g_mn[grp].v);
    const float D = __fadd_rn(__fmul_rn(Cst, rng), eps);
    const float invD = __fdiv_rn(1.f, D);
    float vc[V], gc[V], bc[V];
    float ymax = 0.f;
#pragma unroll
    for (int k = 0; k < V; ++k) {
        vc[k] = v[(int64_t)node * pstride + c0 + k];
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
        bc[k] = beta[(int64_t)node * pstride + c0 + k];
    }
    const float *rs = RES ? res + sample * (int64_t)HW * C : nullptr;
    auto emit = [&](int pp, const float (&xv)[V], const float (&rv)[V]) {
        float yv[V];
#pragma unroll
        for (int k = 0; k < V; ++k) {
            float u = __fmul_rn(vc[k], xv[k]);
            float m = __fmul_rn(xv[k], hsig(u));
            yv[k] = __fadd_rn(__fmul_rn(__fmul_rn(gc[k], m), invD), bc[k]);
            if (RES) yv[k] = __fadd_rn(yv[k], rv[k]);           // fused identity shortcut: y = REN(x) + res
            ymax = fmaxf(ymax, fabsf(yv[k]));
        }
        VecLoad<V>::st(ys + (int64_t)pp * C + c0, yv);
    };
    constexpr int kU2 = RES ? 2 : 4;
    p = p_lo + row0;
    for (; p + (kU2 - 1) * rstep < p_end; p += kU2 * rstep) {
        float xv[kU2][V], rv[kU2][V];
#pragma unroll
        for (int j = 0; j < kU2; ++j) {
            VecLoad<V>::ld(xs + (int64_t)(p + j * rstep) * C + c0, xv[j]);
            if (RES) VecLoad<V>::ld(rs + (int64_t)(p + j * rstep) * C + c0, rv[j]);
        }
#pragma unroll
        for (int j = 0; j < kU2; ++j) emit(p + j * rstep, xv[j], rv[j]);
    }
    for (; p < p_end; p += rstep) {
        float xv[V], rv[V];
        VecLoad<V>::ld(xs + (int64_t)p * C + c0, xv);
        if (RES) VecLoad<V>::ld(rs + (int64_t)p * C + c0, rv);
        emit(p, xv, rv);
    }
    if (amax_out) block_amax_to(ymax, amax_out + node);
    if (R > 1) cg::this_cluster().barrier_wait();      // nobody still reads this CTA's shared memory
}

// Asynchronous 16-byte copy global -> shared (bypasses registers) and its group bookkeeping.
__device__ __forceinline__ void cp_async16(void *smem_dst, const void *gsrc) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// Symmetric 8-bit code of x for a tensor whose max|x| gave inv = 127 / max|x| (round to nearest even, clamped):
// the arithmetic of the library's quantizer, so that a producer writing codes itself gives the same codes.
__device__ __forceinline__ int ren_q_sym_rne(float x, float inv) {
    float r = rintf(__fmul_rn(x, inv));
    r = fminf(fmaxf(r, -127.f), 127.f);
    return (int)r;
}

// ---- Kernels that write 8-bit codes themselves (requantize inside the producer) ------------------------
// The node-wide range must be known before the first code is written, so the CTAs of a node meet once:
// one CTA per sample keeps its fp32 result in shared memory, adds its max|.| to the node's word and
// arrives at the node's counter; when all B samples of the node have arrived every CTA reads the node's
// maximum and rounds what it holds.  Samples are handed out by a ticket counter in the order in which CTAs
// start, so whenever a CTA waits for its node, every sample of every earlier node and every lower sample of
// its own node is held by a CTA that has started; the missing samples are the next tickets and go to the
// next CTAs that start.  At most B - 1 CTAs can wait for an incomplete node, so with room for at least
// 2 B resident CTAs (checked by the host) some CTA always makes progress.  The wait is bounded all the
// same: after kNodeWaitLimitNs it records LPDT_ERR_TIMEOUT and the CTA returns without writing codes.
//
// Control block (int32 words, zero before the first launch; the kernels leave it zero again):
//   [0, nodes) arrivals   [nodes, 2 nodes) departures   [2 nodes, 3 nodes) bits of max|.|
//   [3 nodes] ticket      [3 nodes + 1] CTAs finished
constexpr unsigned long long kNodeWaitLimitNs = 2000000000ull;

__device__ __forceinline__ unsigned long long ren_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ int ld_acquire_gpu(const int *p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// Sample index for this CTA: the next ticket, or -1 (with LPDT_ERR_INVALID_ARG recorded) when the control
// block was not zero at launch and the ticket is no sample of this call.  Every thread of the CTA must call.
__device__ __forceinline__ int take_ticket(int *ctl, int nodes, int B, int32_t *dev_status) {
    __shared__ int s_ticket;
    if (threadIdx.x == 0) {
        int tk = atomicAdd(ctl + 3 * nodes, 1);
        if (tk < 0 || tk >= nodes * B) {
            if (dev_status) atomicExch(dev_status, (int32_t)LPDT_ERR_INVALID_ARG);
            tk = -1;
        }
        s_ticket = tk;
    }
    __syncthreads();
    return s_ticket;
}

// Meet the other samples of the node, then round the held sample (n_el fp32 values at `hold`, maximum
// magnitude `cta_max` as found by this thread) to codes at q.  Every thread of the CTA must call.
__device__ __forceinline__ void node_meet_and_quantize(float cta_max, const float *hold, int n_el, int nodes, int B,
                                                       int node, int64_t sample, int *ctl, int8_t *__restrict__ q,
                                                       float *__restrict__ scale, float *__restrict__ amax_out,
                                                       int32_t *dev_status) {
    __shared__ float s_warp[32];
    __shared__ float s_node_amax;
    __shared__ int s_abort;
    const int T = blockDim.x, t = threadIdx.x;
    cta_max = warp_max(cta_max);
    if ((t & 31) == 0) s_warp[t >> 5] = cta_max;
    __syncthreads();                                     // also: the held sample is complete
    if (t < 32) {
        float m = t < ((T + 31) >> 5) ? s_warp[t] : 0.f;
        m = warp_max(m);
        if (t == 0) {
            int *arrive = ctl + node;
            unsigned *bits = reinterpret_cast<unsigned *>(ctl + 2 * nodes + node);
            atomicMax(bits, __float_as_uint(m));         // non-negative floats order like their bit patterns
            __threadfence();
            atomicAdd(arrive, 1);
            int ok = 1;
            if (ld_acquire_gpu(arrive) < B) {
                const unsigned long long t0 = ren_timer_ns();
                unsigned spins = 0;
                while (ld_acquire_gpu(arrive) < B) {
                    __nanosleep(64);
                    if ((++spins & 63u) == 0 && ren_timer_ns() - t0 > kNodeWaitLimitNs) {
                        if (dev_status) atomicExch(dev_status, (int32_t)LPDT_ERR_TIMEOUT);
                        ok = 0;
                        break;
                    }
                }
            }
            s_abort = !ok;
            s_node_amax = __uint_as_float(*reinterpret_cast<volatile unsigned *>(bits));
        }
    }
    __syncthreads();
    if (s_abort) return;
    const float amax = s_node_amax;
    float s, inv;
    if (amax == 0.f) { s = 1.f; inv = 0.f; }
    else { s = __fdiv_rn(amax, 127.f); inv = __fdiv_rn(127.f, amax); }
    const float4 *h4 = reinterpret_cast<const float4 *>(hold);
    char4 *q4 = reinterpret_cast<char4 *>(q + sample * (int64_t)n_el);
    for (int i = t; i < n_el / 4; i += T) {
        const float4 a = h4[i];
        q4[i] = make_char4((signed char)ren_q_sym_rne(a.x, inv), (signed char)ren_q_sym_rne(a.y, inv),
                           (signed char)ren_q_sym_rne(a.z, inv), (signed char)ren_q_sym_rne(a.w, inv));
    }
    if (t == 0) {
        // the last sample of the node to get here clears the node's words (everybody has read the maximum
        // by then) and writes the scale; the last CTA of the grid clears the ticket
        if (atomicAdd(ctl + nodes + node, 1) == B - 1) {
            scale[node] = s;
            if (amax_out) amax_out[node] = amax;
            ctl[node] = 0; ctl[nodes + node] = 0; ctl[2 * nodes + node] = 0;
        }
        __threadfence();
        if (atomicAdd(ctl + 3 * nodes + 1, 1) == nodes * B - 1) { ctl[3 * nodes] = 0; ctl[3 * nodes + 1] = 0; }
    }
}

// Forward that also hands y on as 8-bit codes: one CTA per sample.  The sample arrives in shared memory by
// asynchronous copies (all of it in flight at once), its group extrema are found there, y replaces x in
// place (and goes to global memory as fp32 only when `y` is given), then the node's CTAs meet and every CTA
// rounds its sample.  x is read from global memory once: 4 B in and 1 B out per element when only the codes
// are wanted.  Vector columns of 4 channels only.
template <bool RES>
__global__ void __launch_bounds__(256, 3)
ren_fwd_q8_kernel(int HW, int C, int groups, float eps, float Cst,
                  const float *__restrict__ x, const float *__restrict__ v,
                  const float *__restrict__ gamma, const float *__restrict__ beta, int64_t pstride,
                  int nodes, int B, float *__restrict__ y, float *__restrict__ gmin, float *__restrict__ gmax,
                  int32_t *__restrict__ argmin, int32_t *__restrict__ argmax, float *__restrict__ amax_out,
                  const float *__restrict__ res, int8_t *__restrict__ q, float *__restrict__ scale,
                  int *ctl, int32_t *dev_status, unsigned hold_off) {
    constexpr int V = 4;
    pdl_enter();
    extern __shared__ unsigned char smem_raw[];
    const int T = blockDim.x, t = threadIdx.x;
    Ext *s_mn = reinterpret_cast<Ext *>(smem_raw);
    Ext *s_mx = s_mn + T;
    Ext *g_mn = s_mx + T;
    Ext *g_mx = g_mn + groups;
    float *hold = reinterpret_cast<float *>(smem_raw + hold_off);
    const int CV = C / V, cpg = C / groups;
    const int col = t % CV, row0 = t / CV, rstep = T / CV;
    const int c0 = col * V, grp = c0 / cpg;
    const int n_el = HW * C;
    const int64_t sample = take_ticket(ctl, nodes, B, dev_status);
    if (sample < 0) return;
    const int node = (int)(sample / B);
    {
        const float *xs = x + sample * (int64_t)n_el;
        for (int p = row0; p < HW; p += rstep) cp_async16(hold + p * C + c0, xs + (int64_t)p * C + c0);
        cp_async_commit();
    }
    float vc[V], gc[V], bc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        vc[k] = v[(int64_t)node * pstride + c0 + k];
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
        bc[k] = beta[(int64_t)node * pstride + c0 + k];
    }
    const float *rs = RES ? res + sample * (int64_t)n_el : nullptr;
    float *ys = y ? y + sample * (int64_t)n_el : nullptr;
    cp_async_wait<0>();
    // every thread reads only what its own copies brought: no barrier needed here
    Ext mn, mx; mn.v = INFINITY; mn.idx = 0x7fffffff; mx.v = -INFINITY; mx.idx = 0x7fffffff;
    for (int p = row0; p < HW; p += rstep) {
        const float4 a = *reinterpret_cast<const float4 *>(hold + p * C + c0);
        const float xv[V] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const int idx = p * C + c0 + j;
            if (xv[j] > mx.v) { mx.v = xv[j]; mx.idx = idx; }
            if (xv[j] < mn.v) { mn.v = xv[j]; mn.idx = idx; }
        }
    }
    reduce_groups<V>(mn, mx, s_mn, s_mx, g_mn, g_mx, CV, cpg, groups);
    if (t < groups) {
        const int64_t sg = sample * groups + t;
        gmin[sg] = g_mn[t].v; gmax[sg] = g_mx[t].v; argmin[sg] = g_mn[t].idx; argmax[sg] = g_mx[t].idx;
    }
    const float rng = __fsub_rn(g_mx[grp].v, g_mn[grp].v);
    const float D = __fadd_rn(__fmul_rn(Cst, rng), eps);
    const float invD = __fdiv_rn(1.f, D);
    float ymax = 0.f;
    auto emit = [&](int pp, const float (&rv)[V]) {
        const float4 a = *reinterpret_cast<const float4 *>(hold + pp * C + c0);
        const float xv[V] = {a.x, a.y, a.z, a.w};
        float yv[V];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            float u = __fmul_rn(vc[j], xv[j]);
            float m = __fmul_rn(xv[j], hsig(u));
            yv[j] = __fadd_rn(__fmul_rn(__fmul_rn(gc[j], m), invD), bc[j]);
            if (RES) yv[j] = __fadd_rn(yv[j], rv[j]);
            ymax = fmaxf(ymax, fabsf(yv[j]));
        }
        *reinterpret_cast<float4 *>(hold + pp * C + c0) = make_float4(yv[0], yv[1], yv[2], yv[3]);
        if (ys) VecLoad<V>::st(ys + (int64_t)pp * C + c0, yv);
    };
    constexpr int kU = RES ? 4 : 1;
    int p = row0;
    for (; p + (kU - 1) * rstep < HW; p += kU * rstep) {
        float rv[kU][V];
#pragma unroll
        for (int j = 0; j < kU; ++j)
            if (RES) VecLoad<V>::ld(rs + (int64_t)(p + j * rstep) * C + c0, rv[j]);
#pragma unroll
        for (int j = 0; j < kU; ++j) emit(p + j * rstep, rv[j]);
    }
    for (; p < HW; p += rstep) {
        float rv[V];
        if (RES) VecLoad<V>::ld(rs + (int64_t)p * C + c0, rv);
        emit(p, rv);
    }
    node_meet_and_quantize(ymax, hold, n_el, nodes, B, node, sample, ctl, q, scale, amax_out, dev_status);
}

// Backward of one sample by the whole CTA: the local term of dx and the correction at the group extrema go to
// `dxs` (the sample's place in global memory, or a copy of it held in shared memory), the per-sample partial
// sums of the parameter gradients to `acc`; `dmax` takes max|dx|.  Leaves no asynchronous copy pending.
// DEPTH > 0 (V = 4 only): every thread keeps its next DEPTH rows of x and dy in flight as asynchronous copies into
// a private shared-memory ring, so the bytes in flight per SM (what a streaming kernel of 13-60 us lives
// on) no longer depend on the register budget; the first DEPTH rows are requested before the group
// statistics and parameters are read.  DEPTH = 0: rows are loaded into registers, two per trip.
// XHOLD (with DEPTH > 0): the sample's x has been requested into `dxs` (shared memory) as the oldest pending
// copy group; only dy goes through the ring, and dx overwrites x in place.
template <int V, int DEPTH, bool XHOLD = false>
__device__ __forceinline__ void ren_bwd_sample(unsigned char *smem_raw, int HW, int C, int groups, float eps, float Cst,
                                               const float *__restrict__ dy, const float *__restrict__ x,
                                               const float *__restrict__ v, const float *__restrict__ gamma,
                                               int64_t pstride, const float *__restrict__ gmin,
                                               const float *__restrict__ gmax, const int32_t *__restrict__ argmin,
                                               const int32_t *__restrict__ argmax, double *__restrict__ acc,
                                               int64_t sample, int node, float *dxs, float &dmax) {
    const int T = blockDim.x, t = threadIdx.x;
    // When the column count divides the warp, lanes that share a column are folded with shuffles and
    // every warp keeps its own partial sums (no atomics, fixed order); otherwise one shared set of
    // fp64 accumulators takes atomic adds.
    const bool fold = ((C / V) <= 32) && (32 % (C / V) == 0);
    const int nsets = fold ? (T >> 5) : 1;
    double *s_ch = reinterpret_cast<double *>(smem_raw);      // [nsets][3][C]
    double *s_S = s_ch + nsets * 3 * C;                       // [T]
    double *g_S = s_S + T;                                    // [groups]
    // ring of DEPTH slots: slot s holds, for every thread, 16 bytes of x and 16 bytes of dy (XHOLD: of dy)
    constexpr int kPerSlot = XHOLD ? 1 : 2;
    float4 *ring = reinterpret_cast<float4 *>(smem_raw + (((size_t)(nsets * 3 * C + T + groups) * sizeof(double) + 15) & ~(size_t)15));
    const int CV = C / V, cpg = C / groups;
    const int col = t % CV, row0 = t / CV, rstep = T / CV;
    const int c0 = col * V, grp = c0 / cpg;
    const float *xs = x + sample * (int64_t)HW * C;
    const float *dys = dy + sample * (int64_t)HW * C;
    const int iters = (HW - 1) / rstep + 1;          // same trip count for every thread (rows are predicated)
    auto request = [&](int j) {                      // row j of this thread -> slot j % DEPTH; one group per row, even when empty
        if (DEPTH > 0) {
            const int p = row0 + j * rstep;
            if (j < iters && p < HW) {
                float4 *slot = ring + (size_t)(j % (DEPTH > 0 ? DEPTH : 1)) * kPerSlot * T + t;
                if (!XHOLD) cp_async16(slot, xs + (int64_t)p * C + c0);
                cp_async16(slot + (kPerSlot - 1) * T, dys + (int64_t)p * C + c0);
            }
            cp_async_commit();
        }
    };
    if (DEPTH > 0) {
#pragma unroll
        for (int j = 0; j < (DEPTH > 0 ? DEPTH : 1); ++j) request(j);
    }
    for (int i = t; i < nsets * 3 * C; i += T) s_ch[i] = 0.0;

    const int64_t sg = sample * groups + grp;
    const float rng = __fsub_rn(gmax[sg], gmin[sg]);
    const float D = __fadd_rn(__fmul_rn(Cst, rng), eps);
    const float invD = __fdiv_rn(1.f, D);
    const float sixth = __fdiv_rn(1.f, 6.f);
    float vc[V], gc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        vc[k] = v[(int64_t)node * pstride + c0 + k];
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
    }
    // Every sum is accumulated in double term by term: S feeds dx (and through it the next
    // quantizer), and the per-channel parameter-gradient sums then differ from a serial double
    // sum of the same fp32 terms only by double rounding noise.
    // max|dx| for the consumer's quantizer: the two extremum positions are left out here and
    // added after their correction
    const int g_amx = argmax[sg], g_amn = argmin[sg];
    double S = 0.0;
    double fb[V], fg[V], fv[V];
#pragma unroll
    for (int k = 0; k < V; ++k) { fb[k] = 0.0; fg[k] = 0.0; fv[k] = 0.0; }
    __syncthreads();   // s_ch zeroed
    auto term = [&](int p, const float (&xv)[V], const float (&dv_)[V]) {
        float o[V];
#pragma unroll
        for (int k = 0; k < V; ++k) {
            float u = __fmul_rn(vc[k], xv[k]);
            float hs = hsig(u);
            float hp = (u > -3.f && u < 3.f) ? sixth : 0.f;
            float m = __fmul_rn(xv[k], hs);
            float tt = __fmul_rn(dv_[k], gc[k]);
            S += (double)__fmul_rn(tt, m);
            o[k] = __fmul_rn(__fmul_rn(tt, __fadd_rn(hs, __fmul_rn(u, hp))), invD);
            const int idx = p * C + c0 + k;
            if (idx != g_amx && idx != g_amn) dmax = fmaxf(dmax, fabsf(o[k]));
            fb[k] += (double)dv_[k];
            fg[k] += (double)__fmul_rn(dv_[k], __fmul_rn(m, invD));
            fv[k] += (double)__fmul_rn(__fmul_rn(__fmul_rn(tt, __fmul_rn(xv[k], xv[k])), hp), invD);
        }
        VecLoad<V>::st(dxs + (int64_t)p * C + c0, o);
    };
    if (DEPTH > 0) {
        for (int j = 0; j < iters; ++j) {
            cp_async_wait<(DEPTH > 0 ? DEPTH - 1 : 0)>();                // the oldest pending group, row j, has landed
            const int p = row0 + j * rstep;
            if (p < HW) {
                const float4 *slot = ring + (size_t)(j % (DEPTH > 0 ? DEPTH : 1)) * kPerSlot * T + t;
                const float4 a = XHOLD ? *reinterpret_cast<const float4 *>(dxs + (size_t)p * C + c0) : slot[0];
                const float4 b = slot[(kPerSlot - 1) * T];
                const float xa[4] = {a.x, a.y, a.z, a.w}, da[4] = {b.x, b.y, b.z, b.w};
                term(p, reinterpret_cast<const float (&)[V]>(xa), reinterpret_cast<const float (&)[V]>(da));
            }
            request(j + DEPTH);                                  // the slot just read takes row j + DEPTH
        }
        cp_async_wait<0>();
    }
    // DEPTH = 0, two rows per trip: four independent 16-byte loads in flight per thread
    for (int i = 0; DEPTH == 0 && i < iters; i += 2) {
        const int p0 = row0 + i * rstep, p1 = p0 + rstep;
        const bool ok0 = p0 < HW, ok1 = (i + 1 < iters) && (p1 < HW);
        float xa[V], da[V], xb[V], db[V];
        if (ok0) { VecLoad<V>::ld(xs + (int64_t)p0 * C + c0, xa); VecLoad<V>::ld(dys + (int64_t)p0 * C + c0, da); }
        if (ok1) { VecLoad<V>::ld(xs + (int64_t)p1 * C + c0, xb); VecLoad<V>::ld(dys + (int64_t)p1 * C + c0, db); }
        if (ok0) term(p0, xa, da);
        if (ok1) term(p1, xb, db);
    }
#pragma unroll
    for (int k = 0; k < V; ++k) {
        double a = fv[k], b = fg[k], c = fb[k];
        if (fold) {
            for (int o = 16; o >= CV; o >>= 1) {
                a += __shfl_xor_sync(0xffffffffu, a, o);
                b += __shfl_xor_sync(0xffffffffu, b, o);
                c += __shfl_xor_sync(0xffffffffu, c, o);
            }
            if ((t & 31) < CV) {                 // this lane alone owns these three slots of its warp's set
                double *mine = s_ch + (size_t)(t >> 5) * 3 * C + c0 + k;
                mine[0] = a; mine[C] = b; mine[2 * C] = c;
            }
        } else {
            atomicAdd(&s_ch[0 * C + c0 + k], a);
            atomicAdd(&s_ch[1 * C + c0 + k], b);
            atomicAdd(&s_ch[2 * C + c0 + k], c);
        }
    }
    s_S[t] = S;
    __syncthreads();
    {   // fixed-order group sums: one warp per group, lanes stride the members
        const int lane = t & 31, warp = t >> 5, nw = T >> 5;
        const int cols = cpg / V, rows = T / CV, members = cols * rows;
        for (int g = warp; g < groups; g += nw) {
            double a = 0.0;
            for (int m = lane; m < members; m += 32) a += s_S[(m / cols) * CV + g * cols + (m % cols)];
            a = warp_sum(a);
            if (lane == 0) g_S[g] = a;
        }
    }
    for (int i = t; i < 3 * C; i += T) {      // warp sets in order; summed over the batch by the finalize kernel
        double a = s_ch[i];
        for (int w = 1; w < nsets; ++w) a += s_ch[(size_t)w * 3 * C + i];
        acc[sample * 3 * C + i] = a;
    }
    __syncthreads();
    // The group sum only enters dx at the two extremum positions: one thread per group
    // applies the correction to the local term already stored there (same operation order
    // as a fused evaluation: local term first, then -coef at argmax, +coef at argmin).
    if (t < groups) {
        const int64_t sgg = sample * groups + t;
        const int amx = argmax[sgg], amn = argmin[sgg];
        if (amx != amn) {
            const float rng_g = __fsub_rn(gmax[sgg], gmin[sgg]);
            const float invDg = __fdiv_rn(1.f, __fadd_rn(__fmul_rn(Cst, rng_g), eps));
            float coef = __fmul_rn(Cst, (float)g_S[t]);
            coef = __fmul_rn(coef, invDg);
            coef = __fmul_rn(coef, invDg);
            const float va = __fsub_rn(dxs[amx], coef), vb = __fadd_rn(dxs[amn], coef);
            dxs[amx] = va; dxs[amn] = vb;
            dmax = fmaxf(dmax, fmaxf(fabsf(va), fabsf(vb)));
        } else {
            dmax = fmaxf(dmax, fabsf(dxs[amx]));
        }
    }
}

// One CTA per (node, sample).  MAXT = 256: three CTAs per SM at 80 registers (the thirteen double accumulators
// of a thread stay in registers); MAXT = 512 serves the rare plans with more than 256 threads.
template <int V, int MAXT, int DEPTH>
__global__ void __launch_bounds__(MAXT, MAXT == 256 ? 3 : 1)
ren_bwd_kernel(int HW, int C, int groups, float eps, float Cst,
               const float *__restrict__ dy, const float *__restrict__ x,
               const float *__restrict__ v, const float *__restrict__ gamma, int64_t pstride, int B,
               const float *__restrict__ gmin, const float *__restrict__ gmax,
               const int32_t *__restrict__ argmin, const int32_t *__restrict__ argmax,
               float *__restrict__ dx, double *__restrict__ acc /*[nodes][B][3][C] per-sample partial sums*/,
               float *__restrict__ amax_out) {
    pdl_enter();
    extern __shared__ unsigned char smem_raw[];
    const int64_t sample = blockIdx.x;
    const int node = (int)(sample / B);
    float dmax = 0.f;
    ren_bwd_sample<V, DEPTH>(smem_raw, HW, C, groups, eps, Cst, dy, x, v, gamma, pstride, gmin, gmax, argmin, argmax, acc,
                             sample, node, dx + sample * (int64_t)HW * C, dmax);
    if (amax_out) block_amax_to(dmax, amax_out + node);
}

// Backward that hands the layer gradient on as 8-bit codes: one CTA per sample.  x arrives in shared memory
// by asynchronous copies (all of it in flight at once), dy through the ring; dx replaces x in place and never
// reaches global memory as fp32 - the node's CTAs meet and every CTA rounds its sample: 8 B read and 1 B
// written per element instead of 8 + 4 and another 4 + 1 in a separate quantizer launch.  The codes equal
// those of the two-kernel form bit for bit (same dx, same maximum, same rounding).
template <int MAXT, int MINB, int DEPTH>
__global__ void __launch_bounds__(MAXT, MINB)
ren_bwd_q8_kernel(int HW, int C, int groups, float eps, float Cst,
                  const float *__restrict__ dy, const float *__restrict__ x,
                  const float *__restrict__ v, const float *__restrict__ gamma, int64_t pstride, int nodes, int B,
                  const float *__restrict__ gmin, const float *__restrict__ gmax,
                  const int32_t *__restrict__ argmin, const int32_t *__restrict__ argmax,
                  double *__restrict__ acc, int8_t *__restrict__ q, float *__restrict__ scale,
                  float *__restrict__ amax_out, int *ctl, int32_t *dev_status,
                  unsigned hold_off /*byte offset of the held sample*/) {
    constexpr int V = 4;
    pdl_enter();
    extern __shared__ unsigned char smem_raw[];
    const int T = blockDim.x, t = threadIdx.x;
    const int64_t sample = take_ticket(ctl, nodes, B, dev_status);
    if (sample < 0) return;
    const int node = (int)(sample / B);
    float *hold = reinterpret_cast<float *>(smem_raw + hold_off);
    const int n_el = HW * C;
    {
        const int CV = C / V, col = t % CV, row0 = t / CV, rstep = T / CV, c0 = col * V;
        const float *xs = x + sample * (int64_t)n_el;
        for (int p = row0; p < HW; p += rstep) cp_async16(hold + p * C + c0, xs + (int64_t)p * C + c0);
        cp_async_commit();
    }
    float dmax = 0.f;
    ren_bwd_sample<V, DEPTH, true>(smem_raw, HW, C, groups, eps, Cst, dy, x, v, gamma, pstride, gmin, gmax, argmin, argmax,
                                   acc, sample, node, hold, dmax);
    node_meet_and_quantize(dmax, hold, n_el, nodes, B, node, sample, ctl, q, scale, amax_out, dev_status);
}

// Sum the per-sample partials of a node and round once.  One warp per output: lane l adds samples
// l, l+32, ... in order and the lanes combine in a fixed shuffle tree, so the result is deterministic.
__global__ void ren_bwd_finalize(const double *__restrict__ acc, int nodes, int B, int C,
                                 float *__restrict__ dv, float *__restrict__ dgamma,
                                 float *__restrict__ dbeta, int64_t gstride) {
    pdl_enter();
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (i >= nodes * 3 * C) return;
    const int node = i / (3 * C), j = i % (3 * C), which = j / C, c = j % C;
    const double *a = acc + (int64_t)node * B * 3 * C + j;
    double s = 0.0;
    for (int b = lane; b < B; b += 32) s += a[(int64_t)b * 3 * C];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if (lane == 0) {
        float *dst = which == 0 ? dv : which == 1 ? dgamma : dbeta;
        dst[(int64_t)node * gstride + c] = (float)s;
    }
}

// The same reduction for many layers in one launch: layer l owns warps [start[l], start[l+1]).
constexpr int kMaxRenBatch = 64;
struct RenBatch {
    int count;
    const double *acc[kMaxRenBatch];      // per-sample partial sums of the layer [nodes][B][3][C]
    int C[kMaxRenBatch];
    long long off[kMaxRenBatch];          // element offset of the layer's v gradient inside a node's gradient row
    int start[kMaxRenBatch + 1];          // first warp of each layer
};
__global__ void ren_bwd_finalize_batch(RenBatch rb, int nodes, int B, float *__restrict__ grads, int64_t gstride) {
    pdl_enter();
    const int w = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (w >= rb.start[rb.count]) return;
    int l = 0;
    while (w >= rb.start[l + 1]) ++l;                       // at most 64 layers: a short scan, uniform per warp
    const int C = rb.C[l], i = w - rb.start[l];
    const int node = i / (3 * C), j = i % (3 * C), which = j / C, c = j % C;
    const double *a = rb.acc[l] + (int64_t)node * B * 3 * C + j;
    double s = 0.0;
    for (int b = lane; b < B; b += 32) s += a[(int64_t)b * 3 * C];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    // the layer's three parameter vectors sit back to back in the gradient row: v, gamma, beta
    if (lane == 0) grads[(int64_t)node * gstride + rb.off[l] + (int64_t)which * C + c] = (float)s;
}

struct RenPlan { int V, threads; };

static bool plan(int C, int groups, bool aligned16, RenPlan *pl, int cap = 256) {
    const int cpg = C / groups;
    int V = (aligned16 && C % 4 == 0 && cpg % 4 == 0) ? 4 : 1;
    int CV = C / V;
    if (CV > 512) return false;
    pl->V = V;
    pl->threads = CV <= cap ? CV * (cap / CV) : (CV <= 256 ? CV * (256 / CV) : CV);
    if (pl->threads % 32) {                      // keep whole warps: pad down to a multiple of lcm
        int th = pl->threads;
        while (th > 0 && (th % 32 || th % CV)) th -= CV;
        if (th <= 0) return false;
        pl->threads = th;
    }
    return true;
}

// CTAs per sample of the forward kernel (cluster size: 1, 2, 4 or 8).  Two reasons to split a sample:
// the samples in flight (one per resident CTA or cluster, 4 CTAs of 256 threads per SM) should fit
// well inside the 126 MB L2 together with the output being written, so that pass 2 reads from L2; and a
// small batch should still give every SM a few CTAs.  LPDT_REN_CLUSTER=1|2|4|8 overrides (parity tests).
static int ren_cluster_size(int64_t samples, int HW, int C, int rstep) {
    static int forced = -1;
    if (forced < 0) { const char *e = getenv("LPDT_REN_CLUSTER"); forced = e ? atoi(e) : 0; }
    const int rows = (int)ceil_div(HW, rstep);               // thread rows of a sample
    int cap = 1;
    while (cap < 8 && cap * 2 <= rows) cap *= 2;             // every CTA keeps at least one thread row
    if (forced == 1 || forced == 2 || forced == 4 || forced == 8) return forced < cap ? forced : cap;
    const double sample_bytes = (double)HW * C * 4.0;
    const int64_t slots = (int64_t)kNumSMs * 4;
    int R = 1;
    while (R < cap) {
        const int64_t in_flight = samples < slots / R ? samples : slots / R;
        const bool l2_ok = (double)in_flight * sample_bytes <= 40.0 * 1024 * 1024;
        const bool fills = samples * R >= 2 * (int64_t)kNumSMs;
        if (l2_ok && fills) break;
        R *= 2;
    }
    return R;
}

static float ren_const(int cpg) { return (float)(1.0 / sqrt(2.0 * log((double)cpg))); }

}  // namespace lpdt

using namespace lpdt;

extern "C" lpdt_status lpdt_range_evonorm_fwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                              int32_t groups, float eps, const float *x, const float *v,
                                              const float *gamma, const float *beta, int64_t pstride,
                                              float *y, float *gmin, float *gmax, int32_t *argmin,
                                              int32_t *argmax, float *amax_out, const float *res, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && groups > 0);
    LPDT_CHECK_ARG(C % groups == 0 && C / groups >= 2);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && v && gamma && beta && y && gmin && gmax && argmin && argmax);
    LPDT_CHECK_ARG(pstride >= C || nodes == 1);
    if ((int64_t)H * W * C > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    RenPlan pl;
    static int tforce = -1;
    if (tforce < 0) { const char *e = getenv("LPDT_REN_FWD_THREADS"); tforce = e ? atoi(e) : 0; }
    if (!plan(C, groups, aligned(x, 16) && aligned(y, 16) && (!res || aligned(res, 16)), &pl, tforce == 128 ? 128 : 256))
        return LPDT_ERR_UNSUPPORTED;
    size_t smem = (size_t)(2 * pl.threads + 4 * groups) * sizeof(Ext);
    if (smem > 48 * 1024) return LPDT_ERR_UNSUPPORTED;
    const float Cst = ren_const(C / groups);
    const int R = ren_cluster_size((int64_t)nodes * B, H * W, C, pl.threads / (C / pl.V));
    const int rstep = pl.threads / (C / pl.V);
    const int ppc = (int)ceil_div(ceil_div(H * W, R), rstep) * rstep;       // whole thread rows per CTA
    if ((int64_t)nodes * B * R > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    dim3 grid((unsigned)((int64_t)nodes * B * R));
    using Fn = void (*)(int, int, int, float, float, const float *, const float *, const float *, const float *, int64_t,
                        int, float *, float *, float *, int32_t *, int32_t *, float *, const float *, int, int);
    static const Fn fns[2][2] = {{ren_fwd_kernel<1, false>, ren_fwd_kernel<1, true>},
                                 {ren_fwd_kernel<4, false>, ren_fwd_kernel<4, true>}};
    launch_k_cluster(fns[pl.V == 4 ? 1 : 0][res ? 1 : 0], grid, pl.threads, smem, as_stream(stream), R, H * W, C, groups, eps,
                     Cst, x, v, gamma, beta, pstride, B, y, gmin, gmax, argmin, argmax, amax_out, res, R, ppc);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" size_t lpdt_range_evonorm_bwd_workspace_size(int32_t nodes, int32_t B, int32_t C) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)(B > 0 ? B : 1) * 3 * (size_t)(C > 0 ? C : 1) *
                    sizeof(double), 256);
}

extern "C" lpdt_status lpdt_range_evonorm_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                              int32_t groups, float eps, const float *dy, const float *x,
                                              const float *v, const float *gamma, int64_t pstride,
                                              const float *gmin, const float *gmax,
                                              const int32_t *argmin, const int32_t *argmax,
                                              float *dx, float *dv, float *dgamma, float *dbeta,
                                              int64_t gstride, float *amax_out, void *ws, size_t ws_bytes,
                                              void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && groups > 0);
    LPDT_CHECK_ARG(C % groups == 0 && C / groups >= 2);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dy && x && v && gamma && gmin && gmax && argmin && argmax && dx);
    const bool deferred = !dv && !dgamma && !dbeta;       // parameter gradients left as partial sums in ws
    LPDT_CHECK_ARG(deferred || (dv && dgamma && dbeta));
    LPDT_CHECK_ARG((pstride >= C && (deferred || gstride >= C)) || nodes == 1);
    if ((int64_t)H * W * C > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < lpdt_range_evonorm_bwd_workspace_size(nodes, B, C) || !aligned(ws, 8))
        return LPDT_ERR_WORKSPACE;
    RenPlan pl;
    // Samples of up to 64 KB with few channel columns run as 128-thread CTAs, six per SM instead of three: the
    // serial head and tail of such a short CTA (statistics, reductions, the patch at the extrema) then overlap
    // with the streaming phase of more neighbours (measured: 16x16x32 samples 0.041 -> 0.033 ms, 32x32x16
    // 0.058 -> 0.053 ms; 256 KB samples lose 5 %).  LPDT_REN_BWD_THREADS=128|256 overrides (A/B timing).
    static int tforce = -1;
    if (tforce < 0) { const char *e = getenv("LPDT_REN_BWD_THREADS"); tforce = e ? atoi(e) : 0; }
    const bool v4 = aligned(x, 16) && aligned(dy, 16) && aligned(dx, 16) && C % 4 == 0 && (C / groups) % 4 == 0;
    int cap = ((int64_t)H * W * C * 4 <= 64 * 1024 && C / (v4 ? 4 : 1) <= 32) ? 128 : 256;
    if (tforce == 128 || tforce == 256) cap = tforce;
    if (!plan(C, groups, aligned(x, 16) && aligned(dy, 16) && aligned(dx, 16), &pl, cap)) return LPDT_ERR_UNSUPPORTED;
    const int cv = C / pl.V;
    const int nsets = (cv <= 32 && 32 % cv == 0) ? pl.threads / 32 : 1;      // as in the kernel
    size_t smem = (size_t)(nsets * 3 * C + pl.threads + groups) * sizeof(double);
    if (smem > 48 * 1024) return LPDT_ERR_UNSUPPORTED;
    // rows in flight per thread (V = 4): 8 with up to 256 threads, or 6 when the sums' shared memory would push a
    // CTA past its share of the SM's shared memory (three CTAs per SM, six of 128 threads) and a thread has more
    // than 8 rows anyway (with 8 or fewer, all of a thread's rows are requested at once); 4 beyond 256 threads
    int depth = pl.V == 4 ? (pl.threads <= 256 ? 8 : 4) : 0;
    const size_t third = (size_t)(227 * 1024) / (pl.threads <= 128 ? 6 : 3) - 1024;
    const int rows_per_thread = (int)ceil_div((int64_t)H * W, pl.threads / cv);
    if (depth == 8 && rows_per_thread > 8 && align_up(smem, 16) + (size_t)8 * 2 * pl.threads * 16 > third) depth = 6;
    smem = align_up(smem, 16) + (size_t)depth * 2 * pl.threads * 16;
    cudaStream_t st = as_stream(stream);
    double *acc = (double *)ws;
    const float Cst = ren_const(C / groups);
    dim3 grid((unsigned)((int64_t)nodes * B));
    using Fn = void (*)(int, int, int, float, float, const float *, const float *, const float *, const float *, int64_t, int,
                        const float *, const float *, const int32_t *, const int32_t *, float *, double *, float *);
    static const Fn fns[2][3] = {{ren_bwd_kernel<1, 256, 0>, ren_bwd_kernel<1, 512, 0>, ren_bwd_kernel<1, 256, 0>},
                                 {ren_bwd_kernel<4, 256, 8>, ren_bwd_kernel<4, 512, 4>, ren_bwd_kernel<4, 256, 6>}};
    static PerDeviceOnce attr;
    int dev;
    if (attr.pending(&dev)) {
        for (int i = 0; i < 3; ++i) {
            LPDT_CUDA(cudaFuncSetAttribute(fns[1][i], cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
            // the rings of three (six) resident CTAs need nearly all of the SM's shared memory
            LPDT_CUDA(cudaFuncSetAttribute(fns[1][i], cudaFuncAttributePreferredSharedMemoryCarveout,
                                           (int)cudaSharedmemCarveoutMaxShared));
        }
        attr.mark(dev);
    }
    launch_k(fns[pl.V == 4 ? 1 : 0][pl.threads > 256 ? 1 : depth == 6 ? 2 : 0], grid, pl.threads, smem, st, H * W, C, groups, eps, Cst, dy, x,
             v, gamma, pstride, B, gmin, gmax, argmin, argmax, dx, acc, amax_out);
    LPDT_LAUNCH_CHECK();
    if (deferred) return LPDT_OK;
    launch_k(ren_bwd_finalize, (nodes * 3 * C + 7) / 8, 256, 0, st, acc, nodes, B, C, dv, dgamma, dbeta, gstride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

namespace lpdt {

using RenFwdQ8Fn = void (*)(int, int, int, float, float, const float *, const float *, const float *, const float *, int64_t,
                            int, int, float *, float *, float *, int32_t *, int32_t *, float *, const float *, int8_t *,
                            float *, int *, int32_t *, unsigned);
using RenBwdQ8Fn = void (*)(int, int, int, float, float, const float *, const float *, const float *, const float *, int64_t,
                            int, int, const float *, const float *, const int32_t *, const int32_t *, double *, int8_t *,
                            float *, float *, int *, int32_t *, unsigned);

struct RenQ8Plan { int threads, depth; unsigned hold_off; size_t smem; RenBwdQ8Fn bwd; };

static int q8_threads_forced() {
    static int tforce = -1;
    if (tforce < 0) { const char *e = getenv("LPDT_REN_Q8_THREADS"); tforce = e ? atoi(e) : 0; }
    return tforce;
}

// CTAs of this kernel, CTA size and shared memory that can be resident on the device at once (asked of the
// driver once per shape and device).  The kernels that meet per node need room for 2 B of them.
static int q8_resident_ctas(const void *fn, int threads, size_t smem) {
    static std::mutex mu;
    static std::map<std::tuple<int, const void *, int, size_t>, int> seen;
    std::lock_guard<std::mutex> lock(mu);
    int d = 0;
    (void)cudaGetDevice(&d);
    const auto key = std::make_tuple(d, fn, threads, smem);
    auto it = seen.find(key);
    if (it == seen.end()) {
        int per_sm = 0, sms = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, smem) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, d) != cudaSuccess) {
            (void)cudaGetLastError();
            per_sm = 0;
        }
        it = seen.emplace(key, per_sm * sms).first;
    }
    return it->second;
}

static bool q8_kernel_attrs(const void *fn) {
    return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024) == cudaSuccess &&
           cudaFuncSetAttribute(fn, cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared) ==
               cudaSuccess;
}

// Launch shape of the forward that writes 8-bit codes: shared memory [extrema scratch | the sample].
static bool ren_fwd_q8_plan(int B, int HW, int C, int groups, bool res, RenQ8Plan *out) {
    if (C % 4 || (C / groups) % 4 || (int64_t)HW * C > (1 << 24)) return false;
    static PerDeviceOnce attr;
    int dev;
    if (attr.pending(&dev)) {
        if (!q8_kernel_attrs((const void *)ren_fwd_q8_kernel<false>) || !q8_kernel_attrs((const void *)ren_fwd_q8_kernel<true>)) {
            (void)cudaGetLastError();
            return false;
        }
        attr.mark(dev);
    }
    const void *fn = res ? (const void *)ren_fwd_q8_kernel<true> : (const void *)ren_fwd_q8_kernel<false>;
    const size_t hold = (size_t)HW * C * 4;
    int cap = hold <= 16 * 1024 ? 128 : 256;
    const int tf = q8_threads_forced();
    if (tf == 128 || tf == 256) cap = tf;
    RenPlan pl;
    if (!plan(C, groups, true, &pl, cap) || pl.V != 4 || pl.threads > 256) return false;
    const size_t scratch = align_up((size_t)(2 * pl.threads + 2 * groups) * sizeof(Ext), 16);
    const size_t smem = scratch + hold;
    if (scratch > 48 * 1024 || smem > 226 * 1024) return false;
    if (q8_resident_ctas(fn, pl.threads, smem) < 2 * B) return false;
    out->threads = pl.threads; out->depth = 0; out->hold_off = (unsigned)scratch; out->smem = smem; out->bwd = nullptr;
    return true;
}

// Launch shape of the backward that writes 8-bit codes: shared memory [sums | dy ring | the sample].
static bool ren_bwd_q8_plan(int B, int HW, int C, int groups, RenQ8Plan *out) {
    if (C % 4 || (C / groups) % 4 || (int64_t)HW * C > (1 << 24)) return false;
    // <threads, CTAs per SM the register budget is compiled for, ring depth>
    static const RenBwdQ8Fn fns[3] = {ren_bwd_q8_kernel<256, 3, 8>, ren_bwd_q8_kernel<256, 3, 4>, ren_bwd_q8_kernel<384, 2, 4>};
    static PerDeviceOnce attr;
    int dev;
    if (attr.pending(&dev)) {
        for (int i = 0; i < 3; ++i)
            if (!q8_kernel_attrs((const void *)fns[i])) { (void)cudaGetLastError(); return false; }
        attr.mark(dev);
    }
    const size_t hold = (size_t)HW * C * 4;
    int cap = hold <= 32 * 1024 && C / 4 <= 32 ? 128 : 256;
    const int tf = q8_threads_forced();
    if (tf == 128 || tf == 256 || tf == 384) cap = tf;
    RenPlan pl;
    if (!plan(C, groups, true, &pl, cap) || pl.V != 4 || pl.threads > 384) return false;
    const int cv = C / 4;
    const int nsets = (cv <= 32 && 32 % cv == 0) ? pl.threads / 32 : 1;
    const size_t sums = align_up((size_t)(nsets * 3 * C + pl.threads + groups) * sizeof(double), 16);
    if (sums > 48 * 1024) return false;
    static int dforce = -1;
    if (dforce < 0) { const char *e = getenv("LPDT_REN_Q8_DEPTH"); dforce = e ? atoi(e) : 0; }
    int depth = pl.threads > 256 ? 4 : 8;
    if (dforce == 4 || (dforce == 8 && pl.threads <= 256)) depth = dforce;
    const size_t smem = sums + (size_t)depth * pl.threads * 16 + hold;
    if (smem > 226 * 1024) return false;
    RenBwdQ8Fn fn = pl.threads > 256 ? fns[2] : depth == 8 ? fns[0] : fns[1];
    if (q8_resident_ctas((const void *)fn, pl.threads, smem) < 2 * B) return false;
    out->threads = pl.threads; out->depth = depth; out->hold_off = (unsigned)(sums + (size_t)depth * pl.threads * 16);
    out->smem = smem; out->bwd = fn;
    return true;
}

}  // namespace lpdt

extern "C" size_t lpdt_range_evonorm_q8_ctl_size(int32_t nodes) {
    return align_up((size_t)(3 * (size_t)(nodes > 0 ? nodes : 1) + 2) * sizeof(int32_t), 256);
}

extern "C" int32_t lpdt_range_evonorm_fwd_q8_fits(int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups) {
    if (B <= 0 || H <= 0 || W <= 0 || C <= 0 || groups <= 0 || C % groups || C / groups < 2) return 0;
    if ((int64_t)H * W * C > 0x7fffffff) return 0;
    RenQ8Plan qp;
    return ren_fwd_q8_plan(B, H * W, C, groups, false, &qp) && ren_fwd_q8_plan(B, H * W, C, groups, true, &qp) ? 1 : 0;
}

extern "C" lpdt_status lpdt_range_evonorm_fwd_q8(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                                 int32_t groups, float eps, const float *x, const float *v,
                                                 const float *gamma, const float *beta, int64_t pstride,
                                                 float *y, float *gmin, float *gmax, int32_t *argmin,
                                                 int32_t *argmax, float *amax_out, const float *res, int8_t *q,
                                                 float *scale, void *ctl, size_t ctl_bytes, int32_t *dev_status,
                                                 void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && groups > 0);
    LPDT_CHECK_ARG(C % groups == 0 && C / groups >= 2);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && v && gamma && beta && gmin && gmax && argmin && argmax && q && scale);
    LPDT_CHECK_ARG(pstride >= C || nodes == 1);
    if ((int64_t)H * W * C > 0x7fffffff || (int64_t)nodes * B > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    if (!ctl || ctl_bytes < lpdt_range_evonorm_q8_ctl_size(nodes) || !aligned(ctl, 4)) return LPDT_ERR_WORKSPACE;
    if (!aligned(x, 16) || (y && !aligned(y, 16)) || (res && !aligned(res, 16)) || !aligned(q, 4)) return LPDT_ERR_UNSUPPORTED;
    RenQ8Plan qp;
    if (!ren_fwd_q8_plan(B, H * W, C, groups, res != nullptr, &qp)) return LPDT_ERR_UNSUPPORTED;
    const float Cst = ren_const(C / groups);
    RenFwdQ8Fn fn = res ? ren_fwd_q8_kernel<true> : ren_fwd_q8_kernel<false>;
    launch_k(fn, dim3((unsigned)((int64_t)nodes * B)), qp.threads, qp.smem, as_stream(stream), H * W, C, groups, eps, Cst, x, v,
             gamma, beta, pstride, nodes, B, y, gmin, gmax, argmin, argmax, amax_out, res, q, scale, (int *)ctl, dev_status,
             qp.hold_off);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" int32_t lpdt_range_evonorm_bwd_q8_fits(int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups) {
    if (B <= 0 || H <= 0 || W <= 0 || C <= 0 || groups <= 0 || C % groups || C / groups < 2) return 0;
    if ((int64_t)H * W * C > 0x7fffffff) return 0;
    RenQ8Plan qp;
    return ren_bwd_q8_plan(B, H * W, C, groups, &qp) ? 1 : 0;
}

extern "C" lpdt_status lpdt_range_evonorm_bwd_q8(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C,
                                                 int32_t groups, float eps, const float *dy, const float *x,
                                                 const float *v, const float *gamma, int64_t pstride,
                                                 const float *gmin, const float *gmax,
                                                 const int32_t *argmin, const int32_t *argmax,
                                                 int8_t *q, float *scale, float *dv, float *dgamma, float *dbeta,
                                                 int64_t gstride, float *amax_out, void *ws, size_t ws_bytes,
                                                 void *ctl, size_t ctl_bytes, int32_t *dev_status, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && groups > 0);
    LPDT_CHECK_ARG(C % groups == 0 && C / groups >= 2);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dy && x && v && gamma && gmin && gmax && argmin && argmax && q && scale);
    const bool deferred = !dv && !dgamma && !dbeta;
    LPDT_CHECK_ARG(deferred || (dv && dgamma && dbeta));
    LPDT_CHECK_ARG((pstride >= C && (deferred || gstride >= C)) || nodes == 1);
    if ((int64_t)H * W * C > 0x7fffffff || (int64_t)nodes * B > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < lpdt_range_evonorm_bwd_workspace_size(nodes, B, C) || !aligned(ws, 8))
        return LPDT_ERR_WORKSPACE;
    if (!ctl || ctl_bytes < lpdt_range_evonorm_q8_ctl_size(nodes) || !aligned(ctl, 4)) return LPDT_ERR_WORKSPACE;
    if (!aligned(x, 16) || !aligned(dy, 16) || !aligned(q, 4)) return LPDT_ERR_UNSUPPORTED;
    RenQ8Plan qp;
    if (!ren_bwd_q8_plan(B, H * W, C, groups, &qp)) return LPDT_ERR_UNSUPPORTED;
    cudaStream_t st = as_stream(stream);
    double *acc = (double *)ws;
    const float Cst = ren_const(C / groups);
    launch_k(qp.bwd, dim3((unsigned)((int64_t)nodes * B)), qp.threads, qp.smem, st, H * W, C, groups, eps, Cst, dy, x, v, gamma,
             pstride, nodes, B, gmin, gmax, argmin, argmax, acc, q, scale, amax_out, (int *)ctl, dev_status, qp.hold_off);
    LPDT_LAUNCH_CHECK();
    if (deferred) return LPDT_OK;
    launch_k(ren_bwd_finalize, (nodes * 3 * C + 7) / 8, 256, 0, st, acc, nodes, B, C, dv, dgamma, dbeta, gstride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_range_evonorm_bwd_params(int32_t nodes, int32_t B, int32_t C, const void *ws,
                                                     size_t ws_bytes, float *dv, float *dgamma, float *dbeta,
                                                     int64_t gstride, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && C > 0);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dv && dgamma && dbeta && (gstride >= C || nodes == 1));
    if (!ws || ws_bytes < lpdt_range_evonorm_bwd_workspace_size(nodes, B, C) || !aligned(ws, 8))
        return LPDT_ERR_WORKSPACE;
    launch_k(ren_bwd_finalize, (nodes * 3 * C + 7) / 8, 256, 0, as_stream(stream), (const double *)ws, nodes, B, C, dv,
             dgamma, dbeta, gstride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_range_evonorm_bwd_params_batch(int32_t nodes, int32_t B, int32_t n_layers, const int32_t *C,
                                                           const void *const *ws, const int64_t *grad_offsets,
                                                           float *grads, int64_t grad_node_stride, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && n_layers >= 0);
    if (nodes == 0 || B == 0 || n_layers == 0) return LPDT_OK;
    LPDT_CHECK_ARG(C && ws && grad_offsets && grads);
    if (n_layers > kMaxRenBatch) return LPDT_ERR_UNSUPPORTED;
    RenBatch rb;
    rb.count = n_layers;
    int64_t warps = 0;
    for (int l = 0; l < n_layers; ++l) {
        LPDT_CHECK_ARG(C[l] > 0 && ws[l] && aligned(ws[l], 8) && grad_offsets[l] >= 0);
        LPDT_CHECK_ARG(grad_offsets[l] + 3 * (int64_t)C[l] <= grad_node_stride || nodes == 1);
        rb.acc[l] = (const double *)ws[l]; rb.C[l] = C[l]; rb.off[l] = grad_offsets[l];
        rb.start[l] = (int)warps;
        warps += (int64_t)nodes * 3 * C[l];
        if (warps > 0x3fffffff) return LPDT_ERR_UNSUPPORTED;
    }
    rb.start[n_layers] = (int)warps;
    launch_k(ren_bwd_finalize_batch, (unsigned)ceil_div(warps, 8), 256, 0, as_stream(stream), rb, nodes, B, grads,
             grad_node_stride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
