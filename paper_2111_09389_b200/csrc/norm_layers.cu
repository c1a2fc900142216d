// The comparison layers of Section 3: EvoNorm-S0 (Eq. "en": the layer the paper trains with at
// full precision) and range batch-norm (Eq. "rbn"), forward and backward.  Same data layout
// and thread mapping as the Range-EvoNorm kernels: fp32 NHWC, a thread owns a fixed vector of
// V channels and walks pixels, so every global access is a coalesced 16-byte load or store.
// Sums that feed statistics or parameter gradients are accumulated in double.  All four
// passes are HBM-bound streaming kernels.
#include <math.h>
#include <cooperative_groups.h>
#include "common.cuh"

namespace lpdt {

template <int V> struct NVec;
template <> struct NVec<4> {
    static __device__ __forceinline__ void ld(const float *p, float (&o)[4]) {
        float4 t = *reinterpret_cast<const float4 *>(p); o[0] = t.x; o[1] = t.y; o[2] = t.z; o[3] = t.w;
    }
    static __device__ __forceinline__ void st(float *p, const float (&o)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(o[0], o[1], o[2], o[3]);
    }
};
template <> struct NVec<1> {
    static __device__ __forceinline__ void ld(const float *p, float (&o)[1]) { o[0] = *p; }
    static __device__ __forceinline__ void st(float *p, const float (&o)[1]) { *p = o[0]; }
};

// Logistic function from the hardware's base-2 exponential and reciprocal approximations: a few ulp of relative
// error (the exponential's grows with |u|: about 1e-6 at |u| = 10), well inside the 1e-5 these layers are held
// to.  The correctly rounded expf and IEEE division this replaces cost about 30 instructions per element and made
// both EvoNorm-S0 kernels instruction-bound (38 / 40 % of the HBM copy peak).
__device__ __forceinline__ float sigmoidf_acc(float u) { return __fdividef(1.f, 1.f + __expf(-u)); }

// ------------------------------------------------------------------ EvoNorm-S0
// One CTA per (node, sample).  Pass 1: per-thread sums of x and x*x in double, folded per group
// through shared memory (fixed order); pass 2 re-reads the sample (an L2 hit) and writes y.
template <int V>
__global__ void __launch_bounds__(256)
evonorm_fwd_kernel(int HW, int C, int groups, float eps, const float *__restrict__ x, const float *__restrict__ v,
                   const float *__restrict__ gamma, const float *__restrict__ beta, int64_t pstride, int B,
                   float *__restrict__ y, float *__restrict__ gmean, float *__restrict__ gvar) {
    pdl_enter();
    extern __shared__ double sm_d[];
    const int T = blockDim.x, t = threadIdx.x;
    double *s_sum = sm_d, *s_sq = sm_d + T, *g_mu = sm_d + 2 * T, *g_inv = g_mu + groups;
    const int CV = C / V, cpg = C / groups;
    const int col = t % CV, row0 = t / CV, rstep = T / CV;
    const int c0 = col * V, grp = c0 / cpg;
    const int64_t sample = blockIdx.x;
    const int node = (int)(sample / B);
    const float *xs = x + sample * (int64_t)HW * C;
    float *ys = y + sample * (int64_t)HW * C;
    double sum = 0.0, sq = 0.0;
#pragma unroll 4
    for (int p = row0; p < HW; p += rstep) {
        float xv[V];
        NVec<V>::ld(xs + (int64_t)p * C + c0, xv);
#pragma unroll
        for (int k = 0; k < V; ++k) { sum += (double)xv[k]; sq += (double)xv[k] * (double)xv[k]; }
    }
    s_sum[t] = sum; s_sq[t] = sq;
    __syncthreads();
    const int cols = cpg / V, members = cols * rstep;
    for (int g = t; g < groups; g += T) {
        double a = 0.0, b = 0.0;
        for (int m = 0; m < members; ++m) {
            const int th = (m / cols) * CV + g * cols + (m % cols);
            a += s_sum[th]; b += s_sq[th];
        }
        const double cnt = (double)HW * cpg, mu = a / cnt;
        double var = b / cnt - mu * mu;
        if (var < 0.0) var = 0.0;
        g_mu[g] = mu; g_inv[g] = 1.0 / sqrt(var + (double)eps);
        gmean[sample * groups + g] = (float)mu; gvar[sample * groups + g] = (float)var;
    }
    __syncthreads();
    const float invD = (float)g_inv[grp];
    float vc[V], gc[V], bc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        vc[k] = v[(int64_t)node * pstride + c0 + k];
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
        bc[k] = beta[(int64_t)node * pstride + c0 + k];
    }
#pragma unroll 4
    for (int p = row0; p < HW; p += rstep) {
        float xv[V], yv[V];
        NVec<V>::ld(xs + (int64_t)p * C + c0, xv);
#pragma unroll
        for (int k = 0; k < V; ++k) yv[k] = gc[k] * (xv[k] * sigmoidf_acc(vc[k] * xv[k])) * invD + bc[k];
        NVec<V>::st(ys + (int64_t)p * C + c0, yv);
    }
}

// Backward: pass 1 accumulates the group sum S = sum t*m and the per-channel parameter-gradient sums
// (double), pass 2 re-reads dy and x and writes dx.  Per-sample channel sums go to `acc`
// [nodes*B][3][C] and are added over the batch by norm_param_finalize.
template <int V>
__global__ void __launch_bounds__(256)
evonorm_bwd_kernel(int HW, int C, int groups, float eps, const float *__restrict__ dy, const float *__restrict__ x,
                   const float *__restrict__ v, const float *__restrict__ gamma, int64_t pstride, int B,
                   const float *__restrict__ gmean, const float *__restrict__ gvar, float *__restrict__ dx,
                   double *__restrict__ acc) {
    pdl_enter();
    extern __shared__ double sm_d[];
    const int T = blockDim.x, t = threadIdx.x;
    double *s_S = sm_d, *g_S = sm_d + T, *s_ch = g_S + groups;      // s_ch: [3][V][T]
    const int CV = C / V, cpg = C / groups;
    const int col = t % CV, row0 = t / CV, rstep = T / CV;
    const int c0 = col * V, grp = c0 / cpg;
    const int64_t sample = blockIdx.x;
    const int node = (int)(sample / B);
    const float *xs = x + sample * (int64_t)HW * C;
    const float *dys = dy + sample * (int64_t)HW * C;
    float *dxs = dx + sample * (int64_t)HW * C;
    const double mu = (double)gmean[sample * groups + grp];
    const double Dd = sqrt((double)gvar[sample * groups + grp] + (double)eps);
    const float invD = (float)(1.0 / Dd);
    float vc[V], gc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        vc[k] = v[(int64_t)node * pstride + c0 + k];
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
    }
    double S = 0.0, sv[V], sg[V], sb[V];
#pragma unroll
    for (int k = 0; k < V; ++k) { sv[k] = 0.0; sg[k] = 0.0; sb[k] = 0.0; }
#pragma unroll 4
    for (int p = row0; p < HW; p += rstep) {
        float xv[V], dv_[V];
        NVec<V>::ld(xs + (int64_t)p * C + c0, xv);
        NVec<V>::ld(dys + (int64_t)p * C + c0, dv_);
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const float sig = sigmoidf_acc(vc[k] * xv[k]);
            const float m = xv[k] * sig, tt = dv_[k] * gc[k];
            S += (double)(tt * m);
            sb[k] += (double)dv_[k];
            sg[k] += (double)(dv_[k] * m * invD);
            sv[k] += (double)(tt * xv[k] * xv[k] * sig * (1.f - sig) * invD);
        }
    }
    s_S[t] = S;
#pragma unroll
    for (int k = 0; k < V; ++k) {
        s_ch[(0 * V + k) * T + t] = sv[k]; s_ch[(1 * V + k) * T + t] = sg[k]; s_ch[(2 * V + k) * T + t] = sb[k];
    }
    __syncthreads();
    const int cols = cpg / V, members = cols * rstep;
    for (int g = t; g < groups; g += T) {
        double a = 0.0;
        for (int m = 0; m < members; ++m) a += s_S[(m / cols) * CV + g * cols + (m % cols)];
        g_S[g] = a;
    }
    for (int i = t; i < 3 * C; i += T) {          // channel sums of this sample: rows of the column in order
        const int which = i / C, c = i % C, cl = c / V, k = c % V;
        double a = 0.0;
        for (int r = 0; r < rstep; ++r) a += s_ch[(which * V + k) * T + r * CV + cl];
        acc[sample * 3 * C + i] = a;
    }
    __syncthreads();
    const double cnt = (double)HW * cpg;
    const float coef = (float)(g_S[grp] / (cnt * Dd * Dd * Dd));
    const float muf = (float)mu;
#pragma unroll 4
    for (int p = row0; p < HW; p += rstep) {
        float xv[V], dv_[V], o[V];
        NVec<V>::ld(xs + (int64_t)p * C + c0, xv);
        NVec<V>::ld(dys + (int64_t)p * C + c0, dv_);
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const float u = vc[k] * xv[k], sig = sigmoidf_acc(u);
            const float tt = dv_[k] * gc[k];
            o[k] = tt * (sig + u * sig * (1.f - sig)) * invD - coef * (xv[k] - muf);
        }
        NVec<V>::st(dxs + (int64_t)p * C + c0, o);
    }
}

// ---- EvoNorm-S0 with the sample held in shared memory ---------------------------------------------------
// The two-pass kernels above read a sample twice; with one CTA per 256 KB sample the samples in flight exceed
// the L2 and the second pass comes from DRAM again (measured: 2.6 % L2 hit rate, 20 B per element instead of
// 12 in the backward kernel).  Here a cluster of R CTAs owns a sample: every CTA copies its share of the pixels
// into shared memory with asynchronous 16-byte copies (all in flight at once), the group sums of the CTAs meet
// through distributed shared memory (added in rank order by every CTA: the same result everywhere), and the
// second pass reads shared memory.  Vector columns of 4 channels only.
__device__ __forceinline__ void nl_cp_async16(void *smem_dst, const void *gsrc) {
    const uint32_t d = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void nl_cp_async_commit_wait() {
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

__global__ void __launch_bounds__(256, 2)
evonorm_fwd_cl_kernel(int HW, int C, int groups, float eps, const float *__restrict__ x, const float *__restrict__ v,
                      const float *__restrict__ gamma, const float *__restrict__ beta, int64_t pstride, int B,
                      float *__restrict__ y, float *__restrict__ gmean, float *__restrict__ gvar, int R, int ppc,
                      unsigned hold_off) {
    namespace cg = cooperative_groups;
    constexpr int V = 4;
    pdl_enter();
    extern __shared__ double sm_d[];
    const int T = blockDim.x, t = threadIdx.x;
    double *s_sum = sm_d, *s_sq = sm_d + T, *part = sm_d + 2 * T;       // part: this CTA's [sum | sum of squares][groups]
    double *g_mu = part + 2 * groups, *g_inv = g_mu + groups;
    float *hold = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(sm_d) + hold_off);
    const int CV = C / V, cpg = C / groups;
    const int col = t % CV, row0 = t / CV, rstep = T / CV;
    const int c0 = col * V, grp = c0 / cpg;
    const int rank = (int)(blockIdx.x % R);
    const int64_t sample = blockIdx.x / R;
    const int node = (int)(sample / B);
    const int p_lo = rank * ppc, p_end = (p_lo + ppc < HW) ? p_lo + ppc : HW;
    const float *xs = x + sample * (int64_t)HW * C;
    float *ys = y + sample * (int64_t)HW * C;
    for (int p = p_lo + row0; p < p_end; p += rstep) nl_cp_async16(hold + (size_t)(p - p_lo) * C + c0, xs + (int64_t)p * C + c0);
    float vc[V], gc[V], bc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        vc[k] = v[(int64_t)node * pstride + c0 + k];
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
        bc[k] = beta[(int64_t)node * pstride + c0 + k];
    }
    nl_cp_async_commit_wait();           // every thread reads back only what its own copies brought
    double sum = 0.0, sq = 0.0;
    for (int p = p_lo + row0; p < p_end; p += rstep) {
        const float4 a = *reinterpret_cast<const float4 *>(hold + (size_t)(p - p_lo) * C + c0);
        const double d0 = a.x, d1 = a.y, d2 = a.z, d3 = a.w;
        sum += d0; sq += d0 * d0; sum += d1; sq += d1 * d1; sum += d2; sq += d2 * d2; sum += d3; sq += d3 * d3;
    }
    s_sum[t] = sum; s_sq[t] = sq;
    __syncthreads();
    const int cols = cpg / V, members = cols * rstep;
    for (int g = t; g < groups; g += T) {
        double a = 0.0, b = 0.0;
        for (int m = 0; m < members; ++m) {
            const int th = (m / cols) * CV + g * cols + (m % cols);
            a += s_sum[th]; b += s_sq[th];
        }
        part[g] = a; part[groups + g] = b;
    }
    cg::cluster_group cluster = cg::this_cluster();
    if (R > 1) cluster.sync(); else __syncthreads();
    for (int g = t; g < groups; g += T) {
        double a = 0.0, b = 0.0;
        for (int r = 0; r < R; ++r) {
            const double *pr = R > 1 ? cluster.map_shared_rank(part, r) : part;
            a += pr[g]; b += pr[groups + g];
        }
        const double cnt = (double)HW * cpg, mu = a / cnt;
        double var = b / cnt - mu * mu;
        if (var < 0.0) var = 0.0;
        g_mu[g] = mu; g_inv[g] = 1.0 / sqrt(var + (double)eps);
        if (rank == 0) { gmean[sample * groups + g] = (float)mu; gvar[sample * groups + g] = (float)var; }
    }
    __syncthreads();
    if (R > 1) cluster.barrier_arrive();          // done reading the others' shared memory; waited for before exit
    const float invD = (float)g_inv[grp];
    for (int p = p_lo + row0; p < p_end; p += rstep) {
        const float4 a = *reinterpret_cast<const float4 *>(hold + (size_t)(p - p_lo) * C + c0);
        const float xv[V] = {a.x, a.y, a.z, a.w};
        float yv[V];
#pragma unroll
        for (int k = 0; k < V; ++k) yv[k] = gc[k] * (xv[k] * sigmoidf_acc(vc[k] * xv[k])) * invD + bc[k];
        NVec<V>::st(ys + (int64_t)p * C + c0, yv);
    }
    if (R > 1) cluster.barrier_wait();
}

__global__ void __launch_bounds__(256, 2)
evonorm_bwd_cl_kernel(int HW, int C, int groups, float eps, const float *__restrict__ dy, const float *__restrict__ x,
                      const float *__restrict__ v, const float *__restrict__ gamma, int64_t pstride, int B,
                      const float *__restrict__ gmean, const float *__restrict__ gvar, float *__restrict__ dx,
                      double *__restrict__ acc, int R, int ppc, unsigned hold_off) {
    namespace cg = cooperative_groups;
    constexpr int V = 4;
    pdl_enter();
    extern __shared__ double sm_d[];
    const int T = blockDim.x, t = threadIdx.x;
    double *s_S = sm_d, *part_S = sm_d + T, *g_S = part_S + groups, *s_ch = g_S + groups;      // s_ch: [3][V][T]
    double *part_ch = s_ch + 3 * V * T;                                                       // [3][C] of this CTA
    float *hx = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(sm_d) + hold_off);
    float *hdy = hx + (size_t)ppc * C;
    const int CV = C / V, cpg = C / groups;
    const int col = t % CV, row0 = t / CV, rstep = T / CV;
    const int c0 = col * V, grp = c0 / cpg;
    const int rank = (int)(blockIdx.x % R);
    const int64_t sample = blockIdx.x / R;
    const int node = (int)(sample / B);
    const int p_lo = rank * ppc, p_end = (p_lo + ppc < HW) ? p_lo + ppc : HW;
    const float *xs = x + sample * (int64_t)HW * C;
    const float *dys = dy + sample * (int64_t)HW * C;
    float *dxs = dx + sample * (int64_t)HW * C;
    for (int p = p_lo + row0; p < p_end; p += rstep) {
        nl_cp_async16(hx + (size_t)(p - p_lo) * C + c0, xs + (int64_t)p * C + c0);
        nl_cp_async16(hdy + (size_t)(p - p_lo) * C + c0, dys + (int64_t)p * C + c0);
    }
    const double mu = (double)gmean[sample * groups + grp];
    const double Dd = sqrt((double)gvar[sample * groups + grp] + (double)eps);
    const float invD = (float)(1.0 / Dd);
    float vc[V], gc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        vc[k] = v[(int64_t)node * pstride + c0 + k];
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
    }
    nl_cp_async_commit_wait();
    // A thread owns at most a few dozen rows of its CTA's share (the share is bounded by the shared memory), so
    // its own partial sums stay in fp32; every combination across threads, CTAs and samples is done in double.
    float S = 0.f, sv[V], sg[V], sb[V];
#pragma unroll
    for (int k = 0; k < V; ++k) { sv[k] = 0.f; sg[k] = 0.f; sb[k] = 0.f; }
    for (int p = p_lo + row0; p < p_end; p += rstep) {
        const float4 a = *reinterpret_cast<const float4 *>(hx + (size_t)(p - p_lo) * C + c0);
        const float4 b = *reinterpret_cast<const float4 *>(hdy + (size_t)(p - p_lo) * C + c0);
        const float xv[V] = {a.x, a.y, a.z, a.w}, dv_[V] = {b.x, b.y, b.z, b.w};
        float loc[V];
#pragma unroll
        for (int k = 0; k < V; ++k) {
            const float u = vc[k] * xv[k], sig = sigmoidf_acc(u);
            const float m = xv[k] * sig, tt = dv_[k] * gc[k];
            S += tt * m;
            sb[k] += dv_[k];
            sg[k] += dv_[k] * m * invD;
            sv[k] += tt * xv[k] * xv[k] * sig * (1.f - sig) * invD;
            loc[k] = tt * (sig + u * sig * (1.f - sig)) * invD;      // the part of dx that needs no group sum
        }
        // dy is not needed again: its place takes the local term, so that the second pass has no logistic to redo
        *reinterpret_cast<float4 *>(hdy + (size_t)(p - p_lo) * C + c0) = make_float4(loc[0], loc[1], loc[2], loc[3]);
    }
    s_S[t] = (double)S;
#pragma unroll
    for (int k = 0; k < V; ++k) {
        s_ch[(0 * V + k) * T + t] = (double)sv[k]; s_ch[(1 * V + k) * T + t] = (double)sg[k];
        s_ch[(2 * V + k) * T + t] = (double)sb[k];
    }
    __syncthreads();
    const int cols = cpg / V, members = cols * rstep;
    for (int g = t; g < groups; g += T) {
        double a = 0.0;
        for (int m = 0; m < members; ++m) a += s_S[(m / cols) * CV + g * cols + (m % cols)];
        part_S[g] = a;
    }
    for (int i = t; i < 3 * C; i += T) {          // channel sums of this CTA's pixels: rows of the column in order
        const int which = i / C, c = i % C, cl = c / V, k = c % V;
        double a = 0.0;
        for (int r = 0; r < rstep; ++r) a += s_ch[(which * V + k) * T + r * CV + cl];
        part_ch[i] = a;
    }
    cg::cluster_group cluster = cg::this_cluster();
    if (R > 1) cluster.sync(); else __syncthreads();
    for (int g = t; g < groups; g += T) {
        double a = 0.0;
        for (int r = 0; r < R; ++r) a += (R > 1 ? cluster.map_shared_rank(part_S, r) : part_S)[g];
        g_S[g] = a;
    }
    if (rank == 0) {
        for (int i = t; i < 3 * C; i += T) {
            double a = 0.0;
            for (int r = 0; r < R; ++r) a += (R > 1 ? cluster.map_shared_rank(part_ch, r) : part_ch)[i];
            acc[sample * 3 * C + i] = a;
        }
    }
    __syncthreads();
    if (R > 1) cluster.barrier_arrive();
    const double cnt = (double)HW * cpg;
    const float coef = (float)(g_S[grp] / (cnt * Dd * Dd * Dd));
    const float muf = (float)mu;
    for (int p = p_lo + row0; p < p_end; p += rstep) {
        const float4 a = *reinterpret_cast<const float4 *>(hx + (size_t)(p - p_lo) * C + c0);
        const float4 b = *reinterpret_cast<const float4 *>(hdy + (size_t)(p - p_lo) * C + c0);
        const float xv[V] = {a.x, a.y, a.z, a.w}, loc[V] = {b.x, b.y, b.z, b.w};
        float o[V];
#pragma unroll
        for (int k = 0; k < V; ++k) o[k] = loc[k] - coef * (xv[k] - muf);
        NVec<V>::st(dxs + (int64_t)p * C + c0, o);
    }
    if (R > 1) cluster.barrier_wait();
}

// Cluster size and pixels per CTA for the kernels above: the smallest power of two (up to 8, and so that every
// CTA keeps a thread row) whose share of `bytes_per_pixel` fits `target` bytes; 0 when even 8 CTAs would need
// more than `limit`.
static int evonorm_cluster(int HW, int rstep, size_t bytes_per_pixel, size_t target, size_t limit, int *ppc_out) {
    const int rows = (int)ceil_div(HW, rstep);
    int R = 1;
    while (true) {
        const int ppc = (int)ceil_div(ceil_div(HW, R), rstep) * rstep;
        const size_t need = (size_t)ppc * bytes_per_pixel;
        if (need <= target || R == 8 || R * 2 > rows) {
            if (need > limit) return 0;
            *ppc_out = ppc;
            return R;
        }
        R *= 2;
    }
}

// out[node][which][c] = sum over the node's samples of acc[node*B + b][which][c], rounded once.
// One warp per output; lanes stride the samples and combine in a fixed shuffle tree.
__global__ void norm_param_finalize(const double *__restrict__ acc, int nodes, int B, int C, int nwhich,
                                    float *__restrict__ o0, float *__restrict__ o1, float *__restrict__ o2,
                                    int64_t gstride) {
    pdl_enter();
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (i >= nodes * nwhich * C) return;
    const int node = i / (nwhich * C), j = i % (nwhich * C), which = j / C, c = j % C;
    const double *a = acc + (int64_t)node * B * nwhich * C + j;
    double s = 0.0;
    for (int b = lane; b < B; b += 32) s += a[(int64_t)b * nwhich * C];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if (lane == 0) {
        float *dst = which == 0 ? o0 : which == 1 ? o1 : o2;
        dst[(int64_t)node * gstride + c] = (float)s;
    }
}

// ------------------------------------------------------------------ range batch-norm
// Statistics run over the node's whole batch per channel, so they are gathered across CTAs:
// the sum by double atomics, the extrema by 64-bit atomicMax on (order-preserving value bits,
// inverted position), which also yields the lowest position among equal values.
struct RbnStat { double sum; unsigned long long maxkey, minkey; double sdy, sdx; };   // zeroed per call

__device__ __forceinline__ uint32_t ordered_bits(float f) {
    const uint32_t b = __float_as_uint(f);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float from_ordered(uint32_t o) {
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}

constexpr int kRbnIters = 32;       // pixel rows per thread in one CTA

template <int V>
__global__ void __launch_bounds__(256)
rbn_stats_kernel(int64_t P, int C, const float *__restrict__ x, RbnStat *__restrict__ stat) {
    pdl_enter();
    extern __shared__ double sm_d[];
    const int T = blockDim.x, t = threadIdx.x;
    double *s_sum = sm_d;                                                         // [V][T]
    unsigned long long *s_mx = reinterpret_cast<unsigned long long *>(sm_d + V * T), *s_mn = s_mx + V * T;
    const int CV = C / V, col = t % CV, row0 = t / CV, rstep = T / CV, c0 = col * V;
    const int node = blockIdx.y;
    const float *xs = x + (int64_t)node * P * C;
    const int64_t p0 = (int64_t)blockIdx.x * rstep * kRbnIters;
    double sum[V]; unsigned long long mx[V], mn[V];
#pragma unroll
    for (int k = 0; k < V; ++k) { sum[k] = 0.0; mx[k] = 0ull; mn[k] = 0ull; }
    // four independent 16-byte loads are issued before any of them is used
    for (int it0 = 0; it0 < kRbnIters; it0 += 4) {
        float xb[4][V];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p < P) NVec<V>::ld(xs + p * C + c0, xb[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p >= P) continue;
            const unsigned long long inv_pos = 0xFFFFFFFFull - (unsigned long long)p;
#pragma unroll
            for (int k = 0; k < V; ++k) {
                sum[k] += (double)xb[u][k];
                // + 0.f turns -0 into +0, so that equal zeros tie (and the lowest position wins) as in a float compare
                const unsigned long long a = ((unsigned long long)ordered_bits(xb[u][k] + 0.f) << 32) | inv_pos;
                const unsigned long long b = ((unsigned long long)ordered_bits(-xb[u][k] + 0.f) << 32) | inv_pos;
                mx[k] = a > mx[k] ? a : mx[k];
                mn[k] = b > mn[k] ? b : mn[k];
            }
        }
    }
#pragma unroll
    for (int k = 0; k < V; ++k) { s_sum[k * T + t] = sum[k]; s_mx[k * T + t] = mx[k]; s_mn[k * T + t] = mn[k]; }
    __syncthreads();
    for (int c = t; c < C; c += T) {
        const int cl = c / V, k = c % V;
        double a = 0.0; unsigned long long m1 = 0ull, m2 = 0ull;
        for (int r = 0; r < rstep; ++r) {
            const int th = r * CV + cl;
            a += s_sum[k * T + th];
            m1 = s_mx[k * T + th] > m1 ? s_mx[k * T + th] : m1;
            m2 = s_mn[k * T + th] > m2 ? s_mn[k * T + th] : m2;
        }
        RbnStat *s = stat + (int64_t)node * C + c;
        atomicAdd(&s->sum, a);
        if (m1) atomicMax(&s->maxkey, m1);
        if (m2) atomicMax(&s->minkey, m2);
    }
}

template <int V>
__global__ void __launch_bounds__(256)
rbn_apply_kernel(int64_t P, int C, float eps, float Cb, const float *__restrict__ x, const float *__restrict__ gamma,
                 const float *__restrict__ beta, int64_t pstride, const RbnStat *__restrict__ stat,
                 float *__restrict__ y, float *__restrict__ cmean, float *__restrict__ cmin, float *__restrict__ cmax,
                 int32_t *__restrict__ argmin, int32_t *__restrict__ argmax) {
    pdl_enter();
    const int T = blockDim.x, t = threadIdx.x;
    const int CV = C / V, col = t % CV, row0 = t / CV, rstep = T / CV, c0 = col * V;
    const int node = blockIdx.y;
    const float *xs = x + (int64_t)node * P * C;
    float *ys = y + (int64_t)node * P * C;
    float mu[V], invD[V], gc[V], bc[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        const RbnStat s = stat[(int64_t)node * C + c0 + k];
        const float mx = from_ordered((uint32_t)(s.maxkey >> 32)), mn = -from_ordered((uint32_t)(s.minkey >> 32));
        const double mean = s.sum / (double)P;
        mu[k] = (float)mean;
        invD[k] = (float)(1.0 / ((double)Cb * ((double)mx - (double)mn) + (double)eps));
        gc[k] = gamma[(int64_t)node * pstride + c0 + k];
        bc[k] = beta[(int64_t)node * pstride + c0 + k];
        if (blockIdx.x == 0 && row0 == 0) {
            const int64_t nc = (int64_t)node * C + c0 + k;
            cmean[nc] = mu[k]; cmin[nc] = mn; cmax[nc] = mx;
            argmax[nc] = (int32_t)(0xFFFFFFFFull - (s.maxkey & 0xFFFFFFFFull));
            argmin[nc] = (int32_t)(0xFFFFFFFFull - (s.minkey & 0xFFFFFFFFull));
        }
    }
    const int64_t p0 = (int64_t)blockIdx.x * rstep * kRbnIters;
    for (int it0 = 0; it0 < kRbnIters; it0 += 4) {
        float xb[4][V];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p < P) NVec<V>::ld(xs + p * C + c0, xb[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p >= P) continue;
            float yv[V];
#pragma unroll
            for (int k = 0; k < V; ++k) yv[k] = gc[k] * (xb[u][k] - mu[k]) * invD[k] + bc[k];
            NVec<V>::st(ys + p * C + c0, yv);
        }
    }
}

template <int V>
__global__ void __launch_bounds__(256)
rbn_bwd_sums_kernel(int64_t P, int C, const float *__restrict__ dy, const float *__restrict__ x,
                    const float *__restrict__ cmean, RbnStat *__restrict__ stat) {
    pdl_enter();
    extern __shared__ double sm_d[];
    const int T = blockDim.x, t = threadIdx.x;
    double *s_a = sm_d, *s_b = sm_d + V * T;
    const int CV = C / V, col = t % CV, row0 = t / CV, rstep = T / CV, c0 = col * V;
    const int node = blockIdx.y;
    const float *xs = x + (int64_t)node * P * C, *dys = dy + (int64_t)node * P * C;
    float mu[V];
    double a[V], b[V];
#pragma unroll
    for (int k = 0; k < V; ++k) { mu[k] = cmean[(int64_t)node * C + c0 + k]; a[k] = 0.0; b[k] = 0.0; }
    const int64_t p0 = (int64_t)blockIdx.x * rstep * kRbnIters;
    for (int it0 = 0; it0 < kRbnIters; it0 += 4) {
        float xb[4][V], db[4][V];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p < P) { NVec<V>::ld(xs + p * C + c0, xb[u]); NVec<V>::ld(dys + p * C + c0, db[u]); }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p >= P) continue;
#pragma unroll
            for (int k = 0; k < V; ++k) { a[k] += (double)db[u][k]; b[k] += (double)db[u][k] * (double)(xb[u][k] - mu[k]); }
        }
    }
#pragma unroll
    for (int k = 0; k < V; ++k) { s_a[k * T + t] = a[k]; s_b[k * T + t] = b[k]; }
    __syncthreads();
    for (int c = t; c < C; c += T) {
        const int cl = c / V, k = c % V;
        double u = 0.0, w = 0.0;
        for (int r = 0; r < rstep; ++r) { u += s_a[k * T + r * CV + cl]; w += s_b[k * T + r * CV + cl]; }
        RbnStat *s = stat + (int64_t)node * C + c;
        atomicAdd(&s->sdy, u);
        atomicAdd(&s->sdx, w);
    }
}

template <int V>
__global__ void __launch_bounds__(256)
rbn_bwd_apply_kernel(int64_t P, int C, float eps, float Cb, const float *__restrict__ dy, const float *__restrict__ gamma,
                     int64_t pstride, const float *__restrict__ cmin, const float *__restrict__ cmax,
                     const int32_t *__restrict__ argmin, const int32_t *__restrict__ argmax,
                     const RbnStat *__restrict__ stat, float *__restrict__ dx, float *__restrict__ dgamma,
                     float *__restrict__ dbeta, int64_t gstride) {
    pdl_enter();
    const int T = blockDim.x, t = threadIdx.x;
    const int CV = C / V, col = t % CV, row0 = t / CV, rstep = T / CV, c0 = col * V;
    const int node = blockIdx.y;
    const float *dys = dy + (int64_t)node * P * C;
    float *dxs = dx + (int64_t)node * P * C;
    float gD[V], shift[V], coef[V];
    int amx[V], amn[V];
#pragma unroll
    for (int k = 0; k < V; ++k) {
        const int64_t nc = (int64_t)node * C + c0 + k;
        const RbnStat s = stat[nc];
        const double D = (double)Cb * ((double)cmax[nc] - (double)cmin[nc]) + (double)eps;
        const double g = (double)gamma[(int64_t)node * pstride + c0 + k];
        gD[k] = (float)(g / D);
        shift[k] = (float)(g * s.sdy / ((double)P * D));
        amx[k] = argmax[nc]; amn[k] = argmin[nc];
        coef[k] = amx[k] != amn[k] ? (float)((double)Cb * g * s.sdx / (D * D)) : 0.f;
        if (blockIdx.x == 0 && row0 == 0) {
            dgamma[(int64_t)node * gstride + c0 + k] = (float)(s.sdx / D);
            dbeta[(int64_t)node * gstride + c0 + k] = (float)s.sdy;
        }
    }
    const int64_t p0 = (int64_t)blockIdx.x * rstep * kRbnIters;
    for (int it0 = 0; it0 < kRbnIters; it0 += 4) {
        float db[4][V];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p < P) NVec<V>::ld(dys + p * C + c0, db[u]);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t p = p0 + row0 + (int64_t)(it0 + u) * rstep;
            if (p >= P) continue;
            float o[V];
#pragma unroll
            for (int k = 0; k < V; ++k) {
                o[k] = db[u][k] * gD[k] - shift[k];
                if (p == (int64_t)amx[k]) o[k] -= coef[k];
                if (p == (int64_t)amn[k]) o[k] += coef[k];
            }
            NVec<V>::st(dxs + p * C + c0, o);
        }
    }
}

struct NormPlan { int V, threads; };

// V = 4 when the channel groups allow 16-byte vectors; threads = whole thread rows of C/V columns, at most 256.
static bool norm_plan(int C, int cpg, bool aligned16, NormPlan *pl) {
    const int V = (aligned16 && C % 4 == 0 && cpg % 4 == 0) ? 4 : 1;
    const int CV = C / V;
    if (CV > 256) return false;
    pl->V = V;
    pl->threads = CV * (256 / CV);
    return true;
}

}  // namespace lpdt

using namespace lpdt;

extern "C" lpdt_status lpdt_evonorm_s0_fwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups,
                                           float eps, const float *x, const float *v, const float *gamma,
                                           const float *beta, int64_t pstride, float *y, float *gmean, float *gvar,
                                           void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && groups > 0 && C % groups == 0);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && v && gamma && beta && y && gmean && gvar && (pstride >= C || nodes == 1));
    if ((int64_t)H * W * C > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    NormPlan pl;
    if (!norm_plan(C, C / groups, aligned(x, 16) && aligned(y, 16), &pl)) return LPDT_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(2 * pl.threads + 2 * groups) * sizeof(double);
    if (smem > 48 * 1024) return LPDT_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)((int64_t)nodes * B));
    static int two_pass = -1;       // LPDT_EVONORM_TWO_PASS=1: the kernels that read a sample twice (A/B timing, parity tests)
    if (two_pass < 0) { const char *e = getenv("LPDT_EVONORM_TWO_PASS"); two_pass = (e && e[0] == '1') ? 1 : 0; }
    if (pl.V == 4 && !two_pass) {
        const int rstep = pl.threads / (C / 4);
        int ppc = 0;
        // shares of up to 64 KB: measured best (clusters of 8 lose to cluster scheduling, 128 KB shares to occupancy)
        const int R = evonorm_cluster(H * W, rstep, (size_t)C * 4, 64 * 1024, 160 * 1024, &ppc);
        const size_t scratch = align_up((size_t)(2 * pl.threads + 4 * groups) * sizeof(double), 16);
        if (R > 0 && scratch <= 32 * 1024 && (int64_t)nodes * B * R <= 0x7fffffff) {
            static PerDeviceOnce attr;
            int dev;
            if (attr.pending(&dev)) {
                LPDT_CUDA(cudaFuncSetAttribute(evonorm_fwd_cl_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
                attr.mark(dev);
            }
            launch_k_cluster(evonorm_fwd_cl_kernel, dim3((unsigned)((int64_t)nodes * B * R)), pl.threads,
                             scratch + (size_t)ppc * C * 4, as_stream(stream), R, H * W, C, groups, eps, x, v, gamma, beta,
                             pstride, B, y, gmean, gvar, R, ppc, (unsigned)scratch);
            LPDT_LAUNCH_CHECK();
            return LPDT_OK;
        }
    }
    if (pl.V == 4) launch_k(evonorm_fwd_kernel<4>, grid, pl.threads, smem, as_stream(stream), H * W, C, groups, eps, x, v, gamma, beta, pstride, B, y, gmean, gvar);
    else launch_k(evonorm_fwd_kernel<1>, grid, pl.threads, smem, as_stream(stream), H * W, C, groups, eps, x, v, gamma, beta, pstride, B, y, gmean, gvar);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" size_t lpdt_evonorm_s0_bwd_workspace_size(int32_t nodes, int32_t B, int32_t C) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)(B > 0 ? B : 1) * 3 * (size_t)(C > 0 ? C : 1) * sizeof(double), 256);
}

extern "C" lpdt_status lpdt_evonorm_s0_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, int32_t groups,
                                           float eps, const float *dy, const float *x, const float *v,
                                           const float *gamma, int64_t pstride, const float *gmean, const float *gvar,
                                           float *dx, float *dv, float *dgamma, float *dbeta, int64_t gstride,
                                           void *ws, size_t ws_bytes, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 0 && H > 0 && W > 0 && C > 0 && groups > 0 && C % groups == 0);
    if (nodes == 0 || B == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dy && x && v && gamma && gmean && gvar && dx && dv && dgamma && dbeta);
    LPDT_CHECK_ARG((pstride >= C && gstride >= C) || nodes == 1);
    if ((int64_t)H * W * C > 0x7fffffff) return LPDT_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < lpdt_evonorm_s0_bwd_workspace_size(nodes, B, C) || !aligned(ws, 8)) return LPDT_ERR_WORKSPACE;
    NormPlan pl;
    if (!norm_plan(C, C / groups, aligned(x, 16) && aligned(dy, 16) && aligned(dx, 16), &pl)) return LPDT_ERR_UNSUPPORTED;
    const size_t smem = (size_t)(pl.threads + groups + 3 * pl.V * pl.threads) * sizeof(double);
    if (smem > 48 * 1024) return LPDT_ERR_UNSUPPORTED;
    cudaStream_t st = as_stream(stream);
    double *acc = (double *)ws;
    const dim3 grid((unsigned)((int64_t)nodes * B));
    static int two_pass = -1;
    if (two_pass < 0) { const char *e = getenv("LPDT_EVONORM_TWO_PASS"); two_pass = (e && e[0] == '1') ? 1 : 0; }
    bool done = false;
    if (pl.V == 4 && !two_pass) {
        const int rstep = pl.threads / (C / 4);
        int ppc = 0;
        const int R = evonorm_cluster(H * W, rstep, (size_t)C * 8, 64 * 1024, 160 * 1024, &ppc);
        const size_t scratch = align_up((size_t)(pl.threads + 2 * groups + 12 * pl.threads + 3 * C) * sizeof(double), 16);
        if (R > 0 && scratch <= 48 * 1024 && (int64_t)nodes * B * R <= 0x7fffffff) {
            static PerDeviceOnce attr;
            int dev;
            if (attr.pending(&dev)) {
                LPDT_CUDA(cudaFuncSetAttribute(evonorm_bwd_cl_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024));
                attr.mark(dev);
            }
            launch_k_cluster(evonorm_bwd_cl_kernel, dim3((unsigned)((int64_t)nodes * B * R)), pl.threads,
                             scratch + (size_t)ppc * C * 8, st, R, H * W, C, groups, eps, dy, x, v, gamma, pstride, B, gmean,
                             gvar, dx, acc, R, ppc, (unsigned)scratch);
            done = true;
        }
    }
    if (!done) {
        if (pl.V == 4) launch_k(evonorm_bwd_kernel<4>, grid, pl.threads, smem, st, H * W, C, groups, eps, dy, x, v, gamma, pstride, B, gmean, gvar, dx, acc);
        else launch_k(evonorm_bwd_kernel<1>, grid, pl.threads, smem, st, H * W, C, groups, eps, dy, x, v, gamma, pstride, B, gmean, gvar, dx, acc);
    }
    LPDT_LAUNCH_CHECK();
    launch_k(norm_param_finalize, (nodes * 3 * C + 7) / 8, 256, 0, st, acc, nodes, B, C, 3, dv, dgamma, dbeta, gstride);
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" size_t lpdt_range_bn_workspace_size(int32_t nodes, int32_t C) {
    return align_up((size_t)(nodes > 0 ? nodes : 1) * (size_t)(C > 0 ? C : 1) * sizeof(RbnStat), 256);
}

static float rbn_const(int B) { return (float)(1.0 / sqrt(2.0 * log((double)B))); }

extern "C" lpdt_status lpdt_range_bn_fwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, float eps,
                                         const float *x, const float *gamma, const float *beta, int64_t pstride,
                                         float *y, float *cmean, float *cmin, float *cmax, int32_t *argmin,
                                         int32_t *argmax, void *ws, size_t ws_bytes, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 2 && H > 0 && W > 0 && C > 0);
    if (nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(x && gamma && beta && y && cmean && cmin && cmax && argmin && argmax && (pstride >= C || nodes == 1));
    const int64_t P = (int64_t)B * H * W;
    if (P > 0x7fffffff || nodes > 65535) return LPDT_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < lpdt_range_bn_workspace_size(nodes, C) || !aligned(ws, 8)) return LPDT_ERR_WORKSPACE;
    NormPlan pl;
    if (!norm_plan(C, C, aligned(x, 16) && aligned(y, 16), &pl)) return LPDT_ERR_UNSUPPORTED;
    cudaStream_t st = as_stream(stream);
    RbnStat *stat = (RbnStat *)ws;
    LPDT_CUDA(cudaMemsetAsync(stat, 0, (size_t)nodes * C * sizeof(RbnStat), st));
    const int rstep = pl.threads / (C / pl.V);
    const dim3 grid((unsigned)ceil_div(P, (int64_t)rstep * kRbnIters), nodes);
    const size_t smem = (size_t)3 * pl.V * pl.threads * sizeof(double);
    if (pl.V == 4) {
        launch_k(rbn_stats_kernel<4>, grid, pl.threads, smem, st, P, C, x, stat);
        launch_k(rbn_apply_kernel<4>, grid, pl.threads, 0, st, P, C, eps, rbn_const(B), x, gamma, beta, pstride, stat, y, cmean, cmin, cmax, argmin, argmax);
    } else {
        launch_k(rbn_stats_kernel<1>, grid, pl.threads, smem, st, P, C, x, stat);
        launch_k(rbn_apply_kernel<1>, grid, pl.threads, 0, st, P, C, eps, rbn_const(B), x, gamma, beta, pstride, stat, y, cmean, cmin, cmax, argmin, argmax);
    }
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}

extern "C" lpdt_status lpdt_range_bn_bwd(int32_t nodes, int32_t B, int32_t H, int32_t W, int32_t C, float eps,
                                         const float *dy, const float *x, const float *gamma, int64_t pstride,
                                         const float *cmean, const float *cmin, const float *cmax,
                                         const int32_t *argmin, const int32_t *argmax, float *dx, float *dgamma,
                                         float *dbeta, int64_t gstride, void *ws, size_t ws_bytes, void *stream) {
    LPDT_CHECK_ARG(nodes >= 0 && B >= 2 && H > 0 && W > 0 && C > 0);
    if (nodes == 0) return LPDT_OK;
    LPDT_CHECK_ARG(dy && x && gamma && cmean && cmin && cmax && argmin && argmax && dx && dgamma && dbeta);
    LPDT_CHECK_ARG((pstride >= C && gstride >= C) || nodes == 1);
    const int64_t P = (int64_t)B * H * W;
    if (P > 0x7fffffff || nodes > 65535) return LPDT_ERR_UNSUPPORTED;
    if (!ws || ws_bytes < lpdt_range_bn_workspace_size(nodes, C) || !aligned(ws, 8)) return LPDT_ERR_WORKSPACE;
    NormPlan pl;
    if (!norm_plan(C, C, aligned(x, 16) && aligned(dy, 16) && aligned(dx, 16), &pl)) return LPDT_ERR_UNSUPPORTED;
    cudaStream_t st = as_stream(stream);
    RbnStat *stat = (RbnStat *)ws;
    LPDT_CUDA(cudaMemsetAsync(stat, 0, (size_t)nodes * C * sizeof(RbnStat), st));
    const int rstep = pl.threads / (C / pl.V);
    const dim3 grid((unsigned)ceil_div(P, (int64_t)rstep * kRbnIters), nodes);
    const size_t smem = (size_t)2 * pl.V * pl.threads * sizeof(double);
    if (pl.V == 4) {
        launch_k(rbn_bwd_sums_kernel<4>, grid, pl.threads, smem, st, P, C, dy, x, cmean, stat);
        launch_k(rbn_bwd_apply_kernel<4>, grid, pl.threads, 0, st, P, C, eps, rbn_const(B), dy, gamma, pstride, cmin, cmax, argmin, argmax, stat, dx, dgamma, dbeta, gstride);
    } else {
        launch_k(rbn_bwd_sums_kernel<1>, grid, pl.threads, smem, st, P, C, dy, x, cmean, stat);
        launch_k(rbn_bwd_apply_kernel<1>, grid, pl.threads, 0, st, P, C, eps, rbn_const(B), dy, gamma, pstride, cmin, cmax, argmin, argmax, stat, dx, dgamma, dbeta, gstride);
    }
    LPDT_LAUNCH_CHECK();
    return LPDT_OK;
}
