// Logit distance distribution kernels of libimm (sm_100a) and their C ABI (declared in imm.h).
//
//   imm_ldd_tv_kl          TV and KL distance between the softmax distributions of two logit rows
//   imm_ldd_topk_distance  L1 distance of a logit row to the nearest row whose top-K set is a given set
//   imm_ldd_tail_fraction  per-request share of steps whose distance exceeds a threshold, and the flag
//
// All three stream rows of float32 logits; the work is bound by HBM.  A row (a vocabulary of
// 10^5 entries or more, Section 6.1 of the paper) is cut into slices, one per block of a thread-block
// cluster.  The blocks of a cluster exchange their slice results over distributed shared memory, so
// no scratch in global memory is needed.  Both distances need a second look at the row once a
// row-wide quantity is known (the softmax normalisers; a lower bound of the K-th largest entry).
// The second pass reads the same slice again while it is still in L2: the slices in flight over
// the whole GPU stay far below the L2 size, so HBM sees every byte once.
#include <cooperative_groups.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "../../include/imm.h"

namespace imm_ldd {

namespace cg = cooperative_groups;

constexpr int THREADS = 512;
constexpr int WARPS = THREADS / 32;
constexpr int MAX_CLUSTER = 8;
constexpr int SLICE = 16384;                  // entries of a row one block takes (before the cluster cap)
constexpr int MAX_K = IMM_LDD_MAX_K;          // largest index set of the Top-K distance
constexpr int COLLECT_CAP = 256;              // entries above the bound a block can hold per pass (a power of two)
constexpr int MAX_REFINE = 6;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float NEG_INF = -INFINITY;

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Slice of block c: [s0, s1), s0 a multiple of 4 so that 16-byte loads stay aligned.
__device__ __forceinline__ void slice_bounds(int64_t n, int nc, int c, int64_t& s0, int64_t& s1)
{
    const int64_t per = ((n + nc - 1) / nc + 3) / 4 * 4;
    s0 = min(n, (int64_t)c * per);
    s1 = min(n, s0 + per);
}

// running (max, sum of exp(x - max)) of a softmax, in base 2 internally
struct MaxSum { float m, s; };

__device__ __forceinline__ void ms_add4(MaxSum& a, float x0, float x1, float x2, float x3)
{
    const float vm = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
    if (vm > a.m) { a.s *= ex2((a.m - vm) * LOG2E); a.m = vm; }
    // (x - max) first: exact for entries near the maximum, whatever the magnitude of the logits
    a.s += ex2((x0 - a.m) * LOG2E) + ex2((x1 - a.m) * LOG2E) + ex2((x2 - a.m) * LOG2E) + ex2((x3 - a.m) * LOG2E);
}

__device__ __forceinline__ void ms_add1(MaxSum& a, float x)
{
    if (x > a.m) { a.s *= ex2((a.m - x) * LOG2E); a.m = x; }
    a.s += ex2((x - a.m) * LOG2E);
}

__device__ __forceinline__ MaxSum ms_merge(MaxSum a, MaxSum b)
{
    const float m = fmaxf(a.m, b.m);
    if (m == NEG_INF) return MaxSum{NEG_INF, 0.f};                    // both empty
    return MaxSum{m, a.s * ex2((a.m - m) * LOG2E) + b.s * ex2((b.m - m) * LOG2E)};
}

__device__ __forceinline__ MaxSum ms_warp(MaxSum a)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MaxSum b{__shfl_xor_sync(0xFFFFFFFFu, a.m, o), __shfl_xor_sync(0xFFFFFFFFu, a.s, o)};
        a = ms_merge(a, b);
    }
    return a;
}

__device__ __forceinline__ float4 ld4(const float* p)
{
    return __ldg(reinterpret_cast<const float4*>(p));
}

// ------------------------------------------------------------------------------------------
// TV and KL distance
// ------------------------------------------------------------------------------------------
// Pass 1 (from HBM): running max and sum of exponentials of both rows, merged over the block and
// then over the cluster.  Pass 2 (from L2): with both normalisers known,
//   tv += |p_v - q_v|,   kl += q_v * (log q_v - log p_v),   p = softmax(x), q = softmax(y).
// x is the deployed row, y the reference row.

template <int NW>
struct TvKlShared {
    MaxSum warp_p[NW], warp_q[NW];
    MaxSum pub_p, pub_q;                  // this block's slice; read by the other blocks
    float max_p, max_q, l2s_p, l2s_q;     // the rows' maxima and log2 of their sums of exp(x - max)
    float warp_tv[NW], warp_kl[NW];
    double pub_tv, pub_kl;                // this block's share; read by block 0
};

template <bool VEC, int NT>
__global__ void __launch_bounds__(NT)
tv_kl_kernel(const float* __restrict__ logits, const float* __restrict__ ref, int64_t n, int64_t ld,
             double* __restrict__ tv_out, double* __restrict__ kl_out)
{
    constexpr int NW = NT / 32;
    __shared__ TvKlShared<NW> sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int nc = (int)cluster.num_blocks(), c = (int)cluster.block_rank();
    const int64_t step = blockIdx.x / nc;
    const float* x = logits + step * ld;
    const float* y = ref + step * ld;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int64_t s0, s1;
    slice_bounds(n, nc, c, s0, s1);

    MaxSum ap{NEG_INF, 0.f}, aq{NEG_INF, 0.f};
    for (int64_t i = s0 + 4 * tid; i < s1; i += 4 * NT) {
        if (VEC && i + 4 <= s1) {
            const float4 a = ld4(x + i), b = ld4(y + i);
            ms_add4(ap, a.x, a.y, a.z, a.w);
            ms_add4(aq, b.x, b.y, b.z, b.w);
        } else {
            for (int64_t e = i; e < min(i + 4, s1); e++) { ms_add1(ap, x[e]); ms_add1(aq, y[e]); }
        }
    }
    ap = ms_warp(ap); aq = ms_warp(aq);
    if (lane == 0) { sh.warp_p[warp] = ap; sh.warp_q[warp] = aq; }
    __syncthreads();
    if (warp == 0) {
        MaxSum p = lane < NW ? sh.warp_p[lane] : MaxSum{NEG_INF, 0.f};
        MaxSum q = lane < NW ? sh.warp_q[lane] : MaxSum{NEG_INF, 0.f};
        p = ms_warp(p); q = ms_warp(q);
        if (lane == 0) { sh.pub_p = p; sh.pub_q = q; }
    }
    cluster.sync();                                        // every block's slice result is published
    if (warp == 0) {
        MaxSum p = lane < nc ? *cluster.map_shared_rank(&sh.pub_p, lane) : MaxSum{NEG_INF, 0.f};
        MaxSum q = lane < nc ? *cluster.map_shared_rank(&sh.pub_q, lane) : MaxSum{NEG_INF, 0.f};
        p = ms_warp(p); q = ms_warp(q);
        if (lane == 0) { sh.max_p = p.m; sh.max_q = q.m; sh.l2s_p = log2f(p.s); sh.l2s_q = log2f(q.s); }
    }
    __syncthreads();
    // entries are taken relative to their row's maximum, so logits of large magnitude lose nothing
    const float mp = sh.max_p, mq = sh.max_q, lp = sh.l2s_p, lq = sh.l2s_q;
    const float dl = (lq - lp) * (1.0f / LOG2E);           // log(sum_q) - log(sum_p), natural units

    float tv = 0.f, kl = 0.f;
    for (int64_t i = s0 + 4 * tid; i < s1; i += 4 * NT) {
        float xs[4], ys[4];
        int cnt = 4;
        if (VEC && i + 4 <= s1) {
            const float4 a = ld4(x + i), b = ld4(y + i);
            xs[0] = a.x; xs[1] = a.y; xs[2] = a.z; xs[3] = a.w;
            ys[0] = b.x; ys[1] = b.y; ys[2] = b.z; ys[3] = b.w;
        } else {
            cnt = (int)(min(i + 4, s1) - i);
            for (int e = 0; e < 4; e++) { xs[e] = e < cnt ? x[i + e] : 0.f; ys[e] = e < cnt ? y[i + e] : 0.f; }
        }
#pragma unroll
        for (int e = 0; e < 4; e++) {
            if (e < cnt) {
                const float xr = xs[e] - mp, yr = ys[e] - mq;
                const float p = ex2(fmaf(xr, LOG2E, -lp)), q = ex2(fmaf(yr, LOG2E, -lq));
                tv += fabsf(p - q);
                kl = fmaf(q, (yr - xr) - dl, kl);            // log q_v - log p_v
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        tv += __shfl_xor_sync(0xFFFFFFFFu, tv, o);
        kl += __shfl_xor_sync(0xFFFFFFFFu, kl, o);
    }
    if (lane == 0) { sh.warp_tv[warp] = tv; sh.warp_kl[warp] = kl; }
    __syncthreads();
    if (tid == 0) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < NW; w++) { a += (double)sh.warp_tv[w]; b += (double)sh.warp_kl[w]; }
        sh.pub_tv = a; sh.pub_kl = b;
    }
    cluster.sync();                                        // every block's share is published
    if (c == 0 && tid == 0) {
        double a = 0.0, b = 0.0;
        for (int cc = 0; cc < nc; cc++) {
            a += *cluster.map_shared_rank(&sh.pub_tv, cc);
            b += *cluster.map_shared_rank(&sh.pub_kl, cc);
        }
        tv_out[step] = 0.5 * a;
        kl_out[step] = b;
    }
    cluster.sync();                                        // block 0 has read the shares: the others may leave
}

// ------------------------------------------------------------------------------------------
// Top-K distance
// ------------------------------------------------------------------------------------------
// Delta(l, I) = min_t  sum_{j not in I} max(l_j - t, 0) + sum_{i in I} max(t - l_i, 0).
// The cost is convex and piecewise linear in t, and below the K-th largest entry outside I its
// slope is <= 0 (at least K entries outside I lie above t, at most K entries of I below).  So a
// minimiser lies at or above that entry, where only the K largest entries outside I contribute,
// and the minimum is attained at one of 2K breakpoints: those K entries and the K entries of I.
// The kernel therefore needs the K largest entries outside I, exactly:
//   pass 1 (HBM): the largest entry outside I of every group of G threads, G chosen so that the
//                 cluster has at least 2K groups; the K-th largest of these maxima is a lower bound
//                 tau of the K-th largest entry outside I, and close to it: for a 128k-entry row
//                 about K + 2 entries lie above it.  Every block finds tau by itself from the
//                 other blocks' maxima (distributed shared memory), by ranking, without a sort;
//   pass 2 (L2):  collect the entries outside I above tau (unless the row is adversarial; then
//                 tau is raised from what was collected and the pass repeats);
//   block 0 ranks what the cluster collected together with K copies of tau (K entries outside I
//   are >= tau), keeps the K largest, and evaluates the cost at the 2K breakpoints in float64.

constexpr int MAX_CAND = 256;                 // group maxima of the whole cluster (>= 2 * MAX_K, <= THREADS)

struct TopkShared {
    float cand[MAX_CAND];                 // this block's group maxima (the first `ncand` entries)
    float all[MAX_CLUSTER * COLLECT_CAP + MAX_K];   // the cluster's maxima; block 0: the collected entries
    float topk[MAX_K];                    // block 0: the K largest entries outside I
    float collected[COLLECT_CAP];         // entries outside I above tau
    float inside[MAX_K];                  // block 0: the entries of I
    double cost[2 * MAX_K];
    float tau, proposal, new_tau;
    int count;                            // entries collected in this pass (may exceed COLLECT_CAP)
    int total, over, bad;
};

// rank of all[i] in descending order, ties broken by position: a permutation of 0..m-1
__device__ __forceinline__ int rank_desc(const float* all, int m, int i)
{
    const float v = all[i];
    int r = 0;
    for (int j = 0; j < m; j++) {
        const float w = all[j];
        r += (w > v || (w == v && j < i)) ? 1 : 0;
    }
    return r;
}

template <bool VEC>
__global__ void __launch_bounds__(THREADS, 3)
topk_distance_kernel(const float* __restrict__ ref, int64_t n, int64_t ld, const int32_t* __restrict__ topk,
                     int K, double* __restrict__ dist_out, int32_t* __restrict__ status)
{
    extern __shared__ uint32_t member[];               // bitmap of the slice's entries that belong to I
    __shared__ TopkShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int nc = (int)cluster.num_blocks(), c = (int)cluster.block_rank();
    const int64_t step = blockIdx.x / nc;
    const int32_t* I = topk + step * K;
    const int tid = threadIdx.x, lane = tid & 31;
    int64_t s0, s1;
    slice_bounds(n, nc, c, s0, s1);
    const float* row = ref + step * ld;
    const float* y = row + s0;                         // this block's slice
    const int len = (int)(s1 - s0);
    const int nvec = VEC ? len >> 2 : 0;               // whole 16-byte vectors; the rest goes entry by entry
    const float4* yv = reinterpret_cast<const float4*>(y);
    const int words = (len + 31) / 32 + 1;

    for (int i = tid; i < words; i += THREADS) member[i] = 0;
    if (tid == 0) { sh.bad = 0; sh.count = 0; }
    __syncthreads();
    if (tid < K) {
        const int64_t idx = I[tid];
        if (idx < 0 || idx >= n) sh.bad = 1;
        else {
            if (c == 0) sh.inside[tid] = row[idx];     // block 0 needs the entries of I at the end
            if (idx >= s0 && idx < s1) {
                const int rel = (int)(idx - s0);
                const uint32_t bit = 1u << (rel & 31);
                if (atomicOr(&member[rel >> 5], bit) & bit) sh.bad = 1;      // the same index twice
            }
        }
    }
    __syncthreads();

    // pass 1: this thread's largest entry outside I
    float best = NEG_INF;
    for (int v = tid; v < nvec; v += THREADS) {
        const float4 q = __ldg(yv + v);
        const uint32_t m = member[v >> 3] >> ((4 * v) & 31);       // four consecutive bits of one word
        best = fmaxf(best, (m & 1u) ? NEG_INF : q.x);
        best = fmaxf(best, (m & 2u) ? NEG_INF : q.y);
        best = fmaxf(best, (m & 4u) ? NEG_INF : q.z);
        best = fmaxf(best, (m & 8u) ? NEG_INF : q.w);
    }
    for (int e = 4 * nvec + tid; e < len; e += THREADS)
        if (!((member[e >> 5] >> (e & 31)) & 1u)) best = fmaxf(best, y[e]);
    const float thread_best = best;

    // group maxima: groups of G = THREADS / ncand threads, ncand the smallest power of two (16 at
    // least: one group per warp) that gives the cluster 2K groups; nc * ncand <= MAX_CAND
    int ncand = WARPS;
    while (ncand * nc < 2 * K) ncand <<= 1;
    const int G = THREADS / ncand;                     // 32, 16, 8 or 4
    for (int o = 1; o < G; o <<= 1) best = fmaxf(best, __shfl_xor_sync(0xFFFFFFFFu, best, o));
    if ((tid % G) == 0) sh.cand[tid / G] = best;
    cluster.sync();                                    // every block's group maxima are in place

    // tau = K-th largest of the cluster's group maxima; every block works it out by itself
    const int total = nc * ncand;
    if (tid < total) sh.all[tid] = cluster.map_shared_rank(sh.cand, tid / ncand)[tid % ncand];
    __syncthreads();
    if (tid < total && rank_desc(sh.all, total, tid) == K - 1) sh.tau = sh.all[tid];
    __syncthreads();
    float tau = sh.tau;

    bool failed = false;
    for (int round = 0;; round++) {
        // pass 2: collect the entries outside I above tau
        for (int v = tid; v < nvec; v += THREADS) {
            const float4 q = __ldg(yv + v);
            const uint32_t m = member[v >> 3] >> ((4 * v) & 31);
            const float vals[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int e = 0; e < 4; e++)
                if (!((m >> e) & 1u) && vals[e] > tau) {
                    const int slot = atomicAdd(&sh.count, 1);
                    if (slot < COLLECT_CAP) sh.collected[slot] = vals[e];
                }
        }
        for (int e = 4 * nvec + tid; e < len; e += THREADS)
            if (!((member[e >> 5] >> (e & 31)) & 1u) && y[e] > tau) {
                const int slot = atomicAdd(&sh.count, 1);
                if (slot < COLLECT_CAP) sh.collected[slot] = y[e];
            }
        __syncthreads();
        // A block that could not hold everything proposes a higher bound.  The K-th largest of its
        // threads' maxima, and the K-th largest of the entries it did hold, are both entries outside I
        // with K entries at or above them, so either is still a lower bound; the second one lies
        // above tau, so the bound rises every round.
        if (sh.count > COLLECT_CAP) {
            sh.all[tid] = thread_best;
            __syncthreads();
            if (rank_desc(sh.all, THREADS, tid) == K - 1) sh.proposal = sh.all[tid];
            __syncthreads();
            if (tid < COLLECT_CAP) sh.all[tid] = sh.collected[tid];
            __syncthreads();
            if (tid < COLLECT_CAP && rank_desc(sh.all, COLLECT_CAP, tid) == K - 1) sh.proposal = fmaxf(sh.proposal, sh.all[tid]);
        } else if (tid == 0) sh.proposal = NEG_INF;
        cluster.sync();                                // counts, collected entries and proposals are in place
        if (tid < 32) {
            const int cnt = lane < nc ? *cluster.map_shared_rank(&sh.count, lane) : 0;
            float prop = lane < nc ? *cluster.map_shared_rank(&sh.proposal, lane) : NEG_INF;
            const int bad = lane < nc ? *cluster.map_shared_rank(&sh.bad, lane) : 0;
            const unsigned over = __ballot_sync(0xFFFFFFFFu, cnt > COLLECT_CAP);
            const unsigned anybad = __ballot_sync(0xFFFFFFFFu, bad != 0);
            int sum = min(cnt, COLLECT_CAP);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                prop = fmaxf(prop, __shfl_xor_sync(0xFFFFFFFFu, prop, o));
                sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
            }
            if (lane == 0) { sh.over = over != 0; sh.new_tau = fmaxf(tau, prop); sh.total = sum; if (anybad) sh.bad = 2; }
        }
        __syncthreads();
        if (!sh.over) break;
        if (round + 1 == MAX_REFINE) { failed = true; break; }     // gave up raising the bound
        tau = sh.new_tau;
        cluster.sync();                                // every block has read the counts: they may be reset
        if (tid == 0) sh.count = 0;
        __syncthreads();
    }

    if (c == 0) {
        // what the cluster collected, plus K copies of tau
        int fill = 0;
        for (int cc = 0; cc < nc; cc++) {
            const int cnt = min(*cluster.map_shared_rank(&sh.count, cc), COLLECT_CAP);
            const float* src = cluster.map_shared_rank(sh.collected, cc);
            for (int i = tid; i < cnt; i += THREADS) sh.all[fill + i] = src[i];
            fill += cnt;
        }
        for (int i = tid; i < K; i += THREADS) sh.all[fill + i] = tau;
        fill += K;
        __syncthreads();
        for (int i = tid; i < fill; i += THREADS) {
            const int r = rank_desc(sh.all, fill, i);
            if (r < K) sh.topk[r] = sh.all[i];
        }
        __syncthreads();
        // cost at the 2K breakpoints, in double
        if (tid < 2 * K) {
            const double t = tid < K ? (double)sh.topk[tid] : (double)sh.inside[tid - K];
            double cost = INFINITY;
            if (t > -INFINITY) {                       // a row with fewer than K entries outside I pads with -inf
                cost = 0.0;
                for (int k = 0; k < K; k++) {
                    cost += fmax((double)sh.topk[k] - t, 0.0);
                    cost += fmax(t - (double)sh.inside[k], 0.0);
                }
            }
            sh.cost[tid] = cost;
        }
        __syncthreads();
        if (tid < 32) {
            double best_cost = INFINITY;
            for (int i = lane; i < 2 * K; i += 32) best_cost = fmin(best_cost, sh.cost[i]);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) best_cost = fmin(best_cost, __shfl_xor_sync(0xFFFFFFFFu, best_cost, o));
            if (lane == 0) {
                const bool bad = sh.bad != 0;
                dist_out[step] = (bad || failed) ? NAN : best_cost;
                status[step] = bad ? IMM_ERR_ARG : failed ? IMM_ERR_LIMIT : IMM_OK;
            }
        }
    }
    cluster.sync();                                    // block 0 has read the other blocks' memory
}

// ------------------------------------------------------------------------------------------
// per-request tail statistic
// ------------------------------------------------------------------------------------------
// p[r] = |{ steps of request r with distance > t1 }| / (steps of request r);  flag[r] = p[r] > t2.

__global__ void __launch_bounds__(256)
tail_fraction_kernel(const double* __restrict__ dist, const int64_t* __restrict__ offsets, double t1, double t2,
                     double* __restrict__ p_out, int32_t* __restrict__ flag_out)
{
    __shared__ int warp_cnt[8];
    const int64_t r = blockIdx.x;
    const int64_t b = offsets[r], e = offsets[r + 1];
    int cnt = 0;
    for (int64_t i = b + threadIdx.x; i < e; i += blockDim.x) cnt += dist[i] > t1 ? 1 : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xFFFFFFFFu, cnt, o);
    if ((threadIdx.x & 31) == 0) warp_cnt[threadIdx.x >> 5] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t total = 0;
        for (int w = 0; w < 8; w++) total += warp_cnt[w];
        const double p = e > b ? (double)total / (double)(e - b) : 0.0;
        p_out[r] = p;
        if (flag_out) flag_out[r] = p > t2 ? 1 : 0;
    }
}

int cluster_size(int64_t n)
{
    int nc = 1;
    while (nc < MAX_CLUSTER && (int64_t)nc * SLICE < n) nc *= 2;
    return nc;
}

template <typename... Args>
cudaError_t launch_cluster(void (*kernel)(Args...), int64_t steps, int nc, int threads, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(steps * nc));
    cfg.blockDim = dim3((unsigned)threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr;
    memset(&attr, 0, sizeof(attr));
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = (unsigned)nc;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

bool rows_aligned(const void* p, int64_t ld) { return ((uintptr_t)p % 16 == 0) && (ld % 4 == 0); }

}  // namespace imm_ldd

extern "C" {

int imm_ldd_tv_kl(const float* d_logits, const float* d_ref_logits, int64_t steps, int64_t n, int64_t ld,
                  double* d_tv, double* d_kl, void* stream)
{
    using namespace imm_ldd;
    if (!d_logits || !d_ref_logits || !d_tv || !d_kl) return IMM_ERR_ARG;
    if (steps < 0 || n <= 0 || ld < n || n > IMM_LDD_MAX_N || steps > IMM_LDD_MAX_STEPS) return IMM_ERR_SHAPE;
    if ((uintptr_t)d_logits % 4 || (uintptr_t)d_ref_logits % 4 || (uintptr_t)d_tv % 8 || (uintptr_t)d_kl % 8) return IMM_ERR_ALIGN;
    if (steps == 0) return IMM_OK;
    const int nc = cluster_size(n);
    const bool vec = rows_aligned(d_logits, ld) && rows_aligned(d_ref_logits, ld);
    int nt = 512, ncl = nc;
    if (const char* v = getenv("IMM_LDD_THREADS")) nt = atoi(v) == 256 ? 256 : atoi(v) == 1024 ? 1024 : 512;
    if (const char* v = getenv("IMM_LDD_CLUSTER")) { int c = atoi(v); if (c == 1 || c == 2 || c == 4 || c == 8 || c == 16) ncl = c; }
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
#define TVKL_LAUNCH(V, T) do { \
        if (ncl > 8) cudaFuncSetAttribute(tv_kl_kernel<V, T>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1); \
        e = launch_cluster(tv_kl_kernel<V, T>, steps, ncl, T, 0, st, d_logits, d_ref_logits, n, ld, d_tv, d_kl); } while (0)
    if (!vec) TVKL_LAUNCH(false, 512);
    else if (nt == 256) TVKL_LAUNCH(true, 256);
    else if (nt == 1024) TVKL_LAUNCH(true, 1024);
    else TVKL_LAUNCH(true, 512);
#undef TVKL_LAUNCH
    return e == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
}

int imm_ldd_topk_distance(const float* d_ref_logits, int64_t steps, int64_t n, int64_t ld,
                          const int32_t* d_topk, int k, double* d_dist, int32_t* d_status, void* stream)
{
    using namespace imm_ldd;
    if (!d_ref_logits || !d_topk || !d_dist || !d_status) return IMM_ERR_ARG;
    if (steps < 0 || n <= 0 || ld < n || n > IMM_LDD_MAX_N || steps > IMM_LDD_MAX_STEPS) return IMM_ERR_SHAPE;
    if (k <= 0 || k > IMM_LDD_MAX_K || k > n) return IMM_ERR_SHAPE;
    if ((uintptr_t)d_ref_logits % 4 || (uintptr_t)d_topk % 4 || (uintptr_t)d_dist % 8 || (uintptr_t)d_status % 4) return IMM_ERR_ALIGN;
    if (steps == 0) return IMM_OK;
    const int nc = cluster_size(n);
    const bool vec = rows_aligned(d_ref_logits, ld);
    const int64_t per = ((n + nc - 1) / nc + 3) / 4 * 4;                     // entries per block (see slice_bounds)
    const size_t smem = (size_t)((per + 31) / 32 + 2) * sizeof(uint32_t);    // the membership bitmap (<= 16 KiB)
    cudaError_t e = vec ? launch_cluster(topk_distance_kernel<true>, steps, nc, THREADS, smem, (cudaStream_t)stream, d_ref_logits, n, ld, d_topk, k, d_dist, d_status)
                        : launch_cluster(topk_distance_kernel<false>, steps, nc, THREADS, smem, (cudaStream_t)stream, d_ref_logits, n, ld, d_topk, k, d_dist, d_status);
    return e == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
}

int imm_ldd_tail_fraction(const double* d_dist, const int64_t* d_offsets, int64_t nrequests, double t1, double t2,
                          double* d_p, int32_t* d_flag, void* stream)
{
    using namespace imm_ldd;
    if (!d_dist || !d_offsets || !d_p) return IMM_ERR_ARG;
    if (nrequests < 0 || nrequests > IMM_LDD_MAX_STEPS) return IMM_ERR_SHAPE;
    if ((uintptr_t)d_dist % 8 || (uintptr_t)d_offsets % 8 || (uintptr_t)d_p % 8 || (uintptr_t)d_flag % 4) return IMM_ERR_ALIGN;
    if (nrequests == 0) return IMM_OK;
    tail_fraction_kernel<<<(unsigned)nrequests, 256, 0, (cudaStream_t)stream>>>(d_dist, d_offsets, t1, t2, d_p, d_flag);
    return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
}

}  // extern "C"
