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
constexpr int MAX_CLUSTER = 8;
constexpr int SLICE = 16384;                  // entries of a row one block takes (before the cluster cap)
constexpr int MAX_K = IMM_LDD_MAX_K;          // largest index set of the Top-K distance
constexpr int COLLECT_CAP = 256;              // entries above the bound a block can hold per pass (a power of two)
constexpr int MAX_REFINE = 6;
constexpr float LOG2E = 1.4426950408889634f;
constexpr float NEG_INF = -INFINITY;
// Running maxima start at the lowest finite float, not at -inf: a masked logit (-inf, probability
// 0) then always meets a finite maximum, so (x - max) is -inf and its exponential 0, never the
// NaN of (-inf) - (-inf).
constexpr float EMPTY_MAX = -3.402823466e+38f;

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Slice of block c: [s0, s1), s0 a multiple of 4 so that 16-byte loads stay aligned.
__device__ __forceinline__ void slice_bounds(int64_t n, int nc, int c, int64_t& s0, int64_t& s1)
{
    const int64_t per = (((uint32_t)n + (uint32_t)nc - 1) / (uint32_t)nc + 3) / 4 * 4;     // (n <= 2^20: a 32-bit division)
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

// Merge over a warp: the maximum first, then every lane rescales its own sum once and the sums are
// added (one exponential per lane instead of two per merge step).
__device__ __forceinline__ MaxSum ms_warp(MaxSum a)
{
    float m = a.m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    float s = a.s * ex2((a.m - m) * LOG2E);                // (an empty lane holds sum 0 and contributes nothing)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    return MaxSum{m, s};
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
    double share_tv[MAX_CLUSTER], share_kl[MAX_CLUSTER];   // block 0: every block's share, stored here by its owner
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

    MaxSum ap{EMPTY_MAX, 0.f}, aq{EMPTY_MAX, 0.f};
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
        MaxSum p = lane < NW ? sh.warp_p[lane] : MaxSum{EMPTY_MAX, 0.f};
        MaxSum q = lane < NW ? sh.warp_q[lane] : MaxSum{EMPTY_MAX, 0.f};
        p = ms_warp(p); q = ms_warp(q);
        if (lane == 0) { sh.pub_p = p; sh.pub_q = q; }
    }
    cluster.sync();                                        // every block's slice result is published
    if (warp == 0) {
        MaxSum p = lane < nc ? *cluster.map_shared_rank(&sh.pub_p, lane) : MaxSum{EMPTY_MAX, 0.f};
        MaxSum q = lane < nc ? *cluster.map_shared_rank(&sh.pub_q, lane) : MaxSum{EMPTY_MAX, 0.f};
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
                // q_v (log q_v - log p_v) without its constant part (below); 0 log 0 = 0, so an entry
                // without reference mass is skipped (its yr - xr may be -inf or NaN)
                if (q > 0.f) kl = fmaf(q, yr - xr, kl);
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
    if (tid == 0) {                                        // this block's share goes into block 0's shared memory
        double a = 0.0, b = 0.0;                           // (every block is running: the barrier above was passed)
        for (int w = 0; w < NW; w++) { a += (double)sh.warp_tv[w]; b += (double)sh.warp_kl[w]; }
        *cluster.map_shared_rank(&sh.share_tv[c], 0) = a;
        *cluster.map_shared_rank(&sh.share_kl[c], 0) = b;
    }
    cluster.sync();                                        // the shares have arrived; nobody reads another block any more
    if (c == 0 && tid == 0) {
        double a = 0.0, b = 0.0;
        for (int cc = 0; cc < nc; cc++) { a += sh.share_tv[cc]; b += sh.share_kl[cc]; }
        // a row without a finite entry has sum 0 (log2 = -inf) and no distribution: both distances are NaN
        const bool dead = !(lp > NEG_INF) || !(lq > NEG_INF);
        tv_out[step] = dead ? (double)NAN : 0.5 * a;
        kl_out[step] = dead ? (double)NAN : b - (double)dl;   // sum_v q_v (log S_q - log S_p) = log S_q - log S_p: q sums to 1
    }
}

// ------------------------------------------------------------------------------------------
// Top-K distance
// ------------------------------------------------------------------------------------------
// Delta(l, I) = min_t  sum_{j not in I} max(l_j - t, 0) + sum_{i in I} max(t - l_i, 0).
// The cost is convex and piecewise linear in t, and below the K-th largest entry outside I its
// slope is <= 0 (at least K entries outside I lie above t, at most K entries of I below).  So a
// minimiser lies at or above that entry, where only the K largest entries outside I contribute,
// and the minimum is attained at one of 2K breakpoints: those K entries and the K entries of I.
// The kernel therefore needs the K largest entries outside I, exactly.  They are among the K
// largest of every slice, and the blocks that take the slices of a row never wait for one another:
//   a thread loads its 32 entries of the slice once and keeps them in registers; the largest entry
//   outside I of every group of G threads (at least 2K groups) gives, as the K-th largest of these
//   maxima, a lower bound tau of the slice's K-th largest entry outside I, and a close one: about
//   1.3 K entries lie above it; the entries outside I above tau are collected from the registers
//   (unless the slice is adversarial; then tau is raised from what was collected and the collection
//   repeats);
//   the K largest of what was collected, padded with copies of tau (K entries outside I are >=
//   tau), go to the workspace.  A second, small kernel merges the slices' lists of every row,
//   keeps the K largest, and evaluates the cost at the 2K breakpoints in float64.

#ifndef IMM_LDD_TK_THREADS
#define IMM_LDD_TK_THREADS 256
#endif
constexpr int TK_THREADS = IMM_LDD_TK_THREADS;   // threads per block of the Top-K kernel
constexpr int TK_SLICE = 32 * TK_THREADS;         // entries of a row per block: 32 per thread, in registers
constexpr int MAX_CAND = 128;                 // group maxima per block (>= 2 * MAX_K)
constexpr int MERGE_CAP = (IMM_LDD_MAX_N / TK_SLICE) * MAX_K;   // a row's lists, held at once by the merging block
constexpr int TK_MERGE_THREADS = 128;         // >= 2 * MAX_K

struct TopkShared {
    float work[TK_THREADS + COLLECT_CAP]; // thread maxima / group maxima / collected entries plus copies of tau
    float collected[COLLECT_CAP];         // entries above tau ...
    int collected_at[COLLECT_CAP];        // ... and where in the slice they sit
    int member_at[MAX_K];                 // the entries of I that fall into this slice
    float tau, proposal;
    int count;                            // entries collected in this pass (may exceed COLLECT_CAP)
    int members, bad;
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

// The entries of I are not masked while streaming (that would cost more instructions per entry
// than everything else together).  With m of them in the slice, the (K + m)-th largest group
// maximum still has K entries outside I at or above it, so it is a valid bound; entries of I
// that get collected are dropped afterwards by their position.
template <bool VEC>
__global__ void __launch_bounds__(TK_THREADS, 1024 / TK_THREADS)
topk_slice_kernel(const float* __restrict__ ref, int64_t n, int64_t ld, const int32_t* __restrict__ topk,
                  int K, int nslices, float* __restrict__ lists, int32_t* __restrict__ flags)
{
    __shared__ TopkShared sh;
    const int64_t step = blockIdx.x / nslices;
    const int c = (int)(blockIdx.x % nslices);
    const int32_t* I = topk + step * K;
    const int tid = threadIdx.x;
    const int64_t s0 = (int64_t)c * TK_SLICE, s1 = min(n, s0 + TK_SLICE);
    const float* y = ref + step * ld + s0;             // this block's slice
    const int len = (int)(s1 - s0);
    const int nvec = VEC ? len >> 2 : 0;               // whole 16-byte vectors; the rest goes entry by entry
    const float4* yv = reinterpret_cast<const float4*>(y);

    // The thread's 32 entries of the slice stay in registers: all loads are issued at once (before
    // anything else, so that the set-up below runs while they are in flight), and the second look
    // at the data, once tau is known, needs no memory access.  Slots past the end hold -inf.
    constexpr int PER = TK_SLICE / TK_THREADS;         // 32 entries per thread
    float vals[PER];
    if (VEC) {
        if (len == TK_SLICE) {
#pragma unroll
            for (int u = 0; u < PER / 4; u++) {
                const float4 q = __ldg(yv + tid + u * TK_THREADS);
                vals[4 * u] = q.x; vals[4 * u + 1] = q.y; vals[4 * u + 2] = q.z; vals[4 * u + 3] = q.w;
            }
        } else {
#pragma unroll
            for (int u = 0; u < PER / 4; u++) {
                const int v = tid + u * TK_THREADS;
                const float4 q = v < nvec ? __ldg(yv + v) : make_float4(NEG_INF, NEG_INF, NEG_INF, NEG_INF);
                vals[4 * u] = q.x; vals[4 * u + 1] = q.y; vals[4 * u + 2] = q.z; vals[4 * u + 3] = q.w;
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < PER; j++) {
            const int e = tid + j * TK_THREADS;
            vals[j] = e < len ? y[e] : NEG_INF;
        }
    }
    // aligned rows: the up to three entries after the last whole vector
    const int tail_at = 4 * nvec + tid;
    const float tail = (VEC && tail_at < len) ? y[tail_at] : NEG_INF;

    if (tid == 0) { sh.bad = 0; sh.count = 0; sh.members = 0; }
    __syncthreads();
    if (tid < K) {
        const int64_t idx = I[tid];
        if (idx < 0 || idx >= n) sh.bad = 1;
        else if (idx >= s0 && idx < s1) sh.member_at[atomicAdd(&sh.members, 1)] = (int)(idx - s0);
    }
    __syncthreads();
    const int members = sh.members;
    if (tid < members)                                 // the same index twice?
        for (int k = 0; k < tid; k++)
            if (sh.member_at[k] == sh.member_at[tid]) sh.bad = 1;

    float best = tail;
#pragma unroll
    for (int j = 0; j < PER; j++) best = fmaxf(best, vals[j]);
    const float thread_best = best;                    // (before the group reduction below)

    // group maxima: ncand groups, the smallest power of two (32 at least) above K + m, so that the
    // bound's rank K + m - 1 exists; fewer groups make the ranking below cheaper
    int ncand = 32;
    while (ncand <= K + members) ncand <<= 1;          // <= MAX_CAND
    static_assert(MAX_CAND >= 2 * MAX_K && MAX_CAND <= TK_THREADS, "group maxima must fit the block");
    const int G = TK_THREADS / ncand;
    for (int o = 1; o < G; o <<= 1) best = fmaxf(best, __shfl_xor_sync(0xFFFFFFFFu, best, o));
    if ((tid % G) == 0) sh.work[tid / G] = best;
    __syncthreads();
    const int want = K + members - 1;                  // rank of the bound: K entries outside I are at or above it
    if (tid < ncand && rank_desc(sh.work, ncand, tid) == want) sh.tau = sh.work[tid];
    __syncthreads();
    float tau = sh.tau;

    bool failed = false;
    for (int round = 0;; round++) {
        // collect the entries above tau (from registers)
        if (thread_best > tau) {                       // rare: about K + a few threads of the block
#pragma unroll
            for (int j = 0; j < PER; j++)
                if (vals[j] > tau) {
                    const int slot = atomicAdd(&sh.count, 1);
                    if (slot < COLLECT_CAP) {
                        sh.collected[slot] = vals[j];
                        sh.collected_at[slot] = VEC ? 4 * (tid + (j >> 2) * TK_THREADS) + (j & 3) : tid + j * TK_THREADS;
                    }
                }
            if (tail > tau) {
                const int slot = atomicAdd(&sh.count, 1);
                if (slot < COLLECT_CAP) { sh.collected[slot] = tail; sh.collected_at[slot] = tail_at; }
            }
        }
        __syncthreads();
        if (sh.count <= COLLECT_CAP) break;
        if (round + 1 == MAX_REFINE) { failed = true; break; }     // gave up raising the bound
        // More than the block can hold: raise the bound.  The (K + m)-th largest of the threads'
        // maxima, and the (K + m)-th largest of the entries that were held, both have K entries
        // outside I at or above them, so either is still a lower bound; the second one lies above
        // tau, so the bound rises every round.
        sh.work[tid] = thread_best;
        __syncthreads();
        if (rank_desc(sh.work, TK_THREADS, tid) == want) sh.proposal = sh.work[tid];
        __syncthreads();
        if (tid < COLLECT_CAP) sh.work[tid] = sh.collected[tid];
        __syncthreads();
        if (tid < COLLECT_CAP && rank_desc(sh.work, COLLECT_CAP, tid) == want) sh.proposal = fmaxf(sh.proposal, sh.work[tid]);
        __syncthreads();
        tau = fmaxf(tau, sh.proposal);
        if (tid == 0) sh.count = 0;
        __syncthreads();
    }

    // this slice's K largest entries outside I: what was collected, without the entries of I, plus
    // K copies of tau
    {
        const int cnt = min(sh.count, COLLECT_CAP);
        for (int i = tid; i < cnt; i += TK_THREADS) {
            float v = sh.collected[i];
            const int at = sh.collected_at[i];
            for (int k = 0; k < members; k++) if (sh.member_at[k] == at) v = NEG_INF;
            sh.work[i] = v;
        }
        for (int i = tid; i < K; i += TK_THREADS) sh.work[cnt + i] = tau;
        __syncthreads();
        float* mine = lists + ((int64_t)step * nslices + c) * K;
        for (int i = tid; i < cnt + K; i += TK_THREADS) {
            const int r = rank_desc(sh.work, cnt + K, i);
            if (r < K) mine[r] = sh.work[i];
        }
    }
    if (tid == 0) flags[(int64_t)step * nslices + c] = (sh.bad ? 1 : 0) | (failed ? 2 : 0);
}

// One block per row: the K largest of the slices' lists, the entries of I, the cost at the 2K
// breakpoints in float64.  The lists are sorted, so their first h entries (h chosen to give 2K
// heads in all) bound the K-th largest entry from below, and only the few entries above that
// bound need ranking.
__global__ void __launch_bounds__(TK_MERGE_THREADS)
topk_merge_kernel(const float* __restrict__ ref, int64_t n, int64_t ld, const int32_t* __restrict__ topk,
                  int K, int nslices, const float* __restrict__ lists, const int32_t* __restrict__ flags,
                  double* __restrict__ dist_out, int32_t* __restrict__ status)
{
    __shared__ float all[MERGE_CAP + MAX_K];
    __shared__ float heads[2 * MAX_K + IMM_LDD_MAX_N / TK_SLICE];
    __shared__ float top[MAX_K], inside[MAX_K];
    __shared__ double top_d[MAX_K], inside_d[MAX_K];       // converted once: float -> double conversions are slow
    __shared__ double cost[2 * MAX_K];
    __shared__ float bound;
    __shared__ int bad, count;
    const int64_t step = blockIdx.x;
    const int tid = threadIdx.x;
    const float* row = ref + step * ld;
    const int32_t* I = topk + step * K;
    const float* mine = lists + step * nslices * K;
    const int m = nslices * K;                             // <= MERGE_CAP (checked on the host)
    if (tid == 0) { bad = 0; count = 0; }
    if (tid < K) {
        const int64_t idx = I[tid];
        inside[tid] = (idx >= 0 && idx < n) ? row[idx] : 0.f;
    }
    const int h = min(K, (2 * K + nslices - 1) / nslices), nh = nslices * h;
    for (int i = tid; i < nh; i += TK_MERGE_THREADS) heads[i] = mine[(i / h) * K + i % h];
    __syncthreads();
    for (int i = tid; i < nslices; i += TK_MERGE_THREADS) {
        const int f = flags[step * nslices + i];
        if (f) atomicOr(&bad, f);
    }
    for (int i = tid; i < nh; i += TK_MERGE_THREADS)
        if (rank_desc(heads, nh, i) == K - 1) bound = heads[i];    // K entries outside I are at or above it
    __syncthreads();
    const float t0 = bound;
    for (int i = tid; i < m; i += TK_MERGE_THREADS) {
        const float v = mine[i];
        if (v > t0) all[atomicAdd(&count, 1)] = v;
    }
    __syncthreads();
    const int cnt = count;
    for (int i = tid; i < K; i += TK_MERGE_THREADS) all[cnt + i] = t0;
    __syncthreads();
    for (int i = tid; i < cnt + K; i += TK_MERGE_THREADS) {
        const int r = rank_desc(all, cnt + K, i);
        if (r < K) top[r] = all[i];
    }
    __syncthreads();
    if (tid < K) { top_d[tid] = (double)top[tid]; inside_d[tid] = (double)inside[tid]; }
    __syncthreads();
    if (tid < 2 * K) {
        const double t = tid < K ? top_d[tid] : inside_d[tid - K];
        double c = INFINITY;
        if (t > -INFINITY) {                               // a row with fewer than K entries outside I pads with -inf
            c = 0.0;
            for (int k = 0; k < K; k++) {
                c += fmax(top_d[k] - t, 0.0);
                c += fmax(t - inside_d[k], 0.0);
            }
        }
        cost[tid] = c;
    }
    __syncthreads();
    if (tid < 32) {
        double best_cost = INFINITY;
        for (int i = tid; i < 2 * K; i += 32) best_cost = fmin(best_cost, cost[i]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) best_cost = fmin(best_cost, __shfl_xor_sync(0xFFFFFFFFu, best_cost, o));
        if (tid == 0) {
            const bool bad_index = (bad & 1) != 0, gave_up = (bad & 2) != 0;
            dist_out[step] = (bad_index || gave_up) ? NAN : best_cost;
            status[step] = bad_index ? IMM_ERR_ARG : gave_up ? IMM_ERR_LIMIT : IMM_OK;
        }
    }
}

// ------------------------------------------------------------------------------------------
// short rows: one warp per row
// ------------------------------------------------------------------------------------------
// Expert routing (n = 64...256 logits per decision, K = 2...8) has millions of short rows: a
// cluster per row would spend its time on launch and barriers.  Up to SMALL_N entries a warp
// takes a whole row: lane l holds entries l, l + 32, ... in registers, everything else is warp
// shuffles.  The same arithmetic as the long-row kernels (float32 terms, float64 final sums and
// costs), so the same tolerances hold.

constexpr int SMALL_N = 1024;
constexpr int SMALL_WARPS = 8;                // rows per block

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
    return v;
}
__device__ __forceinline__ float warp_add(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

template <int SLOTS>
__global__ void __launch_bounds__(SMALL_WARPS * 32)
tv_kl_small_kernel(const float* __restrict__ logits, const float* __restrict__ ref, int64_t steps, int n, int64_t ld,
                   double* __restrict__ tv_out, double* __restrict__ kl_out)
{
    const int lane = threadIdx.x & 31;
    const int64_t step = (int64_t)blockIdx.x * SMALL_WARPS + (threadIdx.x >> 5);
    if (step >= steps) return;                         // (whole warp)
    const float* x = logits + step * ld;
    const float* y = ref + step * ld;
    float xs[SLOTS], ys[SLOTS];
    float mx = NEG_INF, my = NEG_INF;
#pragma unroll
    for (int j = 0; j < SLOTS; j++) {
        const int e = lane + 32 * j;
        xs[j] = e < n ? x[e] : NEG_INF;
        ys[j] = e < n ? y[e] : NEG_INF;
        mx = fmaxf(mx, xs[j]); my = fmaxf(my, ys[j]);
    }
    mx = warp_max(mx); my = warp_max(my);
    float sx = 0.f, sy = 0.f;
#pragma unroll
    for (int j = 0; j < SLOTS; j++) {                  // slots past the end hold -inf: they add 0
        sx += ex2((xs[j] - mx) * LOG2E);
        sy += ex2((ys[j] - my) * LOG2E);
    }
    const float lp = log2f(warp_add(sx)), lq = log2f(warp_add(sy));
    const float dl = (lq - lp) * (1.0f / LOG2E);
    float tv = 0.f, kl = 0.f;
#pragma unroll
    for (int j = 0; j < SLOTS; j++) {
        if (lane + 32 * j < n) {
            const float xr = xs[j] - mx, yr = ys[j] - my;
            const float p = ex2(fmaf(xr, LOG2E, -lp)), q = ex2(fmaf(yr, LOG2E, -lq));
            tv += fabsf(p - q);
            if (q > 0.f) kl = fmaf(q, (yr - xr) - dl, kl);       // 0 log 0 = 0
        }
    }
    double dtv = (double)tv, dkl = (double)kl;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        dtv += __shfl_xor_sync(0xFFFFFFFFu, dtv, o);
        dkl += __shfl_xor_sync(0xFFFFFFFFu, dkl, o);
    }
    const bool dead = !(lp > NEG_INF) || !(lq > NEG_INF);      // a row without a finite entry: NaN
    if (lane == 0) { tv_out[step] = dead ? (double)NAN : 0.5 * dtv; kl_out[step] = dead ? (double)NAN : dkl; }
}

// Rows of at most 256 entries: a group of LPR lanes per row (8 or 16 lanes, sixteen entries per
// lane), 32 / LPR rows per warp: the shuffle steps are fewer and serve every row of the warp.
template <int LPR>
__global__ void __launch_bounds__(SMALL_WARPS * 32)
tv_kl_sub_kernel(const float* __restrict__ logits, const float* __restrict__ ref, int64_t steps, int n, int64_t ld,
                 double* __restrict__ tv_out, double* __restrict__ kl_out)
{
    constexpr int RPW = 32 / LPR, SLOTS = 16;
    const int lane = threadIdx.x & 31, g = lane / LPR, gl = lane % LPR;
    const int64_t step = ((int64_t)blockIdx.x * SMALL_WARPS + (threadIdx.x >> 5)) * RPW + g;
    const bool live = step < steps;                    // (lanes of a row past the end idle along)
    const float* x = logits + (live ? step : 0) * ld;
    const float* y = ref + (live ? step : 0) * ld;
    float xs[SLOTS], ys[SLOTS];
    float mx = NEG_INF, my = NEG_INF;
#pragma unroll
    for (int j = 0; j < SLOTS; j++) {
        const int e = gl + LPR * j;
        xs[j] = (live && e < n) ? x[e] : NEG_INF;
        ys[j] = (live && e < n) ? y[e] : NEG_INF;
        mx = fmaxf(mx, xs[j]); my = fmaxf(my, ys[j]);
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) {
        mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, o));
        my = fmaxf(my, __shfl_xor_sync(0xFFFFFFFFu, my, o));
    }
    if (!live) { mx = 0.f; my = 0.f; }                 // (keeps the idle lanes' arithmetic finite)
    float sx = 0.f, sy = 0.f;
#pragma unroll
    for (int j = 0; j < SLOTS; j++) {                  // slots past the end hold -inf: they add 0
        sx += ex2((xs[j] - mx) * LOG2E);
        sy += ex2((ys[j] - my) * LOG2E);
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) {
        sx += __shfl_xor_sync(0xFFFFFFFFu, sx, o);
        sy += __shfl_xor_sync(0xFFFFFFFFu, sy, o);
    }
    const float lp = log2f(sx), lq = log2f(sy);
    const float dl = (lq - lp) * (1.0f / LOG2E);
    float tv = 0.f, kl = 0.f;
#pragma unroll
    for (int j = 0; j < SLOTS; j++) {
        if (live && gl + LPR * j < n) {
            const float xr = xs[j] - mx, yr = ys[j] - my;
            const float p = ex2(fmaf(xr, LOG2E, -lp)), q = ex2(fmaf(yr, LOG2E, -lq));
            tv += fabsf(p - q);
            if (q > 0.f) kl = fmaf(q, (yr - xr) - dl, kl);       // 0 log 0 = 0
        }
    }
    double dtv = (double)tv, dkl = (double)kl;
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) {
        dtv += __shfl_xor_sync(0xFFFFFFFFu, dtv, o);
        dkl += __shfl_xor_sync(0xFFFFFFFFu, dkl, o);
    }
    const bool dead = !(lp > NEG_INF) || !(lq > NEG_INF);      // a row without a finite entry: NaN
    if (live && gl == 0) { tv_out[step] = dead ? (double)NAN : 0.5 * dtv; kl_out[step] = dead ? (double)NAN : dkl; }
}

// Top-K distance of a short row.  The K largest entries outside I are pulled out one at a time
// (K warp-wide arg-max rounds over the registers); the cost is then evaluated at the 2K
// breakpoints in float64, as in the long-row kernel.
template <int SLOTS>
__global__ void __launch_bounds__(SMALL_WARPS * 32)
topk_small_kernel(const float* __restrict__ ref, int64_t steps, int n, int64_t ld, const int32_t* __restrict__ topk, int K,
                  double* __restrict__ dist_out, int32_t* __restrict__ status)
{
    __shared__ double outside[SMALL_WARPS][MAX_K], inside[SMALL_WARPS][MAX_K];   // as doubles: converted once
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t step = (int64_t)blockIdx.x * SMALL_WARPS + w;
    if (step >= steps) return;                         // (whole warp)
    const float* y = ref + step * ld;
    const int32_t* I = topk + step * K;
    float v[SLOTS];
#pragma unroll
    for (int j = 0; j < SLOTS; j++) {
        const int e = lane + 32 * j;
        v[j] = e < n ? y[e] : NEG_INF;
    }
    // the entries of I: remember their values, then take them out of the running
    bool bad = false;
    uint32_t mine = 0;                                 // bit j: this lane's slot j belongs to I
    for (int k = 0; k < K; k++) {
        const int idx = I[k];
        if (idx < 0 || idx >= n) { bad = true; continue; }
        if ((idx & 31) == lane) {
            const uint32_t bit = 1u << (idx >> 5);
            if (mine & bit) bad = true;                // the same index twice
            mine |= bit;
        }
    }
    bad = __any_sync(0xFFFFFFFFu, bad);
    for (int k = lane; k < K; k += 32) {
        const int idx = I[k];
        inside[w][k] = (idx >= 0 && idx < n) ? (double)y[idx] : 0.0;
    }
#pragma unroll
    for (int j = 0; j < SLOTS; j++) if ((mine >> j) & 1u) v[j] = NEG_INF;
    for (int r = 0; r < K; r++) {
        float best = NEG_INF;
        int slot = 0;
#pragma unroll
        for (int j = 0; j < SLOTS; j++) if (v[j] > best) { best = v[j]; slot = j; }
        const float top = warp_max(best);
        const unsigned holders = __ballot_sync(0xFFFFFFFFu, best == top);
        const int winner = __ffs(holders) - 1;         // lowest lane holding the maximum
        if (lane == winner) {
            outside[w][r] = (double)top;               // (-inf once fewer than K entries are left outside I)
#pragma unroll
            for (int j = 0; j < SLOTS; j++) if (j == slot) v[j] = NEG_INF;
        }
    }
    __syncwarp();
    double best_cost = INFINITY;
    for (int cnd = lane; cnd < 2 * K; cnd += 32) {
        const double t = cnd < K ? outside[w][cnd] : inside[w][cnd - K];
        if (t > -INFINITY) {
            double c = 0.0;
            for (int k = 0; k < K; k++) {
                c += fmax(outside[w][k] - t, 0.0);
                c += fmax(t - inside[w][k], 0.0);
            }
            best_cost = fmin(best_cost, c);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best_cost = fmin(best_cost, __shfl_xor_sync(0xFFFFFFFFu, best_cost, o));
    if (lane == 0) {
        dist_out[step] = bad ? NAN : best_cost;
        status[step] = bad ? IMM_ERR_ARG : IMM_OK;
    }
}

// slots per lane a row of n entries needs, rounded to the instantiated sizes
inline int small_slots(int64_t n) { return n <= 128 ? 4 : n <= 256 ? 8 : n <= 512 ? 16 : 32; }

// Rows of at most 256 entries with a small K: a group of LPR lanes per row (LPR = 8 or 16, sixteen
// entries per lane), so a warp works on 32 / LPR rows at once and every shuffle, ballot and compare
// instruction serves all of them.  Same selection as topk_small_kernel: K rounds of a group-wide
// arg-max over the entries outside I, then the cost at the 2K breakpoints in float64.
constexpr int SUB_SLOTS = 16;
constexpr int SUB_MAX_K = 16;

template <int LPR>
__global__ void __launch_bounds__(SMALL_WARPS * 32)
topk_sub_kernel(const float* __restrict__ ref, int64_t steps, int n, int64_t ld, const int32_t* __restrict__ topk, int K,
                double* __restrict__ dist_out, int32_t* __restrict__ status)
{
    constexpr int RPW = 32 / LPR;                          // rows per warp
    __shared__ double outside[SMALL_WARPS][RPW][SUB_MAX_K], inside[SMALL_WARPS][RPW][SUB_MAX_K];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int g = lane / LPR, gl = lane % LPR;             // the row of this lane within the warp, its lane within the row
    const unsigned gmask = (LPR == 32 ? 0xFFFFFFFFu : ((1u << LPR) - 1u)) << (g * LPR);
    const int64_t step = ((int64_t)blockIdx.x * SMALL_WARPS + w) * RPW + g;
    const bool live = step < steps;                        // (lanes of a row past the end idle along: the shuffles are warp-wide)
    const float* y = ref + (live ? step : 0) * ld;
    const int32_t* I = topk + (live ? step : 0) * K;
    float v[SUB_SLOTS];
#pragma unroll
    for (int j = 0; j < SUB_SLOTS; j++) {
        const int e = gl + LPR * j;
        v[j] = (live && e < n) ? y[e] : NEG_INF;
    }
    bool bad = false;
    uint32_t mine = 0;                                     // bit j: this lane's slot j belongs to I
    for (int k = 0; k < K; k++) {
        const int idx = live ? I[k] : 0;
        if (idx < 0 || idx >= n) { bad = true; continue; }
        if (idx % LPR == gl) {
            const uint32_t bit = 1u << (idx / LPR);
            if (mine & bit) bad = true;                    // the same index twice
            mine |= bit;
        }
    }
    bad = (__ballot_sync(0xFFFFFFFFu, bad) & gmask) != 0;
    if (live)
        for (int k = gl; k < K; k += LPR) {
            const int idx = I[k];
            inside[w][g][k] = (idx >= 0 && idx < n) ? (double)y[idx] : 0.0;
        }
#pragma unroll
    for (int j = 0; j < SUB_SLOTS; j++) if ((mine >> j) & 1u) v[j] = NEG_INF;
    // every lane sorts its sixteen entries once (bitonic network in registers, descending); a round then
    // compares the lanes' heads only, and the winner moves its list up by one
#pragma unroll
    for (int k = 2; k <= SUB_SLOTS; k <<= 1)
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1)
#pragma unroll
            for (int i = 0; i < SUB_SLOTS; i++) {
                const int l = i ^ j;
                if (l > i) {
                    const float hi = fmaxf(v[i], v[l]), lo = fminf(v[i], v[l]);
                    const bool desc = (i & k) == 0;
                    v[i] = desc ? hi : lo;
                    v[l] = desc ? lo : hi;
                }
            }
    for (int r = 0; r < K; r++) {
        float top = v[0];
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) top = fmaxf(top, __shfl_xor_sync(0xFFFFFFFFu, top, o));
        const unsigned holders = __ballot_sync(0xFFFFFFFFu, v[0] == top) & gmask;
        const int winner = __ffs(holders) - 1;             // lowest lane of the row holding its maximum
        if (lane == winner) {
            outside[w][g][r] = (double)top;                // (-inf once fewer than K entries are left outside I)
#pragma unroll
            for (int j = 0; j + 1 < SUB_SLOTS; j++) v[j] = v[j + 1];
            v[SUB_SLOTS - 1] = NEG_INF;
        }
    }
    __syncwarp();
    double best_cost = INFINITY;
    for (int cnd = gl; cnd < 2 * K; cnd += LPR) {
        const double t = cnd < K ? outside[w][g][cnd] : inside[w][g][cnd - K];
        if (t > -INFINITY) {
            double c = 0.0;
            for (int k = 0; k < K; k++) {
                c += fmax(outside[w][g][k] - t, 0.0);
                c += fmax(t - inside[w][g][k], 0.0);
            }
            best_cost = fmin(best_cost, c);
        }
    }
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) best_cost = fmin(best_cost, __shfl_xor_sync(0xFFFFFFFFu, best_cost, o));
    if (live && gl == 0) {
        dist_out[step] = bad ? NAN : best_cost;
        status[step] = bad ? IMM_ERR_ARG : IMM_OK;
    }
}

// ------------------------------------------------------------------------------------------
// per-request tail statistic
// ------------------------------------------------------------------------------------------
// p[r] = |{ steps of request r with distance > t1 }| / (steps of request r);  flag[r] = p[r] > t2.
// A step counts unless its distance is known to be <= t1: a NaN distance (a malformed index set, a
// row without a finite logit) counts as exceeding the threshold, so it can never lower p.

__global__ void __launch_bounds__(256)
tail_fraction_kernel(const double* __restrict__ dist, const int64_t* __restrict__ offsets, double t1, double t2,
                     double* __restrict__ p_out, int32_t* __restrict__ flag_out)
{
    __shared__ int warp_cnt[8];
    const int64_t r = blockIdx.x;
    const int64_t b = offsets[r], e = offsets[r + 1];
    int cnt = 0;
    for (int64_t i = b + threadIdx.x; i < e; i += blockDim.x) cnt += !(dist[i] <= t1) ? 1 : 0;
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
    cudaStream_t st = (cudaStream_t)stream;
    if (n <= 256) {                                    // very short rows: several rows per warp
        if (n <= 128) {
            const unsigned g2 = (unsigned)((steps + SMALL_WARPS * 4 - 1) / (SMALL_WARPS * 4));
            tv_kl_sub_kernel<8><<<g2, SMALL_WARPS * 32, 0, st>>>(d_logits, d_ref_logits, steps, (int)n, ld, d_tv, d_kl);
        } else {
            const unsigned g2 = (unsigned)((steps + SMALL_WARPS * 2 - 1) / (SMALL_WARPS * 2));
            tv_kl_sub_kernel<16><<<g2, SMALL_WARPS * 32, 0, st>>>(d_logits, d_ref_logits, steps, (int)n, ld, d_tv, d_kl);
        }
        return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
    }
    if (n <= SMALL_N) {                                // short rows: one warp per row
        const unsigned grid = (unsigned)((steps + SMALL_WARPS - 1) / SMALL_WARPS);
        switch (small_slots(n)) {
        case 4: tv_kl_small_kernel<4><<<grid, SMALL_WARPS * 32, 0, st>>>(d_logits, d_ref_logits, steps, (int)n, ld, d_tv, d_kl); break;
        case 8: tv_kl_small_kernel<8><<<grid, SMALL_WARPS * 32, 0, st>>>(d_logits, d_ref_logits, steps, (int)n, ld, d_tv, d_kl); break;
        case 16: tv_kl_small_kernel<16><<<grid, SMALL_WARPS * 32, 0, st>>>(d_logits, d_ref_logits, steps, (int)n, ld, d_tv, d_kl); break;
        default: tv_kl_small_kernel<32><<<grid, SMALL_WARPS * 32, 0, st>>>(d_logits, d_ref_logits, steps, (int)n, ld, d_tv, d_kl); break;
        }
        return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
    }
    const int nc = cluster_size(n);
    const bool vec = rows_aligned(d_logits, ld) && rows_aligned(d_ref_logits, ld);
    // 512 threads and clusters of up to 8 blocks measured best (256 / 1024 threads and 16-block clusters were tried)
    cudaError_t e = vec ? launch_cluster(tv_kl_kernel<true, THREADS>, steps, nc, THREADS, 0, st, d_logits, d_ref_logits, n, ld, d_tv, d_kl)
                        : launch_cluster(tv_kl_kernel<false, THREADS>, steps, nc, THREADS, 0, st, d_logits, d_ref_logits, n, ld, d_tv, d_kl);
    return e == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
}

size_t imm_ldd_topk_workspace(int64_t steps, int64_t n, int k)
{
    using namespace imm_ldd;
    if (steps < 0 || n <= 0 || n > IMM_LDD_MAX_N || steps > IMM_LDD_MAX_STEPS || k <= 0 || k > IMM_LDD_MAX_K) return 0;
    const int64_t nslices = (n + TK_SLICE - 1) / TK_SLICE;
    // one flag word per slice, then every slice's K largest entries
    return (size_t)((steps * nslices * 4 + 255) / 256 * 256) + (size_t)steps * nslices * k * sizeof(float) + 256;
}

int imm_ldd_topk_distance(const float* d_ref_logits, int64_t steps, int64_t n, int64_t ld,
                          const int32_t* d_topk, int k, double* d_dist, int32_t* d_status,
                          void* d_ws, size_t ws_bytes, void* stream)
{
    using namespace imm_ldd;
    if (!d_ref_logits || !d_topk || !d_dist || !d_status || !d_ws) return IMM_ERR_ARG;
    if (steps < 0 || n <= 0 || ld < n || n > IMM_LDD_MAX_N || steps > IMM_LDD_MAX_STEPS) return IMM_ERR_SHAPE;
    if (k <= 0 || k > IMM_LDD_MAX_K || k > n) return IMM_ERR_SHAPE;
    if ((uintptr_t)d_ref_logits % 4 || (uintptr_t)d_topk % 4 || (uintptr_t)d_dist % 8 || (uintptr_t)d_status % 4 ||
        (uintptr_t)d_ws % 16)
        return IMM_ERR_ALIGN;
    if (ws_bytes < imm_ldd_topk_workspace(steps, n, k)) return IMM_ERR_WORKSPACE;
    if (steps == 0) return IMM_OK;
    if (n <= SMALL_N) {                                // short rows: one warp per row, no workspace traffic
        const unsigned grid = (unsigned)((steps + SMALL_WARPS - 1) / SMALL_WARPS);
        cudaStream_t sst = (cudaStream_t)stream;
        if (n <= 16 * SUB_SLOTS && k <= SUB_MAX_K) {       // very short rows: several rows per warp
            if (n <= 8 * SUB_SLOTS) {
                const unsigned g2 = (unsigned)((steps + SMALL_WARPS * 4 - 1) / (SMALL_WARPS * 4));
                topk_sub_kernel<8><<<g2, SMALL_WARPS * 32, 0, sst>>>(d_ref_logits, steps, (int)n, ld, d_topk, k, d_dist, d_status);
            } else {
                const unsigned g2 = (unsigned)((steps + SMALL_WARPS * 2 - 1) / (SMALL_WARPS * 2));
                topk_sub_kernel<16><<<g2, SMALL_WARPS * 32, 0, sst>>>(d_ref_logits, steps, (int)n, ld, d_topk, k, d_dist, d_status);
            }
            return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
        }
        switch (small_slots(n)) {
        case 4: topk_small_kernel<4><<<grid, SMALL_WARPS * 32, 0, sst>>>(d_ref_logits, steps, (int)n, ld, d_topk, k, d_dist, d_status); break;
        case 8: topk_small_kernel<8><<<grid, SMALL_WARPS * 32, 0, sst>>>(d_ref_logits, steps, (int)n, ld, d_topk, k, d_dist, d_status); break;
        case 16: topk_small_kernel<16><<<grid, SMALL_WARPS * 32, 0, sst>>>(d_ref_logits, steps, (int)n, ld, d_topk, k, d_dist, d_status); break;
        default: topk_small_kernel<32><<<grid, SMALL_WARPS * 32, 0, sst>>>(d_ref_logits, steps, (int)n, ld, d_topk, k, d_dist, d_status); break;
        }
        return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
    }
    const int64_t nslices = (n + TK_SLICE - 1) / TK_SLICE;
    if (nslices * k > MERGE_CAP || steps * nslices > 0x7FFFFFFF) return IMM_ERR_SHAPE;     // (cannot happen within the limits)
    cudaStream_t st = (cudaStream_t)stream;
    int32_t* flags = (int32_t*)d_ws;
    float* lists = (float*)((char*)d_ws + (steps * nslices * 4 + 255) / 256 * 256);
    const bool vec = rows_aligned(d_ref_logits, ld);
    const unsigned grid = (unsigned)(steps * nslices);
    if (vec) topk_slice_kernel<true><<<grid, TK_THREADS, 0, st>>>(d_ref_logits, n, ld, d_topk, k, (int)nslices, lists, flags);
    else topk_slice_kernel<false><<<grid, TK_THREADS, 0, st>>>(d_ref_logits, n, ld, d_topk, k, (int)nslices, lists, flags);
    if (cudaGetLastError() != cudaSuccess) return IMM_ERR_CUDA;
    topk_merge_kernel<<<(unsigned)steps, TK_MERGE_THREADS, 0, st>>>(d_ref_logits, n, ld, d_topk, k, (int)nslices, lists, flags,
                                                                    d_dist, d_status);
    return cudaGetLastError() == cudaSuccess ? IMM_OK : IMM_ERR_CUDA;
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
