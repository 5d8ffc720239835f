// CUDA kernels of libimm (sm_100a): eq tables, eq-vector x matrix contractions mod p, and the
// sumcheck rounds.  Host-side launch wrappers are at the end; the C ABI lives in imm_api.cu.
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <type_traits>

#include <cooperative_groups.h>

#include "gl64.cuh"
#include "imm_kernels.h"
#include "imm_plan.h"
#include "sha256.cuh"

namespace imm {

// ------------------------------------------------------------------------------------------
// small device helpers
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ uint64_t shfl_xor_u64(uint64_t v, int mask)
{
    return __shfl_xor_sync(0xFFFFFFFFu, v, mask);
}

__device__ __forceinline__ uint64_t shfl_idx_u64(uint64_t v, int src_lane)
{
    return __shfl_sync(0xFFFFFFFFu, v, src_lane);
}

__device__ __forceinline__ uint64_t warp_sum_fe(uint64_t v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = gl::add(v, shfl_xor_u64(v, o));
    return v;
}

// Sum of one canonical element per thread over the block; result valid in every thread.
// `scratch` holds one word per warp plus one.
__device__ __forceinline__ uint64_t block_sum_fe(uint64_t v, uint64_t* scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
    v = warp_sum_fe(v);
    __syncthreads();                       // scratch may still be read from a previous call
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (warp == 0) {
        uint64_t t = lane < nwarp ? scratch[lane] : 0;
        t = warp_sum_fe(t);
        if (lane == 0) scratch[32] = t;
    }
    __syncthreads();
    return scratch[32];
}

// 128-bit streaming load (read once: do not keep in L1)
__device__ __forceinline__ uint4 ld_stream_v4(const void* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// sign-extended byte `K` of a 32-bit word: one byte-permute with sign replication
template <int K>
__device__ __forceinline__ int32_t sext_byte(uint32_t w)
{
    int32_t r;
    constexpr uint32_t sel = (uint32_t)K | ((uint32_t)(K | 8) << 4) | ((uint32_t)(K | 8) << 8) |
                             ((uint32_t)(K | 8) << 12);
    asm("prmt.b32 %0, %1, %1, %2;" : "=r"(r) : "r"(w), "n"(sel));
    return r;
}

// acc += x * y  (signed 32 x 32 -> 64 multiply-add)
__device__ __forceinline__ void mad_wide(int64_t& acc, int32_t x, int32_t y)
{
    asm("mad.wide.s32 %0, %1, %2, %0;" : "+l"(acc) : "r"(x), "r"(y));
}

// Find the job a tile belongs to: jobs are ordered by tile0 and jobs[0].tile0 = 0.  The lanes of
// a warp probe 32 evenly spaced jobs at once, so 1024 jobs take two dependent loads instead of
// ten.  Called by whole warps.
__device__ __forceinline__ int find_job(const MatJob* jobs, int njobs, uint32_t tile)
{
    const int lane = threadIdx.x & 31;
    int lo = 0, n = njobs;
    while (n > 1) {
        const int step = (n + 31) >> 5;
        const int idx = lo + lane * step;
        const bool ok = idx < lo + n && jobs[idx].tile0 <= tile;
        const uint32_t mask = __ballot_sync(0xFFFFFFFFu, ok) | 1u;      // the probes that hold form a prefix
        const int k = 31 - __clz(mask);
        const int end = lo + n;
        lo += k * step;
        n = min(step, end - lo);
    }
    return lo;
}

// ------------------------------------------------------------------------------------------
// element-wise field arithmetic (test hook for the device field code)
// ------------------------------------------------------------------------------------------

__global__ void field_binop_kernel(int op, const imm_fe* x, const imm_fe* y, imm_fe* out, int64_t n)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t step = (int64_t)gridDim.x * blockDim.x;
    for (; i < n; i += step) {
        uint64_t a = x[i], b = y[i];
        out[i] = op == 0 ? gl::add(a, b) : op == 1 ? gl::sub(a, b) : gl::mul(a, b);
    }
}

// ------------------------------------------------------------------------------------------
// eq tables
// ------------------------------------------------------------------------------------------
// E[i] = eq(r, i), variable 0 = most significant index bit.  The index is split into a high
// part (variables 0..nhi-1) and a low part (the rest); both small tables are built by doubling
// in shared memory and E[i] = hi[i >> nlo] * lo[i & (2^nlo - 1)].  One block per table.

__device__ void eq_build_small(uint64_t* tbl, const uint64_t* r, int cnt)
{
    if (threadIdx.x == 0) tbl[0] = 1;
    __syncthreads();
    for (int t = 0; t < cnt; t++) {
        const int len = 1 << t;
        uint64_t v = 0;
        const bool act = (int)threadIdx.x < len;
        if (act) v = tbl[threadIdx.x];
        __syncthreads();
        if (act) {
            uint64_t h = gl::mul(v, r[t]);
            tbl[2 * threadIdx.x + 1] = h;
            tbl[2 * threadIdx.x] = gl::sub(v, h);
        }
        __syncthreads();
    }
}

__device__ void eq_fill(imm_fe* out, int nvars, const uint64_t* r_sh, uint64_t* lo_t, uint64_t* hi_t)
{
    const int nlo = (nvars + 1) / 2, nhi = nvars - nlo;
    eq_build_small(hi_t, r_sh, nhi);
    eq_build_small(lo_t, r_sh + nhi, nlo);
    const int64_t total = (int64_t)1 << nvars;
    const uint32_t mask = (1u << nlo) - 1;
    for (int64_t i = threadIdx.x; i < total; i += blockDim.x)
        out[i] = gl::mul(hi_t[i >> nlo], lo_t[(uint32_t)i & mask]);
}

__global__ void __launch_bounds__(1024) eq_direct_kernel(EqDirect rr, int nvars, imm_fe* out)
{
    __shared__ uint64_t r_sh[MAX_EQ_VARS];
    __shared__ uint64_t lo_t[1024], hi_t[1024];
    if ((int)threadIdx.x < nvars) r_sh[threadIdx.x] = rr.r[threadIdx.x];
    __syncthreads();
    eq_fill(out, nvars, r_sh, lo_t, hi_t);
}

// ------------------------------------------------------------------------------------------
// contraction building blocks
// ------------------------------------------------------------------------------------------
// The eq weight e is consumed as two signed 32-bit halves (gl::balanced_halves) and the matrix
// entries as signed 32-bit values, so one entry costs a handful of 32 x 32 -> 64 multiply-adds
// into 64-bit accumulators with NO modular reduction in the loop (lazy accumulation):
//   int8 :  L += e_lo*v, H += e_hi*v                       |term| < 2^38, > 2^24 terms of headroom
//   int32:  v = v_hi*2^16 + v_lo (v_lo unsigned 16 bit):   |term| < 2^47, 2^16 terms of headroom
//           LL += e_lo*v_lo, LH += e_lo*v_hi, HL += e_hi*v_lo, HH += e_hi*v_hi
// The exact integer sum is rebuilt and reduced once per output.

template <typename T> struct Elem;
template <> struct Elem<int8_t>  { static constexpr int EPV = 16; static constexpr int NACC = 2; };
template <> struct Elem<int32_t> { static constexpr int EPV = 4;  static constexpr int NACC = 4; };

// element-wise gather of up to EPV entries into the layout of a 16-byte vector load
template <typename T>
__device__ __forceinline__ uint4 load_elems(const T* p, int nvalid)
{
    union { uint4 v; T e[Elem<T>::EPV]; } u;
    u.v = make_uint4(0, 0, 0, 0);
#pragma unroll
    for (int j = 0; j < Elem<T>::EPV; j++)
        if (j < nvalid) u.e[j] = p[j];
    return u.v;
}

template <typename T, bool VEC>
__device__ __forceinline__ uint4 load_vec(const char* p, bool full, int nvalid)
{
    if (VEC && full) return ld_stream_v4(p);
    return load_elems<T>(reinterpret_cast<const T*>(p), nvalid);
}

template <int K>
__device__ __forceinline__ void mac_word_i8(int64_t* acc /* [4][2] */, uint32_t w, int32_t el, int32_t eh)
{
    int32_t v = sext_byte<K>(w);
    mad_wide(acc[2 * K], el, v);
    mad_wide(acc[2 * K + 1], eh, v);
}

// acc layout int8: [16 columns][2] = (L, H); int32: [4 columns][4] = (LL, LH, HL, HH)
__device__ __forceinline__ void mac_vec(int64_t (&acc)[32], uint4 w, int32_t el, int32_t eh, int8_t)
{
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int q = 0; q < 4; q++) {
        mac_word_i8<0>(&acc[8 * q], ww[q], el, eh);
        mac_word_i8<1>(&acc[8 * q], ww[q], el, eh);
        mac_word_i8<2>(&acc[8 * q], ww[q], el, eh);
        mac_word_i8<3>(&acc[8 * q], ww[q], el, eh);
    }
}

__device__ __forceinline__ void mac_vec(int64_t (&acc)[16], uint4 w, int32_t el, int32_t eh, int32_t)
{
    const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
    for (int q = 0; q < 4; q++) {
        int32_t vlo = (int32_t)(ww[q] & 0xFFFFu);
        int32_t vhi = (int32_t)ww[q] >> 16;
        mad_wide(acc[4 * q + 0], el, vlo);
        mad_wide(acc[4 * q + 1], el, vhi);
        mad_wide(acc[4 * q + 2], eh, vlo);
        mad_wide(acc[4 * q + 3], eh, vhi);
    }
}

// exact integer accumulators of one column -> canonical field element
__device__ __forceinline__ uint64_t finish_col(const int64_t* a, int8_t)
{
    return gl::add(gl::from_i64(a[0]), gl::shl(gl::from_i64(a[1]), 32));
}
__device__ __forceinline__ uint64_t finish_col(const int64_t* a, int32_t)
{
    uint64_t lo = gl::add(gl::from_i64(a[0]), gl::shl(gl::from_i64(a[1]), 16));
    uint64_t hi = gl::add(gl::shl(gl::from_i64(a[2]), 32), gl::shl(gl::from_i64(a[3]), 48));
    return gl::add(lo, hi);
}

// ------------------------------------------------------------------------------------------
// row binding:  out[y] = sum_i eq_row[i] * M[i,y]   (POINT: then dotted with eq_col)
// ------------------------------------------------------------------------------------------
// One tile = tile_rows rows x (ROWBIND_THREADS * EPV) columns.  A thread owns one 16-byte vector
// of columns and walks down the rows; a warp therefore reads 512 contiguous bytes of each row.

template <typename T, bool POINT, bool VEC>
__device__ __forceinline__ void rowbind_tile(const MatJob& job, uint32_t local, int2* sE, uint64_t* red)
{
    constexpr int EPV = Elem<T>::EPV, NACC = Elem<T>::NACC;
    const int rbi = local / job.ncc, cci = local % job.ncc;
    const int r0 = rbi * job.tile_rows;
    const int nrows = min(job.tile_rows, job.rows - r0);
    const int col = (cci * ROWBIND_THREADS + threadIdx.x) * EPV;
    const int nvalid = min(EPV, job.cols - col);          // <= 0: this thread has no columns
    const bool full = nvalid == EPV;

    for (int i = threadIdx.x; i < nrows; i += ROWBIND_THREADS) {
        int32_t lo, hi;
        gl::balanced_halves(job.eq_row[r0 + i], lo, hi);
        sE[i] = make_int2(lo, hi);
    }
    __syncthreads();

    int64_t acc[EPV * NACC];
#pragma unroll
    for (int j = 0; j < EPV * NACC; j++) acc[j] = 0;

    if (nvalid > 0) {
        const int64_t pitch = job.ld * (int64_t)sizeof(T);
        const char* p = (const char*)job.mat + ((int64_t)r0 * job.ld + col) * (int64_t)sizeof(T);
        int i = 0;
        for (; i + 4 <= nrows; i += 4) {
            uint4 w0 = load_vec<T, VEC>(p, full, nvalid);
            uint4 w1 = load_vec<T, VEC>(p + pitch, full, nvalid);
            uint4 w2 = load_vec<T, VEC>(p + 2 * pitch, full, nvalid);
            uint4 w3 = load_vec<T, VEC>(p + 3 * pitch, full, nvalid);
            p += 4 * pitch;
            int2 e0 = sE[i], e1 = sE[i + 1], e2 = sE[i + 2], e3 = sE[i + 3];
            mac_vec(acc, w0, e0.x, e0.y, T());
            mac_vec(acc, w1, e1.x, e1.y, T());
            mac_vec(acc, w2, e2.x, e2.y, T());
            mac_vec(acc, w3, e3.x, e3.y, T());
        }
        for (; i < nrows; i++) {
            uint4 w0 = load_vec<T, VEC>(p, full, nvalid);
            p += pitch;
            int2 e0 = sE[i];
            mac_vec(acc, w0, e0.x, e0.y, T());
        }
    }

    if (!POINT) {
        if (nvalid > 0) {
            imm_fe* o = job.out + (int64_t)rbi * job.cols + col;
#pragma unroll
            for (int j = 0; j < EPV; j++)
                if (j < nvalid) o[j] = finish_col(&acc[NACC * j], T());
        }
    } else {
        uint64_t part = 0;
        if (nvalid > 0) {
#pragma unroll
            for (int j = 0; j < EPV; j++)
                if (j < nvalid)
                    part = gl::add(part, gl::mul(finish_col(&acc[NACC * j], T()), job.eq_col[col + j]));
        }
        part = block_sum_fe(part, red);
        if (threadIdx.x == 0) job.out[local] = part;
    }
}

template <typename T, bool POINT>
__global__ void __launch_bounds__(ROWBIND_THREADS) rowbind_kernel(const MatJob* jobs, int njobs)
{
    __shared__ int2 sE[MAX_TILE_ROWS];
    __shared__ uint64_t red[33];
    const MatJob job = jobs[find_job(jobs, njobs, blockIdx.x)];
    const uint32_t local = blockIdx.x - job.tile0;
    if (job.vec) rowbind_tile<T, POINT, true>(job, local, sE, red);
    else rowbind_tile<T, POINT, false>(job, local, sE, red);
}

// ------------------------------------------------------------------------------------------
// column binding:  out[i] = sum_j M[i,j] * eq_col[j]
// ------------------------------------------------------------------------------------------
// One tile = tile_rows rows x one chunk of COLBIND_VECS vectors of columns.  The chunk's eq
// weights sit in shared memory as balanced halves, laid out [pair of columns][vector] so that a
// warp's 16-byte reads are conflict-free.  A warp takes COLBIND_ROWS_PER_WARP rows at a time:
// each lane loads the weights of its vector once and applies them to all those rows, then the
// per-row integer sums are combined across the warp with shuffles.

template <typename T, bool VEC>
__device__ __forceinline__ void colbind_tile(const MatJob& job, uint32_t local, int4* sE)
{
    constexpr int EPV = Elem<T>::EPV, NACC = Elem<T>::NACC, RW = COLBIND_ROWS_PER_WARP;
    constexpr int PAIRS = EPV / 2;
    const int rbi = local / job.ncc, cci = local % job.ncc;
    const int r0 = rbi * job.tile_rows;
    const int r1 = min(r0 + job.tile_rows, job.rows);
    const int c0 = cci * COLBIND_VECS * EPV;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int NWARP = COLBIND_THREADS / 32;

    // stage the chunk's weights: sE[pair * COLBIND_VECS + vec] = (lo0, hi0, lo1, hi1)
    for (int t = threadIdx.x; t < COLBIND_VECS * PAIRS; t += COLBIND_THREADS) {
        const int vec = t / PAIRS, pair = t % PAIRS;
        const int col = c0 + vec * EPV + 2 * pair;
        int32_t l0 = 0, h0 = 0, l1 = 0, h1 = 0;
        if (col < job.cols) gl::balanced_halves(job.eq_col[col], l0, h0);
        if (col + 1 < job.cols) gl::balanced_halves(job.eq_col[col + 1], l1, h1);
        sE[pair * COLBIND_VECS + vec] = make_int4(l0, h0, l1, h1);
    }
    __syncthreads();

    const int64_t pitch = job.ld * (int64_t)sizeof(T);
    for (int r = r0 + warp * RW; r < r1; r += NWARP * RW) {
        int64_t acc[RW][NACC];
#pragma unroll
        for (int u = 0; u < RW; u++)
#pragma unroll
            for (int a = 0; a < NACC; a++) acc[u][a] = 0;

        for (int vec = lane; vec < COLBIND_VECS; vec += 32) {
            const int col = c0 + vec * EPV;
            const int nvalid = min(EPV, job.cols - col);
            if (nvalid <= 0) break;
            const bool full = nvalid == EPV;
            const char* p = (const char*)job.mat + ((int64_t)r * job.ld + col) * (int64_t)sizeof(T);
            uint4 w[RW];
#pragma unroll
            for (int u = 0; u < RW; u++)
                w[u] = (r + u < r1) ? load_vec<T, VEC>(p + u * pitch, full, nvalid) : make_uint4(0, 0, 0, 0);
            int4 e[PAIRS];
#pragma unroll
            for (int q = 0; q < PAIRS; q++) e[q] = sE[q * COLBIND_VECS + vec];
#pragma unroll
            for (int u = 0; u < RW; u++) {
                const uint32_t ww[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
                if constexpr (sizeof(T) == 1) {
#pragma unroll
                    for (int q = 0; q < 4; q++) {          // word q holds columns 4q..4q+3
                        const int4 ea = e[2 * q], eb = e[2 * q + 1];
                        int32_t v0 = sext_byte<0>(ww[q]), v1 = sext_byte<1>(ww[q]);
                        int32_t v2 = sext_byte<2>(ww[q]), v3 = sext_byte<3>(ww[q]);
                        mad_wide(acc[u][0], ea.x, v0); mad_wide(acc[u][1], ea.y, v0);
                        mad_wide(acc[u][0], ea.z, v1); mad_wide(acc[u][1], ea.w, v1);
                        mad_wide(acc[u][0], eb.x, v2); mad_wide(acc[u][1], eb.y, v2);
                        mad_wide(acc[u][0], eb.z, v3); mad_wide(acc[u][1], eb.w, v3);
                    }
                } else {
#pragma unroll
                    for (int q = 0; q < 4; q++) {          // word q is column q
                        const int4 ee = e[q / 2];
                        const int32_t el = (q & 1) ? ee.z : ee.x, eh = (q & 1) ? ee.w : ee.y;
                        int32_t vlo = (int32_t)(ww[q] & 0xFFFFu), vhi = (int32_t)ww[q] >> 16;
                        mad_wide(acc[u][0], el, vlo);
                        mad_wide(acc[u][1], el, vhi);
                        mad_wide(acc[u][2], eh, vlo);
                        mad_wide(acc[u][3], eh, vhi);
                    }
                }
            }
        }
        // combine across the warp; per-lane sums stay far below 2^63 (see headroom above)
#pragma unroll
        for (int u = 0; u < RW; u++)
#pragma unroll
            for (int a = 0; a < NACC; a++) {
                int64_t v = acc[u][a];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += (int64_t)shfl_xor_u64((uint64_t)v, o);
                acc[u][a] = v;
            }
        if (lane < RW && r + lane < r1) {
            int64_t mine[NACC] = {};
#pragma unroll
            for (int u = 0; u < RW; u++)
                if (u == lane)
#pragma unroll
                    for (int a = 0; a < NACC; a++) mine[a] = acc[u][a];
            job.out[(int64_t)cci * job.rows + r + lane] = finish_col(mine, T());
        }
    }
}

template <typename T>
__global__ void __launch_bounds__(COLBIND_THREADS) colbind_kernel(const MatJob* jobs, int njobs)
{
    __shared__ int4 sE[COLBIND_VECS * (Elem<T>::EPV / 2)];
    const MatJob job = jobs[find_job(jobs, njobs, blockIdx.x)];
    const uint32_t local = blockIdx.x - job.tile0;
    if (job.vec) colbind_tile<T, true>(job, local, sE);
    else colbind_tile<T, false>(job, local, sE);
}

}  // namespace imm

#include "imm_mma.cuh"

namespace imm {

// ------------------------------------------------------------------------------------------
// sum of partial vectors:  out[y] = sum_p parts[p][y]
// ------------------------------------------------------------------------------------------

__global__ void sum_parts_kernel(const imm_fe* parts, int nparts, int64_t len, imm_fe* out)
{
    int64_t y = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (y >= len) return;
    uint64_t s = 0;
    for (int p = 0; p < nparts; p++) s = gl::add(s, parts[(int64_t)p * len + y]);
    out[y] = s;
}

// out[0] = sum of `count` elements (single block)
__global__ void __launch_bounds__(1024) sum_all_kernel(const imm_fe* parts, int64_t count, imm_fe* out)
{
    __shared__ uint64_t red[33];
    uint64_t s = 0;
    for (int64_t i = threadIdx.x; i < count; i += blockDim.x) s = gl::add(s, parts[i]);
    s = block_sum_fe(s, red);
    if (threadIdx.x == 0) out[0] = s;
}

// out[0] = sum of `count` partial sums of a tensor-core point evaluation.  For an int32 matrix the
// kernel summed unsigned bytes, so every entry reads 2^31 too high: 2^31 * (sum of the row weights)
// * (sum of the column weights) comes off (nsr = 0: no offset).
__global__ void __launch_bounds__(1024)
point_finish_kernel(const imm_fe* parts, int64_t count, const imm_fe* sum_row, int nsr, const imm_fe* sum_col,
                    int nsc, imm_fe* out)
{
    __shared__ uint64_t red[33];
    uint64_t s = 0;
    for (int64_t i = threadIdx.x; i < count; i += blockDim.x) s = gl::add(s, parts[i]);
    s = block_sum_fe(s, red);
    if (threadIdx.x == 0) {
        if (nsr > 0) {
            uint64_t sr = 0, sc = 0;
            for (int i = 0; i < nsr; i++) sr = gl::add(sr, sum_row[i]);
            for (int i = 0; i < nsc; i++) sc = gl::add(sc, sum_col[i]);
            s = gl::sub(s, gl::shl(gl::mul(sr, sc), 31));
        }
        out[0] = s;
    }
}

// ------------------------------------------------------------------------------------------
// sumcheck rounds: one thread-block cluster per proof
// ------------------------------------------------------------------------------------------
// Round j works on tables a[], b[] of 2h entries (h = 2^(b-1-j)) and sends
//   g(0) = sum_{y<h} a[y] b[y],  g(1) = sum a[y+h] b[y+h],  g(2) = sum (2a[y+h]-a[y]) (2b[y+h]-b[y]),
// then folds a[y] <- a[y] + r_j (a[y+h] - a[y]) (same for b).
//
// Three facts shape the kernel.  (1) Challenges are public coins, so nothing waits for a round
// polynomial: a pass folds with r_j AND accumulates round j+1's three sums from the values it
// has just produced (four lanes fold the two pairs that form one pair of the next round, one value
// each, and share them by shuffle), and the partial sums of every round are reduced once, after
// the last round, not once per round: a round costs one barrier.  (2) Rounds bind the index from its top bit down, so the first
// J = b - 8 rounds never mix entries whose low 8 index bits differ: block c of the cluster owns
// the entries whose low bits fall in its slice of 256 / (cluster size) values, runs those J
// rounds on its own shared-memory tables, and stores its slice of the 256-entry folded tables
// plus its partial sums into block 0's shared memory (one cluster barrier); block 0 runs the last
// 8 rounds.  (3) Field addition is exact, so the order of these reductions does not change a word.
// The cluster size is chosen per launch: small batches spread each proof over 8 SMs, large ones
// keep one or two blocks per proof so that all proofs run at once.  Proofs of at most
// SC_SOLO_VARS rounds are done by block 0 alone.

constexpr int SC_WARPS = SUMCHECK_THREADS / 32;
constexpr int SC_FINAL_VARS = 8;                 // rounds left to block 0 in a distributed proof
constexpr int SC_FINAL = 1 << SC_FINAL_VARS;
constexpr int SC_SOLO_VARS = 10;
constexpr int SC_MAX_CAP = 8192;                 // entries per shared-memory table (2 x 64 KiB)
constexpr int SC_PORTABLE_CLUSTER = 8;           // larger clusters need an opt-in and are used for k > 2^16 only

struct Sums3 { uint64_t g0, g1, g2; };

__device__ __forceinline__ void sums_add(Sums3& s, uint64_t a0, uint64_t a1, uint64_t b0, uint64_t b1)
{
    s.g0 = gl::add(s.g0, gl::mul(a0, b0));
    s.g1 = gl::add(s.g1, gl::mul(a1, b1));
    uint64_t a2 = gl::sub(gl::add(a1, a1), a0), b2 = gl::sub(gl::add(b1, b1), b0);
    s.g2 = gl::add(s.g2, gl::mul(a2, b2));
}

__device__ __forceinline__ uint64_t fold1(uint64_t lo, uint64_t hi, uint64_t r)
{
    return gl::add(lo, gl::mul(r, gl::sub(hi, lo)));
}

// sum_p parts[p][y]: the loads of eight partial vectors are issued together (the chain is bound by
// memory latency, not by the additions).
// (Loads go to L2, not through the read-only path: the kernel that wrote the partials may still have
// been running when this one was launched, see imm_fused.cuh.)
__device__ __forceinline__ uint64_t sum_parts_at(const imm_fe* parts, int nparts, int len, int y)
{
    const imm_fe* src = parts + y;
    uint64_t s = 0;
    int p = 0;
    for (; p + 8 <= nparts; p += 8) {
        uint64_t v[8];
#pragma unroll
        for (int pp = 0; pp < 8; pp++) v[pp] = __ldcg(src + (int64_t)(p + pp) * len);
#pragma unroll
        for (int pp = 0; pp < 8; pp++) s = gl::add(s, v[pp]);
    }
    if (p < nparts) {
        uint64_t v[8];
#pragma unroll
        for (int pp = 0; pp < 8; pp++) v[pp] = p + pp < nparts ? __ldcg(src + (int64_t)(p + pp) * len) : 0;
#pragma unroll
        for (int pp = 0; pp < 8; pp++) s = gl::add(s, v[pp]);
    }
    return s;
}

}  // namespace imm

#include "imm_fused.cuh"

namespace imm {

// 2^31 * (sum of E_row over the real rows) * (sum of E_col over the real columns): what the claim
// kernel's unsigned view of the int32 entries adds to the sum of its partial results.  The two sums
// come from the eq kernel's slice sums where those exist, else from the challenges in closed form.
// Block-wide call; `red` holds 33 words plus two; valid in every thread.
__device__ __forceinline__ uint64_t claim_offset_block(const ProofDev& pr, uint64_t* red)
{
    if (!pr.c_offset) return 0;
    if (pr.sum_row == nullptr) return gl::shl(offset_sums_closed_form(pr, red + 33), 31);
    uint64_t sr = 0, sc = 0;
    for (int i = threadIdx.x; i < pr.n_sum_row; i += blockDim.x) sr = gl::add(sr, pr.sum_row[i]);
    for (int i = threadIdx.x; i < pr.n_sum_col; i += blockDim.x) sc = gl::add(sc, pr.sum_col[i]);
    sr = block_sum_fe(sr, red);
    sc = block_sum_fe(sc, red);
    return gl::shl(gl::mul(sr, sc), 31);
}

struct ScShared {
    uint64_t r[MAX_K_VARS];                    // round challenges
    uint64_t warp_sums[MAX_K_VARS][SC_WARPS][3];   // sums of a round whose pass ran on several warps
    uint64_t lane_sums[MAX_K_VARS][32][3];     // sums of a round whose pass ran on warp 0 alone (not yet reduced)
    uint64_t block_sums[MAX_K_VARS][3];        // sums of the rounds a block ran alone
    uint64_t gather[SUMCHECK_MAX_CLUSTER][MAX_K_VARS * 3];   // block 0: every block's share of the local rounds' sums
    uint64_t fin[2][SC_FINAL];                 // block 0: the 256-entry tables, written by their owners
    uint64_t red[SC_WARPS];
};

// dst[3 j + comp] = all stashed sums of round j, for j in [j0, j1); one warp per round.  Callers
// put a block barrier before (stashes visible) and a barrier after (results visible); dst may lie in
// another block of the cluster.  (Not inlined, like run_rounds: the kernel is short enough for cold
// instruction fetches to show, so both stages of a proof share one copy of the code.)
__device__ __noinline__ void reduce_round_sums(ScShared& sh, int j0, int j1, uint64_t* dst)
{
    const int lane = threadIdx.x & 31;
    for (int j = j0 + (threadIdx.x >> 5); j < j1; j += SC_WARPS) {
#pragma unroll
        for (int comp = 0; comp < 3; comp++) {
            uint64_t v = sh.lane_sums[j][lane][comp];
            if (lane < SC_WARPS) v = gl::add(v, sh.warp_sums[j][lane][comp]);
            v = warp_sum_fe(v);
            if (lane == 0) dst[3 * j + comp] = v;
        }
    }
}

// A pass is bound by the latency of a thread's chain of field multiplications (the carry flag
// serialises them), not by issue slots, and the kernel is short enough for the size of its code to
// show as cold instruction fetches.  So there is ONE form of pass, spread over four lanes per pair
// of entry pairs: lane role 0..3 folds one of a0, a1, b0, b1, the four exchange their results by
// shuffle, and roles 0..2 form one product each -- two multiplications deep.  A lane keeps ONE sum
// (component `role` of the round's sums).
constexpr int SC_QUADS = SUMCHECK_THREADS / 4;             // quads (or pairs, in the first pass) per sweep of the block

// Keep a pass's sums of round j; `nthreads` (a multiple of 4, at most the block) threads took part.
// Both arrays start at zero and every slot is written at most once per walk over the rounds.
__device__ __forceinline__ void stash_sums(ScShared& sh, int j, uint64_t acc, int nthreads)
{
    const int tid = threadIdx.x, lane = tid & 31, role = tid & 3;
    if (nthreads <= 32) {
        if (tid < 32 && role < 3) sh.lane_sums[j][lane][role] = acc;
    } else if ((tid & ~31) < nthreads) {
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) acc = gl::add(acc, shfl_xor_u64(acc, o));
        if (lane < 3) sh.warp_sums[j][tid >> 5][lane] = acc;
    }
}

// the product a lane owes: g(0) = a0 b0, g(1) = a1 b1, g(2) = (2 a1 - a0)(2 b1 - b0)
__device__ __forceinline__ uint64_t role_product(int role, uint64_t a0, uint64_t a1, uint64_t b0, uint64_t b1)
{
    const uint64_t x = role == 0 ? a0 : role == 1 ? a1 : gl::sub(gl::add(a1, a1), a0);
    const uint64_t y = role == 0 ? b0 : role == 1 ? b1 : gl::sub(gl::add(b1, b1), b0);
    return gl::mul(x, y);
}

// Rounds j0..j1-1 on shared-memory tables of n entries each: one pass for round j0's sums, then
// pass j folds with r_j and accumulates round j+1's sums while j+1 < j1.  Every thread of the
// block calls this, after a block barrier that made the tables visible.  A pass whose writers
// all sit in warp 0 is followed by a warp barrier only (its readers sit in warp 0 too).
// (Not inlined: both stages of a proof share one copy of the code.)
__device__ __noinline__ void run_rounds(ScShared& sh, uint64_t* ta, uint64_t* tb, int n, int j0, int j1)
{
    const int tid = threadIdx.x, role = tid & 3;
    if (j0 >= j1) return;
    {
        const int h = n >> 1;
        uint64_t acc = 0;
        if (role < 3)
            for (int e = tid >> 2; e < h; e += SC_QUADS) acc = gl::add(acc, role_product(role, ta[e], ta[e + h], tb[e], tb[e + h]));
        stash_sums(sh, j0, acc, min(4 * h, SUMCHECK_THREADS));
    }
#pragma unroll 1
    for (int j = j0; j < j1; j++, n >>= 1) {
        const uint64_t r = sh.r[j];
        const int h = n >> 1, q = n >> 2;
        const bool next = j + 1 < j1;
        const int writers = min(4 * q, SUMCHECK_THREADS);  // threads that write table entries in this pass
        if (n == 2) {
            if (tid < 2) { uint64_t* t = tid ? tb : ta; t[0] = fold1(t[0], t[1], r); }
        } else if ((tid & ~31) < writers) {                // whole warps: the shuffles below need every lane
            uint64_t* t = role < 2 ? ta : tb;
            const int shift = (role & 1) * q;              // roles 0, 2: entry e; roles 1, 3: entry e + q
            const int base = tid & 28;                     // the quad's first lane
            uint64_t acc = 0;
#pragma unroll 1
            for (int e0 = 0; e0 < q; e0 += SC_QUADS) {
                const bool live = e0 + (tid >> 2) < q;     // (q < 8 leaves lanes of warp 0 without a quad)
                const int at = (live ? e0 + (tid >> 2) : q - 1) + shift;
                const uint64_t f = fold1(t[at], t[at + h], r);
                if (live) t[at] = f;                       // in place: only this lane reads it
                if (next) {
                    const uint64_t fa0 = shfl_idx_u64(f, base), fa1 = shfl_idx_u64(f, base + 1);
                    const uint64_t fb0 = shfl_idx_u64(f, base + 2), fb1 = shfl_idx_u64(f, base + 3);
                    if (live && role < 3) acc = gl::add(acc, role_product(role, fa0, fa1, fb0, fb1));
                }
            }
            if (next) stash_sums(sh, j + 1, acc, writers);
        }
        if (writers > 32) __syncthreads(); else __syncwarp();
    }
}

__global__ void __launch_bounds__(SUMCHECK_THREADS, 2)
sumcheck_kernel(const ProofDev* proofs, uint64_t seed, imm_fe* transcripts, int64_t stride,
                int32_t* status, int cap /* entries per shared-memory table */)
{
    pdl_launch_dependents();
    namespace cg = cooperative_groups;
    extern __shared__ __align__(16) uint64_t tabs[];       // [2][cap]
    __shared__ ScShared sh;
    cg::cluster_group cluster = cg::this_cluster();
    const int nc = (int)cluster.num_blocks(), c = (int)cluster.block_rank();
    const int proof = blockIdx.x / nc;
    const ProofDev pr = proofs[proof];
    imm_fe* tr = transcripts + (int64_t)proof * stride;
    const int tid = threadIdx.x;
    const int b = pr.b;
    const bool dist = nc > 1 && b > SC_SOLO_VARS;
    if (!dist && c != 0) return;                           // (no cluster barrier is used in that case)

    uint64_t* ta = tabs;
    uint64_t* tb = tabs + cap;
    // slice geometry: local entry e is global entry (e / W) * F + c * W + (e % W)
    const int F = dist ? SC_FINAL : 1, W = dist ? SC_FINAL / nc : 1;
    const int J = dist ? b - SC_FINAL_VARS : b;            // rounds run on the local tables
    const int L = (int)(((int64_t)1 << b) / (dist ? nc : 1));

    if (tid < b) sh.r[tid] = gl::challenge(seed, pr.round_id, 3, (uint32_t)tid);
    for (int i = tid; i < MAX_K_VARS * SC_WARPS * 3; i += SUMCHECK_THREADS) (&sh.warp_sums[0][0][0])[i] = 0;
    for (int i = tid; i < MAX_K_VARS * 32 * 3; i += SUMCHECK_THREADS) (&sh.lane_sums[0][0][0])[i] = 0;
    if (dist) cluster.barrier_arrive();                    // waited for before the first store into block 0's memory
    pdl_wait();                                            // from here on: results of the launches before
    if (pr.tab) {
        // the tables and the claim were finished by reduce_parts_kernel
        if (c == 0) {
            if (tid == 0) { tr[0] = __ldcg(pr.c0_ready); status[proof] = 0; }
            for (int64_t i = 3 * b + 3 + tid; i < stride; i += SUMCHECK_THREADS) tr[i] = 0;
        }
        const int n0 = 1 << b;
#pragma unroll 4
        for (int e = tid; e < L; e += SUMCHECK_THREADS) {
            const int y = (e / W) * F + c * W + (e % W);
            ta[e] = __ldcg(pr.tab + y);
            tb[e] = __ldcg(pr.tab + n0 + y);
        }
    } else {
        if (c == 0) {
            // claim c0 = sum of the partial sums of C
            uint64_t s = 0;
            for (int i = tid; i < pr.n_part_c; i += SUMCHECK_THREADS) s = gl::add(s, pr.part_c[i]);
            s = warp_sum_fe(s);
            if ((tid & 31) == 0) sh.red[tid >> 5] = s;
            __syncthreads();
            if (tid < 32) s = warp_sum_fe(tid < SC_WARPS ? sh.red[tid] : 0);
            if (tid < 32 && pr.c_offset) {
                // the claim kernel summed unsigned bytes: every entry reads 2^31 too high
                uint64_t sr = 0, sc = 0;
                for (int i = tid; i < pr.n_sum_row; i += 32) sr = gl::add(sr, pr.sum_row[i]);
                for (int i = tid; i < pr.n_sum_col; i += 32) sc = gl::add(sc, pr.sum_col[i]);
                sr = warp_sum_fe(sr); sc = warp_sum_fe(sc);
                s = gl::sub(s, gl::shl(gl::mul(sr, sc), 31));
            }
            if (tid == 0) { tr[0] = s; status[proof] = 0; }
            for (int64_t i = 3 * b + 3 + tid; i < stride; i += SUMCHECK_THREADS) tr[i] = 0;
        }
        __syncthreads();

        // build this block's entries from the partial vectors (all threads, one entry of each table
        // at a time), then the local rounds
#pragma unroll 1
        for (int e = tid; e < L; e += SUMCHECK_THREADS) {
            const int y = (e / W) * F + c * W + (e % W);
            const bool live = y < pr.k;                    // entries past k are the zero padding
            ta[e] = live ? sum_parts_at(pr.part_a, pr.n_part_a, pr.k, y) : 0;
            tb[e] = live ? sum_parts_at(pr.part_b, pr.n_part_b, pr.k, y) : 0;
        }
    }
    __syncthreads();
    run_rounds(sh, ta, tb, L, 0, J);
    __syncthreads();
    if (!dist) {
        reduce_round_sums(sh, 0, J, &sh.block_sums[0][0]);
        __syncthreads();
        if (tid < 3 * b) tr[1 + tid] = (&sh.block_sums[0][0])[tid];
        if (tid == 0) { tr[3 * b + 1] = ta[0]; tr[3 * b + 2] = tb[0]; }
        return;
    }

    // every block hands its slice of the folded tables and its share of the sums to block 0 (stores
    // into block 0's shared memory), then one cluster barrier: block 0 goes on, the others leave
    cluster.barrier_wait();                                // (arrived at the top) block 0 is running: its memory may be written
    {
        ScShared* sh0 = cluster.map_shared_rank(&sh, 0);
        if (tid < 2 * W) {
            const int which = tid >= W, w = tid - which * W;
            sh0->fin[which][c * W + w] = (which ? tb : ta)[w];
        }
        reduce_round_sums(sh, 0, J, &sh0->gather[c][0]);
    }
    cluster.sync();                                        // release / acquire: the stores above are visible to block 0
    if (c != 0) return;

    // block 0: the local rounds' sums, then the remaining rounds on the gathered tables
    if (tid < 3 * J) {
        uint64_t v = 0;
        for (int cc = 0; cc < nc; cc++) v = gl::add(v, sh.gather[cc][tid]);
        tr[1 + tid] = v;
    }
    run_rounds(sh, sh.fin[0], sh.fin[1], SC_FINAL, J, b);
    __syncthreads();
    reduce_round_sums(sh, J, b, &sh.block_sums[0][0]);
    __syncthreads();
    if (tid < 3 * (b - J)) tr[1 + 3 * J + tid] = (&sh.block_sums[J][0])[tid];
    if (tid == 0) { tr[3 * b + 1] = sh.fin[0][0]; tr[3 * b + 2] = sh.fin[1][0]; }
}

// ------------------------------------------------------------------------------------------
// non-interactive (Fiat-Shamir) proof: challenges hashed from the statement and the transcript
// ------------------------------------------------------------------------------------------
// H = SHA-256; integers little-endian; a field element is the le64 of its canonical value;
// fe(d) = the first 8 bytes of a digest as a big-endian integer, minus p if not below p.
//   s_0     = H(0x10 || com_A || com_B || com_C || le64(m) || le64(k) || le64(n) || le64(proof_id))
//   r_row[t] = fe(H(0x11 || s_0 || le32(1) || le32(t))),  r_col[t] with le32(2)
//   s_1     = H(0x12 || s_0 || le64(c0))
//   s_{j+2} = H(0x13 || s_{j+1} || le64(g_j(0)) || le64(g_j(2))),  r_j = fe(s_{j+2})
// (g_j(1) is sent but not hashed: the verifier's sum check pins it to the claim; without it the
// message is one SHA-256 block)

__device__ __forceinline__ uint64_t fs_fe(const uint32_t (&h)[8])
{
    const uint64_t v = ((uint64_t)h[0] << 32) | h[1];
    return v >= gl::P ? v - gl::P : v;
}

__device__ __forceinline__ void fs_put_le(uint8_t* dst, uint64_t v, int nbytes)
{
    for (int q = 0; q < nbytes; q++) dst[q] = (uint8_t)(v >> (8 * q));
}

// s <- H(tag || s || le64(vals[0..NV))), NV = 1 or 2.  The message is the word stream
// [s_0..s_7, byte-swapped halves of the values] moved one byte to the right behind the tag, so its
// words are built with shifts instead of byte by byte (the hash sits on the rounds' critical path:
// one thread, nothing to overlap it with).
template <int NV>
__device__ __forceinline__ void fs_absorb(uint32_t (&s)[8], uint32_t tag, const uint64_t (&vals)[NV], uint32_t one)
{
    constexpr int L = 8 + 2 * NV;                          // stream words; the message has 1 + 4 L bytes
    uint32_t st[L];
#pragma unroll
    for (int i = 0; i < 8; i++) st[i] = s[i];
#pragma unroll
    for (int i = 0; i < NV; i++) {
        st[8 + 2 * i] = __byte_perm((uint32_t)vals[i], 0, 0x0123);            // little-endian bytes in stream order
        st[9 + 2 * i] = __byte_perm((uint32_t)(vals[i] >> 32), 0, 0x0123);
    }
    uint32_t w[16];
    w[0] = (tag << 24) | (st[0] >> 8);
#pragma unroll
    for (int i = 1; i < 16; i++) {
        if (i < L) w[i] = (st[i - 1] << 24) | (st[i] >> 8);
        else if (i == L) w[i] = (st[L - 1] << 24) | 0x00800000u;
        else w[i] = 0;
    }
    const uint32_t bits = (1 + 4 * L) * 8;
    constexpr int NBLOCKS = L < 14 ? 1 : 2;                // one block if 0x80 and the length fit behind the words
    if (NBLOCKS == 1) w[15] = bits;
    imm_sha::iv(s);
#pragma unroll 1
    for (int blk = 0; blk < NBLOCKS; blk++) {              // (one copy of the compression in the code)
        if (blk == 1) {
#pragma unroll
            for (int i = 0; i < 15; i++) w[i] = 0;
            w[15] = bits;
        }
        imm_sha::compress(s, w, one);
    }
}

// Sums of three values per thread over the block at once; results valid in thread 0.
__device__ __forceinline__ void block_sum3_fe(uint64_t (&v)[3], uint64_t (*scratch)[32])
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = (blockDim.x + 31) >> 5;
#pragma unroll
    for (int i = 0; i < 3; i++) v[i] = warp_sum_fe(v[i]);
    __syncthreads();                       // scratch may still be read from the previous round
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < 3; i++) scratch[i][warp] = v[i];
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
        for (int i = 0; i < 3; i++) v[i] = warp_sum_fe(lane < nwarp ? scratch[i][lane] : 0);
    }
}

// Statement hash and the two evaluation points of every proof (one block per proof).
__global__ void __launch_bounds__(2 * FS_POINT_SLOTS) fs_points_kernel(const ProofDev* proofs, const FsProof* fs)
{
    __shared__ uint32_t s0[8];
    const ProofDev& pr = proofs[blockIdx.x];
    const FsProof& f = fs[blockIdx.x];
    if (threadIdx.x == 0) {
        uint8_t m[136];
        m[0] = 0x10;
        for (int i = 0; i < 96; i++) m[1 + i] = f.com[i];
        fs_put_le(m + 97, (uint64_t)pr.m, 8);
        fs_put_le(m + 105, (uint64_t)pr.k, 8);
        fs_put_le(m + 113, (uint64_t)pr.n, 8);
        fs_put_le(m + 121, f.proof_id, 8);
        uint32_t h[8];
        imm_sha::sha256_short(m, 129, h, f.one);
        for (int i = 0; i < 8; i++) { s0[i] = h[i]; f.state[i] = h[i]; }
    }
    __syncthreads();
    const int which = threadIdx.x / FS_POINT_SLOTS, t = threadIdx.x % FS_POINT_SLOTS;     // 0: r_row, 1: r_col
    if (t < (which == 0 ? pr.a : pr.c)) {
        uint8_t m[48];
        uint32_t h[8];
        for (int i = 0; i < 8; i++) h[i] = s0[i];
        m[0] = 0x11;
        imm_sha::digest_bytes(h, m + 1);
        fs_put_le(m + 33, (uint64_t)(which + 1), 4);
        fs_put_le(m + 37, (uint64_t)t, 4);
        imm_sha::sha256_short(m, 41, h, f.one);
        f.points[which * FS_POINT_SLOTS + t] = fs_fe(h);
    }
}

// The rounds of one proof by one block: every round's three sums are reduced over the block, hashed
// into the transcript state by thread 0, and only then is the round's challenge known and the fold
// can run.  The two tables live in global memory (they stay in L2).
__global__ void __launch_bounds__(FS_THREADS)
sumcheck_fs_kernel(const ProofDev* proofs, const FsProof* fs, imm_fe* transcripts, int64_t stride, int32_t* status)
{
    __shared__ uint64_t red[35];
    __shared__ uint64_t red3[3][32];
    __shared__ uint64_t r_sh;
    const ProofDev pr = proofs[blockIdx.x];
    const FsProof f = fs[blockIdx.x];
    imm_fe* tr = transcripts + (int64_t)blockIdx.x * stride;
    const int tid = threadIdx.x, b = pr.b;
    imm_fe* ta = f.ta;
    imm_fe* tb = f.tb;

    // claim c0 = sum of the partial sums of C (minus the 2^31 offset of the byte-wise kernel)
    uint64_t s = 0;
    for (int i = tid; i < pr.n_part_c; i += FS_THREADS) s = gl::add(s, pr.part_c[i]);
    s = block_sum_fe(s, red);
    s = gl::sub(s, claim_offset_block(pr, red));
    uint32_t st[8];                                        // the transcript state (thread 0)
    if (tid == 0) {
        tr[0] = s;
        status[blockIdx.x] = 0;
#pragma unroll
        for (int i = 0; i < 8; i++) st[i] = f.state[i];
        const uint64_t c0[1] = {s};
        fs_absorb<1>(st, 0x12, c0, f.one);
    }
    for (int64_t i = 3 * b + 3 + tid; i < stride; i += FS_THREADS) tr[i] = 0;

    // both tables from the partial vectors; entries past k are the zero padding
    const int n0 = 1 << b;
    for (int y = tid; y < n0; y += FS_THREADS) {
        const bool live = y < pr.k;
        ta[y] = live ? sum_parts_at(pr.part_a, pr.n_part_a, pr.k, y) : 0;
        tb[y] = live ? sum_parts_at(pr.part_b, pr.n_part_b, pr.k, y) : 0;
    }
    __syncthreads();

    // round 0's sums come from the tables; every later round's sums are taken from the folded
    // values as the fold of the round before produces them (one pass over the tables per round)
    Sums3 acc = {0, 0, 0};
    for (int e = tid; e < (n0 >> 1); e += FS_THREADS) sums_add(acc, ta[e], ta[e + (n0 >> 1)], tb[e], tb[e + (n0 >> 1)]);
    for (int j = 0, n = n0; j < b; j++, n >>= 1) {
        const int h = n >> 1, q = n >> 2;
        uint64_t g[3] = {acc.g0, acc.g1, acc.g2};
        block_sum3_fe(g, red3);                            // (its barriers also order the fold's writes before the next reads)
        if (tid == 0) {
            tr[1 + 3 * j] = g[0]; tr[2 + 3 * j] = g[1]; tr[3 + 3 * j] = g[2];
            const uint64_t hashed[2] = {g[0], g[2]};
            fs_absorb<2>(st, 0x13, hashed, f.one);
            r_sh = fs_fe(st);
        }
        __syncthreads();
        const uint64_t r = r_sh;
        acc = Sums3{0, 0, 0};
        if (h == 1) {
            if (tid == 0) { ta[0] = fold1(ta[0], ta[1], r); tb[0] = fold1(tb[0], tb[1], r); }
        } else {
            for (int e = tid; e < q; e += FS_THREADS) {    // in place: each thread rewrites only what it alone read
                const uint64_t fa0 = fold1(ta[e], ta[e + h], r), fa1 = fold1(ta[e + q], ta[e + q + h], r);
                const uint64_t fb0 = fold1(tb[e], tb[e + h], r), fb1 = fold1(tb[e + q], tb[e + q + h], r);
                ta[e] = fa0; ta[e + q] = fa1; tb[e] = fb0; tb[e + q] = fb1;
                sums_add(acc, fa0, fa1, fb0, fb1);
            }
        }
    }
    __syncthreads();
    if (tid == 0) { tr[3 * b + 1] = ta[0]; tr[3 * b + 2] = tb[0]; }
}

// ------------------------------------------------------------------------------------------
// batched non-interactive proof: one sumcheck for all members, every coin hashed
// ------------------------------------------------------------------------------------------
//   root  = Merkle tree hash (RFC 6962) over the member statements s_0^(p) (32-byte leaves)
//   T     = H(0x14 || root || le64(batch_id) || le32(P)),   rho_p = fe(H(0x15 || T || le32(p)))
//   s_1   = H(0x12 || T || le64(c0B)), c0B = sum_p rho_p c0_p;  rounds as above on the combined sums.
// Every round needs the sum over ALL members before its challenge exists, so the rounds are a chain
// of small launches (members fold side by side, one block combines and hashes) instead of blocks
// that wait for one another.

__global__ void __launch_bounds__(FS_BATCH_MAX) fsb_seed_kernel(const FsProof* fs, FsBatch fb)
{
    __shared__ imm_sha::Digest sd[FS_BATCH_MAX];
    __shared__ uint32_t T_sh[8];
    const int p = threadIdx.x;
    if (p < fb.nproofs) {                                  // leaf = H(0x00 || s_0^(p))
        uint8_t m[40];
        uint32_t h[8];
        for (int i = 0; i < 8; i++) h[i] = fs[p].state[i];
        m[0] = 0x00;
        imm_sha::digest_bytes(h, m + 1);
        imm_sha::sha256_short(m, 33, h, fb.one);
        for (int i = 0; i < 8; i++) sd[p].h[i] = h[i];
    }
    __syncthreads();
    imm_sha::fold(sd, fb.nproofs, fb.one);
    if (p == 0) {
        uint8_t m[48];
        uint32_t h[8];
        for (int i = 0; i < 8; i++) h[i] = sd[0].h[i];
        m[0] = 0x14;
        imm_sha::digest_bytes(h, m + 1);
        fs_put_le(m + 33, fb.batch_id, 8);
        fs_put_le(m + 41, (uint64_t)fb.nproofs, 4);
        imm_sha::sha256_short(m, 45, h, fb.one);
        for (int i = 0; i < 8; i++) { T_sh[i] = h[i]; fb.T[i] = h[i]; }
    }
    __syncthreads();
    if (p < fb.nproofs) {
        uint8_t m[40];
        uint32_t h[8];
        for (int i = 0; i < 8; i++) h[i] = T_sh[i];
        m[0] = 0x15;
        imm_sha::digest_bytes(h, m + 1);
        fs_put_le(m + 33, (uint64_t)p, 4);
        imm_sha::sha256_short(m, 37, h, fb.one);
        fb.rho[p] = fs_fe(h);
    }
}

// Member p: its claim, its two tables, and rho_p times the sums of round 0.  With no rounds at all
// (every k = 1) the member's three transcript words are complete here.
__global__ void __launch_bounds__(FS_THREADS)
fsb_build_kernel(const ProofDev* proofs, const FsProof* fs, FsBatch fb, imm_fe* tr, int32_t* status)
{
    __shared__ uint64_t red[35];
    __shared__ uint64_t red3[3][32];
    const int p = blockIdx.x, tid = threadIdx.x, b = fb.b;
    const ProofDev pr = proofs[p];
    imm_fe* ta = fs[p].ta;
    imm_fe* tb = fs[p].tb;
    uint64_t s = 0;
    for (int i = tid; i < pr.n_part_c; i += FS_THREADS) s = gl::add(s, pr.part_c[i]);
    s = block_sum_fe(s, red);
    s = gl::sub(s, claim_offset_block(pr, red));
    const int n0 = 1 << b;
    for (int y = tid; y < n0; y += FS_THREADS) {
        const bool live = y < pr.k;
        ta[y] = live ? sum_parts_at(pr.part_a, pr.n_part_a, pr.k, y) : 0;
        tb[y] = live ? sum_parts_at(pr.part_b, pr.n_part_b, pr.k, y) : 0;
    }
    __syncthreads();
    Sums3 acc = {0, 0, 0};
    for (int e = tid; e < (n0 >> 1); e += FS_THREADS) sums_add(acc, ta[e], ta[e + (n0 >> 1)], tb[e], tb[e + (n0 >> 1)]);
    uint64_t g[3] = {acc.g0, acc.g1, acc.g2};
    block_sum3_fe(g, red3);
    if (tid == 0) {
        const uint64_t rho = fb.rho[p];
        fb.c0[p] = s;
        status[p] = 0;
        for (int i = 0; i < 3; i++) fb.partial[3 * p + i] = gl::mul(rho, g[i]);
        imm_fe* tail = tr + 1 + 3 * b + 3 * (int64_t)p;
        tail[0] = s;
        if (b == 0) { tail[1] = ta[0]; tail[2] = tb[0]; }
    }
}

// Round j of the whole batch (one block): the combined sums, the transcript words, the hash, r_j.
// j = 0 also forms the combined claim and starts the transcript state; with b = 0 that is all.
__global__ void __launch_bounds__(FS_BATCH_MAX) fsb_combine_kernel(FsBatch fb, int j, imm_fe* tr)
{
    __shared__ uint64_t red[33];
    __shared__ uint64_t red3[3][32];
    const int tid = threadIdx.x;
    uint32_t st[8];
    if (j == 0) {
        uint64_t c = 0;
        for (int p = tid; p < fb.nproofs; p += (int)blockDim.x) c = gl::add(c, gl::mul(fb.rho[p], fb.c0[p]));
        c = block_sum_fe(c, red);
        if (tid == 0) {
            tr[0] = c;
#pragma unroll
            for (int i = 0; i < 8; i++) st[i] = fb.T[i];
            const uint64_t c0[1] = {c};
            fs_absorb<1>(st, 0x12, c0, fb.one);
            if (fb.b == 0) {
#pragma unroll
                for (int i = 0; i < 8; i++) fb.state[i] = st[i];
            }
        }
        if (fb.b == 0) return;
    } else if (tid == 0) {
#pragma unroll
        for (int i = 0; i < 8; i++) st[i] = fb.state[i];
    }
    uint64_t g[3] = {0, 0, 0};
    for (int p = tid; p < fb.nproofs; p += (int)blockDim.x)
        for (int i = 0; i < 3; i++) g[i] = gl::add(g[i], fb.partial[3 * p + i]);
    block_sum3_fe(g, red3);
    if (tid == 0) {
        tr[1 + 3 * j] = g[0]; tr[2 + 3 * j] = g[1]; tr[3 + 3 * j] = g[2];
        const uint64_t hashed[2] = {g[0], g[2]};
        fs_absorb<2>(st, 0x13, hashed, fb.one);
        fb.r[j] = fs_fe(st);
#pragma unroll
        for (int i = 0; i < 8; i++) fb.state[i] = st[i];
    }
}

// Member p folds with r_j and takes rho_p times the sums of round j + 1 from the folded values; after
// the last round its a_fin, b_fin complete its three transcript words.
__global__ void __launch_bounds__(FS_THREADS)
fsb_fold_kernel(const FsProof* fs, FsBatch fb, int j, imm_fe* tr)
{
    __shared__ uint64_t red3[3][32];
    const int p = blockIdx.x, tid = threadIdx.x, b = fb.b;
    imm_fe* ta = fs[p].ta;
    imm_fe* tb = fs[p].tb;
    const uint64_t r = fb.r[j];
    const int n = 1 << (b - j), h = n >> 1, q = n >> 2;
    if (h == 1) {
        if (tid == 0) {
            imm_fe* tail = tr + 1 + 3 * b + 3 * (int64_t)p;
            tail[1] = fold1(ta[0], ta[1], r);
            tail[2] = fold1(tb[0], tb[1], r);
        }
        return;
    }
    Sums3 acc = {0, 0, 0};
    for (int e = tid; e < q; e += FS_THREADS) {            // in place: each thread rewrites only what it alone read
        const uint64_t fa0 = fold1(ta[e], ta[e + h], r), fa1 = fold1(ta[e + q], ta[e + q + h], r);
        const uint64_t fb0 = fold1(tb[e], tb[e + h], r), fb1 = fold1(tb[e + q], tb[e + q + h], r);
        ta[e] = fa0; ta[e + q] = fa1; tb[e] = fb0; tb[e + q] = fb1;
        sums_add(acc, fa0, fa1, fb0, fb1);
    }
    uint64_t g[3] = {acc.g0, acc.g1, acc.g2};
    block_sum3_fe(g, red3);
    if (tid == 0) {
        const uint64_t rho = fb.rho[p];
        for (int i = 0; i < 3; i++) fb.partial[3 * p + i] = gl::mul(rho, g[i]);
    }
}

// ------------------------------------------------------------------------------------------
// the verifier's own evaluations: c0 = C~(r_row, r_col), a_fin = A~(r_row, r_k), b_fin = B~(r_k, r_col)
// ------------------------------------------------------------------------------------------
// The three contractions are the prover's (partial sums of C, partial vectors of A and B); where the
// prover runs the rounds, the verifier only needs the two inner products with E_k.  One block per proof.
__global__ void __launch_bounds__(SUMCHECK_THREADS)
expected_kernel(const ProofDev* proofs, const ExpectDev* ex, imm_fe* expected, int32_t* status)
{
    __shared__ uint64_t red[35];
    const ProofDev pr = proofs[blockIdx.x];
    const imm_fe* e_k = ex[blockIdx.x].e_k;
    const int tid = threadIdx.x;
    uint64_t s = 0;
    for (int i = tid; i < pr.n_part_c; i += SUMCHECK_THREADS) s = gl::add(s, pr.part_c[i]);
    s = block_sum_fe(s, red);
    s = gl::sub(s, claim_offset_block(pr, red));           // the byte-wise claim kernel read every entry 2^31 too high
    uint64_t a = 0, b = 0;
    for (int y = tid; y < pr.k; y += SUMCHECK_THREADS) {   // entries past k meet the zero padding
        const uint64_t w = e_k[y];
        a = gl::add(a, gl::mul(w, sum_parts_at(pr.part_a, pr.n_part_a, pr.k, y)));
        b = gl::add(b, gl::mul(w, sum_parts_at(pr.part_b, pr.n_part_b, pr.k, y)));
    }
    a = block_sum_fe(a, red);
    b = block_sum_fe(b, red);
    if (tid == 0) {
        expected[3 * (int64_t)blockIdx.x] = s;
        expected[3 * (int64_t)blockIdx.x + 1] = a;
        expected[3 * (int64_t)blockIdx.x + 2] = b;
        status[blockIdx.x] = 0;
    }
}

// ------------------------------------------------------------------------------------------
// launch wrappers
// ------------------------------------------------------------------------------------------

// Streaming multiprocessors of the current device, looked up once per device; 148 (a B200) where no
// device answers, so that the host-side planning calls still work without one.
int sm_count()
{
    static int cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { (void)cudaGetLastError(); return 148; }
    if (cached[dev] == 0) {
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
            (void)cudaGetLastError();
            return 148;
        }
        cached[dev] = v;
    }
    return cached[dev];
}

cudaError_t launch_fs_batched_rounds(const ProofDev* d_proofs, const FsProof* d_fs, const FsBatch& fb, imm_fe* transcript,
                                     int32_t* status, cudaStream_t st)
{
    int ct = (fb.nproofs + 31) / 32 * 32;                  // threads of the combining block: one per member, whole warps
    if (ct > FS_BATCH_MAX) ct = FS_BATCH_MAX;
    fsb_seed_kernel<<<1, FS_BATCH_MAX, 0, st>>>(d_fs, fb);
    fsb_build_kernel<<<fb.nproofs, FS_THREADS, 0, st>>>(d_proofs, d_fs, fb, transcript, status);
    fsb_combine_kernel<<<1, ct, 0, st>>>(fb, 0, transcript);
    for (int j = 0; j < fb.b; j++) {
        if (j > 0) fsb_combine_kernel<<<1, ct, 0, st>>>(fb, j, transcript);
        fsb_fold_kernel<<<fb.nproofs, FS_THREADS, 0, st>>>(d_fs, fb, j, transcript);
    }
    return cudaGetLastError();
}

cudaError_t launch_expected(const ProofDev* d_proofs, const ExpectDev* d_ex, int nproofs, imm_fe* expected,
                            int32_t* status, cudaStream_t st)
{
    expected_kernel<<<nproofs, SUMCHECK_THREADS, 0, st>>>(d_proofs, d_ex, expected, status);
    return cudaGetLastError();
}

cudaError_t launch_fs_points(const ProofDev* d_proofs, const FsProof* d_fs, int nproofs, cudaStream_t st)
{
    fs_points_kernel<<<nproofs, 2 * FS_POINT_SLOTS, 0, st>>>(d_proofs, d_fs);
    return cudaGetLastError();
}

cudaError_t launch_sumcheck_fs(const ProofDev* d_proofs, const FsProof* d_fs, int nproofs, imm_fe* transcripts,
                               int64_t stride, int32_t* status, cudaStream_t st)
{
    sumcheck_fs_kernel<<<nproofs, FS_THREADS, 0, st>>>(d_proofs, d_fs, transcripts, stride, status);
    return cudaGetLastError();
}

cudaError_t launch_field_binop(int op, const imm_fe* x, const imm_fe* y, imm_fe* out, int64_t n,
                               cudaStream_t st)
{
    if (n <= 0) return cudaSuccess;
    int64_t blocks = (n + 255) / 256;
    if (blocks > sm_count() * 16) blocks = sm_count() * 16;
    field_binop_kernel<<<(unsigned)blocks, 256, 0, st>>>(op, x, y, out, n);
    return cudaGetLastError();
}

cudaError_t launch_eq_direct(const EqDirect& r, int nvars, imm_fe* out, cudaStream_t st)
{
    eq_direct_kernel<<<1, 1024, 0, st>>>(r, nvars, out);
    return cudaGetLastError();
}

cudaError_t launch_eq_batch(const EqTask* d_tasks, int ntasks, int64_t max_cover, cudaStream_t st)
{
    if (ntasks <= 0 || max_cover <= 0) return cudaSuccess;
    const int64_t slice = 4 * (int64_t)EQ_SLICE_QUADS;
    dim3 grid((unsigned)((max_cover + slice - 1) / slice), (unsigned)ntasks);
    eq_batch_kernel<<<grid, EQ_BATCH_THREADS, 0, st>>>(d_tasks);
    return cudaGetLastError();
}

cudaError_t launch_rowbind(int dtype, bool point, const MatJob* d_jobs, int njobs, uint32_t ntiles,
                           cudaStream_t st)
{
    if (ntiles == 0) return cudaSuccess;
    if (dtype == 0) {
        if (point) rowbind_kernel<int8_t, true><<<ntiles, ROWBIND_THREADS, 0, st>>>(d_jobs, njobs);
        else rowbind_kernel<int8_t, false><<<ntiles, ROWBIND_THREADS, 0, st>>>(d_jobs, njobs);
    } else {
        if (point) rowbind_kernel<int32_t, true><<<ntiles, ROWBIND_THREADS, 0, st>>>(d_jobs, njobs);
        else rowbind_kernel<int32_t, false><<<ntiles, ROWBIND_THREADS, 0, st>>>(d_jobs, njobs);
    }
    return cudaGetLastError();
}

cudaError_t launch_colbind(int dtype, const MatJob* d_jobs, int njobs, uint32_t ntiles, cudaStream_t st)
{
    if (ntiles == 0) return cudaSuccess;
    if (dtype == 0) colbind_kernel<int8_t><<<ntiles, COLBIND_THREADS, 0, st>>>(d_jobs, njobs);
    else colbind_kernel<int32_t><<<ntiles, COLBIND_THREADS, 0, st>>>(d_jobs, njobs);
    return cudaGetLastError();
}

cudaError_t launch_bytedot(bool i32, bool point, int mt, const MatJob* d_jobs, int njobs, uint32_t ntiles,
                           cudaStream_t st)
{
    if (ntiles == 0) return cudaSuccess;
#define BD_LAUNCH(I, P, M) bytedot_kernel<I, P, M><<<ntiles, BYTEDOT_THREADS, 0, st>>>(d_jobs, njobs)
    if (i32) {
        if (!point) return cudaErrorInvalidValue;          // the offset int32 view serves point evaluation only
        if (mt == 2) BD_LAUNCH(true, true, 2); else BD_LAUNCH(true, true, 1);
    } else {
        if (point) { if (mt == 2) BD_LAUNCH(false, true, 2); else BD_LAUNCH(false, true, 1); }
        else { if (mt == 2) BD_LAUNCH(false, false, 2); else BD_LAUNCH(false, false, 1); }
    }
#undef BD_LAUNCH
    return cudaGetLastError();
}

cudaError_t launch_rowmma(const MatJob* d_jobs, int njobs, uint32_t ntiles, int warps, cudaStream_t st)
{
    if (ntiles == 0) return cudaSuccess;
    if (warps < 1 || warps > ROWMMA_MAX_WARPS) return cudaErrorInvalidValue;
    const size_t smem = (size_t)warps * ROWLDM_STAGES * ROWLDM_STAGE_BYTES;         // 18 KiB per warp
    cudaError_t e = cudaFuncSetAttribute(rowmma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ROWMMA_MAX_WARPS * ROWLDM_STAGES * ROWLDM_STAGE_BYTES);
    if (e != cudaSuccess) return e;
    rowmma_kernel<<<ntiles, 32 * warps, smem, st>>>(d_jobs, njobs);
    return cudaGetLastError();
}

cudaError_t launch_sum_parts(const imm_fe* parts, int nparts, int64_t len, imm_fe* out, cudaStream_t st)
{
    if (len <= 0) return cudaSuccess;
    sum_parts_kernel<<<(unsigned)((len + 255) / 256), 256, 0, st>>>(parts, nparts, len, out);
    return cudaGetLastError();
}

cudaError_t launch_sum_all(const imm_fe* parts, int64_t count, imm_fe* out, cudaStream_t st)
{
    sum_all_kernel<<<1, 1024, 0, st>>>(parts, count, out);
    return cudaGetLastError();
}

cudaError_t launch_point_finish(const imm_fe* parts, int64_t count, const imm_fe* sum_row, int nsr,
                                const imm_fe* sum_col, int nsc, imm_fe* out, cudaStream_t st)
{
    point_finish_kernel<<<1, 1024, 0, st>>>(parts, count, sum_row, nsr, sum_col, nsc, out);
    return cudaGetLastError();
}

// Batched transcript of `nproofs` proofs that ran under shared round challenges (rows of
// `stride` words in `tr`, each 3b+3 long): word w < 1+3b of `out` is sum_p rho_p tr[p][w] with
// rho_p = challenge(seed, batch_id, 4, p) -- one block per word -- and the remaining blocks copy
// every proof's (c0, a_fin, b_fin) behind them.
__global__ void __launch_bounds__(COMBINE_THREADS)
combine_kernel(const imm_fe* tr, int64_t stride, int nproofs, int b, uint64_t seed, uint64_t batch_id, imm_fe* out)
{
    __shared__ uint64_t red[33];
    const int nw = 1 + 3 * b;
    if ((int)blockIdx.x < nw) {
        uint64_t s = 0;
        for (int p = threadIdx.x; p < nproofs; p += COMBINE_THREADS)
            s = gl::add(s, gl::mul(gl::challenge(seed, batch_id, 4, (uint32_t)p), tr[(int64_t)p * stride + blockIdx.x]));
        s = block_sum_fe(s, red);
        if (threadIdx.x == 0) out[blockIdx.x] = s;
        return;
    }
    const int p = ((int)blockIdx.x - nw) * COMBINE_THREADS + threadIdx.x;
    if (p >= nproofs) return;
    const imm_fe* row = tr + (int64_t)p * stride;
    imm_fe* o = out + nw + 3 * (int64_t)p;
    o[0] = row[0];
    o[1] = row[3 * b + 1];
    o[2] = row[3 * b + 2];
}

cudaError_t launch_combine(const imm_fe* tr, int64_t stride, int nproofs, int b, uint64_t seed, uint64_t batch_id,
                           imm_fe* out, cudaStream_t st)
{
    const unsigned blocks = (unsigned)(1 + 3 * b + (nproofs + COMBINE_THREADS - 1) / COMBINE_THREADS);
    combine_kernel<<<blocks, COMBINE_THREADS, 0, st>>>(tr, stride, nproofs, b, seed, batch_id, out);
    return cudaGetLastError();
}

cudaError_t launch_fused_contract(const FusedJob* d_jobs, const FusedSeg* d_segs, const uint32_t* d_block_first,
                                  uint32_t nblocks, cudaStream_t st)
{
    if (nblocks == 0) return cudaSuccess;
    fused_contract_kernel<<<nblocks, BYTEDOT_THREADS, 0, st>>>(d_jobs, d_segs, d_block_first);
    return cudaGetLastError();
}

// Launched as a programmatic dependent of the kernel before it in the stream: it may start while that
// one drains and waits (griddepcontrol.wait) before it reads its results.
cudaError_t launch_reduce_parts(const ProofDev* d_proofs, int nproofs, int max_b, cudaStream_t st)
{
    if (nproofs <= 0) return cudaSuccess;
    const int n0 = 1 << (max_b > 0 ? max_b : 0);
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)((n0 + REDUCE_THREADS - 1) / REDUCE_THREADS + 1), (unsigned)nproofs);
    cfg.blockDim = dim3(REDUCE_THREADS);
    cfg.stream = st;
    cudaLaunchAttribute attr;
    memset(&attr, 0, sizeof(attr));
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, reduce_parts_kernel, d_proofs);
}

cudaError_t launch_sumcheck(const ProofDev* d_proofs, int nproofs, uint64_t seed, imm_fe* transcripts,
                            int64_t stride, int32_t* status, int max_b, int cluster, bool dependent, cudaStream_t st)
{
    if (nproofs <= 0) return cudaSuccess;
    // Blocks per proof: as many as keep every proof of the batch resident at once (two blocks fit
    // an SM), at most 8, and at least what the shared-memory tables need (a block holds its share
    // of the 2^b entries of both tables).
    int nc = 1;
    if (max_b > SC_SOLO_VARS) {
        while (2 * nc <= SC_PORTABLE_CLUSTER && (int64_t)2 * nc * nproofs <= 2 * sm_count()) nc *= 2;
        if (cluster == 1 || cluster == 2 || cluster == 4 || cluster == 8) nc = cluster;     // caller's choice
        while (nc < SUMCHECK_MAX_CLUSTER && (((int64_t)1 << max_b) / nc) > SC_MAX_CAP) nc *= 2;
    }
    int64_t cap = ((int64_t)1 << (max_b > 0 ? max_b : 0)) / (max_b > SC_SOLO_VARS ? nc : 1);
    if (cap < (1 << SC_SOLO_VARS)) cap = 1 << SC_SOLO_VARS;                // a solo proof inside a cluster launch
    if (cap > SC_MAX_CAP) return cudaErrorInvalidValue;                      // k beyond 2^17
    const size_t smem = (size_t)cap * 2 * sizeof(uint64_t);
    cudaError_t e = cudaFuncSetAttribute(sumcheck_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem);
    if (e != cudaSuccess) return e;
    if (nc > SC_PORTABLE_CLUSTER) {
        e = cudaFuncSetAttribute(sumcheck_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = dim3((unsigned)(nproofs * nc));
    cfg.blockDim = dim3(SUMCHECK_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    memset(attr, 0, sizeof(attr));
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)nc;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;       // see launch_reduce_parts
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 2 : 1;
    return cudaLaunchKernelEx(&cfg, sumcheck_kernel, d_proofs, seed, transcripts, stride, status, (int)cap);
}

}  // namespace imm

// ------------------------------------------------------------------------------------------
// point evaluation without a caller workspace (imm_mle_eval_point_noalloc)
// ------------------------------------------------------------------------------------------
// For callers that may not allocate device memory (code running inside a serving engine whose
// pool owns all of HBM): the per-tile partial sums go to a fixed array in this library's device
// image instead of a workspace.  In host code the array's name is only a stand-in for the
// symbol, not a device address, so the address is looked up once per device with
// cudaGetSymbolAddress and handed to the kernels.

#include <mutex>

#include "../../include/imm.h"

namespace imm {

constexpr int NOALLOC_MAX_DEVICES = 64;

static __device__ __align__(256) imm_fe g_noalloc_partials[IMM_NOALLOC_MAX_TILES];   // 64 KiB per GPU

static imm_fe* g_noalloc_ptr[NOALLOC_MAX_DEVICES];      // device address of the array, per device
static std::mutex g_noalloc_mutex;

// Same tile code as rowbind_kernel<T, POINT>, with the job passed by value (no descriptor upload).
template <typename T>
__global__ void __launch_bounds__(ROWBIND_THREADS) rowbind_point_byvalue_kernel(const MatJob job)
{
    __shared__ int2 sE[MAX_TILE_ROWS];
    __shared__ uint64_t red[33];
    if (job.vec) rowbind_tile<T, true, true>(job, blockIdx.x, sE, red);
    else rowbind_tile<T, true, false>(job, blockIdx.x, sE, red);
}

static cudaError_t noalloc_scratch(imm_fe** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= NOALLOC_MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        imm_fe* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_noalloc_partials);     // set-up: once per device
        if (e != cudaSuccess) return e;
        g_noalloc_ptr[dev] = p;
    }
    *out = g_noalloc_ptr[dev];
    return cudaSuccess;
}

}  // namespace imm

extern "C" int imm_mle_eval_point_noalloc(const void* d_mat, int dtype, int64_t rows, int64_t cols,
                                          int64_t ld, const imm_fe* d_eq_row, const imm_fe* d_eq_col,
                                          imm_fe* d_out, void* stream)
{
    using namespace imm;
    if (!d_mat || !d_eq_row || !d_eq_col || !d_out || (dtype != IMM_I8 && dtype != IMM_I32)) return IMM_ERR_ARG;
    if (rows <= 0 || cols <= 0 || rows > ((int64_t)1 << 20) || cols > ((int64_t)1 << 20) || ld < cols)
        return IMM_ERR_SHAPE;
    if ((uintptr_t)d_out % 8 != 0 || (uintptr_t)d_eq_row % 8 != 0 || (uintptr_t)d_eq_col % 8 != 0) return IMM_ERR_ALIGN;
    const int esz = dtype == IMM_I8 ? 1 : 4;
    const int cols_per_tile = ROWBIND_THREADS * (16 / esz);
    const int64_t ncc = (cols + cols_per_tile - 1) / cols_per_tile;
    // smallest tile height (from 32 rows up) whose tile count fits the fixed array
    int tile_rows = 32;
    while (tile_rows < MAX_TILE_ROWS && ((rows + tile_rows - 1) / tile_rows) * ncc > IMM_NOALLOC_MAX_TILES)
        tile_rows *= 2;
    const int64_t nrb = (rows + tile_rows - 1) / tile_rows;
    if (nrb * ncc > IMM_NOALLOC_MAX_TILES) return IMM_ERR_LIMIT;

    imm_fe* scratch = nullptr;
    if (noalloc_scratch(&scratch) != cudaSuccess) return IMM_ERR_CUDA;

    MatJob j;
    memset(&j, 0, sizeof(j));
    j.mat = d_mat;
    j.eq_row = d_eq_row;
    j.eq_col = d_eq_col;
    j.out = scratch;
    j.ld = ld;
    j.rows = (int32_t)rows;
    j.cols = (int32_t)cols;
    j.tile_rows = tile_rows;
    j.nrb = (int32_t)nrb;
    j.ncc = (int32_t)ncc;
    j.vec = (((uintptr_t)d_mat % 16 == 0) && ((ld * esz) % 16 == 0)) ? 1 : 0;
    cudaStream_t st = (cudaStream_t)stream;
    const unsigned ntiles = (unsigned)(nrb * ncc);
    if (dtype == IMM_I8) rowbind_point_byvalue_kernel<int8_t><<<ntiles, ROWBIND_THREADS, 0, st>>>(j);
    else rowbind_point_byvalue_kernel<int32_t><<<ntiles, ROWBIND_THREADS, 0, st>>>(j);
    if (cudaGetLastError() != cudaSuccess) return IMM_ERR_CUDA;
    sum_all_kernel<<<1, 1024, 0, st>>>(scratch, (int64_t)ntiles, d_out);
    if (cudaGetLastError() != cudaSuccess) return IMM_ERR_CUDA;
    return IMM_OK;
}
