// Small batches: one contraction launch for all three matrix kinds, with the eq weights built inside
// the tiles (included by imm_kernels.cu after imm_mma.cuh).
//
// A batch of a few hundred megabytes is over in tens of microseconds, so every dependent launch in
// front of the streaming (an eq-table kernel, three forked contraction kernels and their joins)
// costs as much as a good part of the streaming itself.  Here a proving pass is three launches chained
// by programmatic dependent launch:
//   fused_contract_kernel   A (row binding), B (column binding) and C (claim) in one persistent grid of
//                           three blocks per SM: the host cuts the work into one run of equal cost per
//                           block (whole tiles of A; row ranges of the column chunks of B and C, cut
//                           on the boundaries of a pass of the eight warps), so the blocks finish
//                           together and a run is long enough to amortise its set-up; a block derives
//                           the challenges, builds small eq tables and cuts the weights it needs into
//                           limbs in shared memory -- no eq table or limb table ever reaches global
//                           memory
//   reduce_parts_kernel     sums the partial vectors into the two round tables of every proof (spread
//                           over all SMs: the partials are megabytes in L2), and the claim
//   sumcheck_kernel         the rounds, reading finished tables
// The kernels after the first are launched early (griddepcontrol.launch_dependents) and run their
// set-up while the one before drains; they read its results only after griddepcontrol.wait.
#pragma once

namespace imm {

__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// sum_{i < m} eq(r, i) over n-variable indices (variable 0 = top bit), m <= 2^n: walk the bits of m
// from the top; where m has a 1, every index that agrees with m above that bit and has a 0 there is
// below m, and the eq values of all completions of the lower bits add up to 1.
__device__ __forceinline__ uint64_t eq_prefix_sum(const uint64_t* r, int n, uint64_t m)
{
    if (m >= ((uint64_t)1 << n)) return 1;
    uint64_t acc = 1, s = 0;
    for (int t = 0; t < n; t++) {
        const uint64_t rt = r[t], omr = gl::sub(1, rt);
        if ((m >> (n - 1 - t)) & 1) { s = gl::add(s, gl::mul(acc, omr)); acc = gl::mul(acc, rt); }
        else acc = gl::mul(acc, omr);
    }
    return s;
}

// (sum of E_row over the real rows) * (sum of E_col over the real columns) of a proof whose eq tables
// were never written out: thread 0 and thread 32 evaluate the closed forms.  Block-wide call (two
// barriers); `scratch` holds two words; the result is valid in every thread.
__device__ __forceinline__ uint64_t offset_sums_closed_form(const ProofDev& pr, uint64_t* scratch)
{
    const int tid = threadIdx.x;
    if (tid == 0 || tid == 32) {
        const bool row = tid == 0;
        const int n = row ? pr.a : pr.c;
        const imm_fe* pt = row ? pr.pt_row : pr.pt_col;
        uint64_t r[MAX_EQ_VARS];
        for (int t = 0; t < n; t++) r[t] = pt ? pt[t] : gl::challenge(pr.seed, pr.proof_id, row ? 1u : 2u, (uint32_t)t);
        scratch[row ? 0 : 1] = eq_prefix_sum(r, n, (uint64_t)(row ? pr.m : pr.n));
    }
    __syncthreads();
    const uint64_t v = gl::mul(scratch[0], scratch[1]);
    __syncthreads();
    return v;
}

// eq(r, i) for i < 2^n as a product of three small tables over the high, middle and low index bits
// (variable 0 = top bit):  E[i] = t2[i >> (l0 + l1)] * t1[(i >> l0) & (2^l1 - 1)] * t0[i & (2^l0 - 1)],
// l0 = min(6, n) low bits, l1 = min(6, n - l0) middle bits, at most 8 high bits (n <= 20).  A block
// builds all three straight from the product definition (at most 8 multiplications per entry, all
// entries in parallel), whatever rows or columns it will need.
struct EqTables {
    uint64_t t0[64], t1[64], t2[256];
    int l0, l1;
};

__device__ __forceinline__ void eq_tables_build(EqTables& T, const uint64_t* r, const uint64_t* omr, int n)
{
    const int l0 = min(6, n), l1 = min(6, n - l0), l2 = n - l0 - l1;
    const int tid = threadIdx.x;                           // BYTEDOT_THREADS = 256 threads
    if (tid < (1 << l2)) T.t2[tid] = eq_product(r, omr, l2, (uint32_t)tid);
    if (tid < 64) { if (tid < (1 << l1)) T.t1[tid] = eq_product(r + l2, omr + l2, l1, (uint32_t)tid); }
    else if (tid < 128) { const int x = tid - 64; if (x < (1 << l0)) T.t0[x] = eq_product(r + l2 + l1, omr + l2 + l1, l0, (uint32_t)x); }
    if (tid == 0) { T.l0 = l0; T.l1 = l1; }
}

__device__ __forceinline__ uint64_t eq_tables_entry(const EqTables& T, uint32_t i)
{
    const int l0 = T.l0, l1 = T.l1;
    return gl::mul(gl::mul(T.t2[i >> (l0 + l1)], T.t1[(i >> l0) & ((1u << l1) - 1)]), T.t0[i & ((1u << l0) - 1)]);
}

#ifndef IMM_FUSED_MT_C
#define IMM_FUSED_MT_C 1
#endif
#ifndef IMM_FUSED_MT_B
#define IMM_FUSED_MT_B 1
#endif
// MMA row tiles (16 rows) per warp pass of the byte-dot code: one measured best for both kinds here (two
// spill registers for the claim at the 128 this kernel may use, and coarser cuts of the row ranges)
constexpr int FUSED_MT_C = IMM_FUSED_MT_C, FUSED_MT_B = IMM_FUSED_MT_B;
#ifndef IMM_FUSED_UNROLL
#define IMM_FUSED_UNROLL 1
#endif
constexpr int FUSED_UNROLL = IMM_FUSED_UNROLL;           // slabs of 256 byte-columns in flight per warp

struct FusedShared {
    union {
        uint4 sW[(BYTEDOT_MAX_CHUNK_BYTES / 256) * 128];  // B, C: weight limbs of the current column chunk (32 KiB)
        uint2 sR[MAX_TILE_ROWS];                          // A: weight limbs of the current tile's rows
    };
    uint64_t e_row[MAX_TILE_ROWS];                        // C: E_row of the rows in hand (a segment goes in pieces of this many)
    EqTables row, col;                                    // eq(r_row, .), eq(r_col, .) of the current job
    uint64_t hm[64];                                      // col.t2[high] * col.t1[.] for the current chunk (its high bits are fixed)
    uint64_t r[2][MAX_EQ_VARS], omr[2][MAX_EQ_VARS];
};

// Four consecutive column weights of the current chunk (absolute indices i0 .. i0 + 3, all inside one
// aligned block of 4096): one multiplication each; zero at or past `extent`.
__device__ __forceinline__ void chunk_quad(const FusedShared& sh, uint32_t i0, int64_t extent, uint64_t (&w)[4])
{
    const int l0 = sh.col.l0, l1 = sh.col.l1;
#pragma unroll
    for (int v = 0; v < 4; v++) {
        const uint32_t i = i0 + v;
        w[v] = (int64_t)i < extent ? gl::mul(sh.hm[(i >> l0) & ((1u << l1) - 1)], sh.col.t0[i & ((1u << l0) - 1)]) : 0;
    }
}

__global__ void __launch_bounds__(BYTEDOT_THREADS, FUSED_BLOCKS_PER_SM)
fused_contract_kernel(const FusedJob* jobs, const FusedSeg* segs, const uint32_t* block_first)
{
    __shared__ FusedShared sh;
    pdl_launch_dependents();                               // the next kernel may start its set-up
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t seg_begin = block_first[blockIdx.x], seg_end = block_first[blockIdx.x + 1];
    int cur_job = -1, cur_cci = -1;
    for (uint32_t si = seg_begin; si < seg_end; si++) {
        const FusedSeg seg = segs[si];
        const FusedJob* fj = jobs + seg.job;
        const MatJob job = fj->mj;
        const int kind = fj->kind;
        if (seg.job != cur_job) {
            // the challenges of this job and the eq tables of the axes it weighs
            __syncthreads();                               // the tables may still be read (previous segment)
            const bool need_row = kind != JOB_COLBIND, need_col = kind != JOB_ROWBIND;
            if (need_row && tid < fj->a) {
                const uint64_t r = fj->pt_row ? fj->pt_row[tid] : gl::challenge(fj->seed, fj->proof_id, 1u, (uint32_t)tid);
                sh.r[0][tid] = r; sh.omr[0][tid] = gl::sub(1, r);
            }
            if (need_col && tid >= 32 && tid < 32 + fj->c) {
                const int t = tid - 32;
                const uint64_t r = fj->pt_col ? fj->pt_col[t] : gl::challenge(fj->seed, fj->proof_id, 2u, (uint32_t)t);
                sh.r[1][t] = r; sh.omr[1][t] = gl::sub(1, r);
            }
            __syncthreads();
            if (need_row) eq_tables_build(sh.row, sh.r[0], sh.omr[0], fj->a);
            if (need_col) eq_tables_build(sh.col, sh.r[1], sh.omr[1], fj->c);
            cur_job = seg.job;
            cur_cci = -1;
            // (the barrier that publishes the tables is the first one below)
        }

        if (kind == JOB_ROWBIND) {
            // weight limbs of the tile's rows, in the fragment order of the row-binding MMA (see eq_batch_kernel)
            __syncthreads();                               // tables ready; sR no longer read
            const int rbi = seg.cci / job.ncc;
            const int r0 = rbi * job.tile_rows;
            const int nrows = min(job.tile_rows, job.rows - r0);
            uint32_t* dst = reinterpret_cast<uint32_t*>(sh.sR);
            for (int u = tid; u < ((nrows + 31) / 32) * 8; u += BYTEDOT_THREADS) {
                const int i0 = 4 * u;
                uint64_t w[4];
#pragma unroll
                for (int v = 0; v < 4; v++) w[v] = r0 + i0 + v < job.rows ? eq_tables_entry(sh.row, (uint32_t)(r0 + i0 + v)) : 0;
                uint32_t limb[8];
                limbs_of4(w, limb);
                const int G = i0 >> 5, h = (i0 >> 4) & 1, t = (i0 >> 2) & 3;
#pragma unroll
                for (int g = 0; g < 8; g++) dst[G * 64 + (4 * g + t) * 2 + h] = limb[g];
            }
            __syncthreads();
            if (job.vec) rowmma_tile<true, false, true>(job, (uint32_t)seg.cci, sh.sR);
            else rowmma_tile<false, false, true>(job, (uint32_t)seg.cci, sh.sR);
            cur_cci = -1;
            continue;
        }

        const bool point = kind == JOB_POINT;
        if (seg.cci != cur_cci) {
            // weight limbs of the chunk's byte-columns; the chunk lies inside one aligned block of 4096
            // columns, so the high table entry is one value, folded into the middle table first
            __syncthreads();                               // tables ready; sW no longer read
            const int64_t cb0 = (int64_t)seg.cci * job.chunk;
            const uint32_t c0e = (uint32_t)(point ? cb0 / 4 : cb0);            // first column of the chunk
            if (tid < 64) sh.hm[tid] = tid < (1 << sh.col.l1) ? gl::mul(sh.col.t2[c0e >> (sh.col.l0 + sh.col.l1)], sh.col.t1[tid]) : 0;
            __syncthreads();
            const int64_t row_bytes = (int64_t)job.cols * (point ? 4 : 1);
            const int nslab = (int)min((int64_t)(job.chunk / 256), (row_bytes - cb0 + 255) / 256);
            if (!point) {
                uint32_t* dst = reinterpret_cast<uint32_t*>(sh.sW);
                for (int u = tid; u < nslab * 64; u += BYTEDOT_THREADS) {     // 64 quads per slab of 256 columns
                    const int i0 = 4 * u;
                    uint64_t w[4];
                    chunk_quad(sh, c0e + (uint32_t)i0, job.cols, w);
                    uint32_t limb[8];
                    limbs_of4(w, limb);
                    const int sl = i0 >> 8, t = (i0 >> 6) & 3, piece = (i0 >> 4) & 3, q = (i0 >> 2) & 3;
#pragma unroll
                    for (int g = 0; g < 8; g++) dst[((sl * 4 + piece) * 32 + 4 * g + t) * 4 + q] = limb[g];
                }
            } else {
                // column j weighs its four bytes by e, e 2^8, e 2^16, e 2^24
                for (int u = tid; u < nslab * 16; u += BYTEDOT_THREADS) {     // 16 quads per slab of 64 columns
                    const int i0 = 4 * u;
                    uint64_t w[4];
                    chunk_quad(sh, c0e + (uint32_t)i0, job.cols, w);
                    uint32_t word[8][4];
#pragma unroll
                    for (int v = 0; v < 4; v++) {
                        const uint64_t shv[4] = {w[v], gl::shl(w[v], 8), gl::shl(w[v], 16), gl::shl(w[v], 24)};
                        uint32_t limb[8];
                        limbs_of4(shv, limb);
#pragma unroll
                        for (int g = 0; g < 8; g++) word[g][v] = limb[g];
                    }
                    const int sl = i0 >> 6, t = (i0 >> 4) & 3, piece = (i0 >> 2) & 3;
#pragma unroll
                    for (int g = 0; g < 8; g++)
                        sh.sW[(sl * 4 + piece) * 32 + 4 * g + t] = make_uint4(word[g][0], word[g][1], word[g][2], word[g][3]);
                }
            }
            __syncthreads();
            cur_cci = seg.cci;
        }
        if (point) {
            // the rows' weights are staged once per piece (all threads, two multiplications per row) rather
            // than formed by the few lanes that hold a row's result at the end of every pass
            uint64_t part = 0;
            for (int p0 = seg.r0; p0 < seg.r1; p0 += MAX_TILE_ROWS) {
                const int p1 = min(p0 + MAX_TILE_ROWS, seg.r1);
                __syncthreads();                           // whoever read e_row before (a piece, a segment) is done
                for (int x = tid; x < p1 - p0; x += BYTEDOT_THREADS) sh.e_row[x] = eq_tables_entry(sh.row, (uint32_t)(p0 + x));
                __syncthreads();
                const uint64_t* er = sh.e_row;
                auto row_weight = [er, p0](int row) { return er[row - p0]; };
                if (job.vec == 2) part = gl::add(part, bytedot_rows<true, true, 2, FUSED_MT_C, FUSED_UNROLL>(job, seg.cci, p0, p1, sh.sW, row_weight));
                else if (job.vec == 1) part = gl::add(part, bytedot_rows<true, true, 1, FUSED_MT_C, FUSED_UNROLL>(job, seg.cci, p0, p1, sh.sW, row_weight));
                else part = gl::add(part, bytedot_rows<true, true, 0, FUSED_MT_C, FUSED_UNROLL>(job, seg.cci, p0, p1, sh.sW, row_weight));
            }
            part = warp_sum_fe(part);
            if (lane == 0) job.out[(int64_t)((int)si - fj->seg0) * (BYTEDOT_THREADS / 32) + warp] = part;
        } else {
            auto none = [](int) { return (uint64_t)0; };
            if (job.vec == 2) bytedot_rows<false, false, 2, FUSED_MT_B, FUSED_UNROLL>(job, seg.cci, seg.r0, seg.r1, sh.sW, none);
            else if (job.vec == 1) bytedot_rows<false, false, 1, FUSED_MT_B, FUSED_UNROLL>(job, seg.cci, seg.r0, seg.r1, sh.sW, none);
            else bytedot_rows<false, false, 0, FUSED_MT_B, FUSED_UNROLL>(job, seg.cci, seg.r0, seg.r1, sh.sW, none);
        }
    }
}

// Both round tables of every proof from the partial vectors (entry y of table a = sum over the row
// blocks of A of their partial avec[y], likewise b over the column chunks of B; zero from k up to
// 2^b), and the claim c0 from the partial sums of C.  Grid: (blocks of 256 entries of the largest
// table + 1, proofs); the extra block of a proof forms its claim.
constexpr int REDUCE_THREADS = 256;

__global__ void __launch_bounds__(REDUCE_THREADS) reduce_parts_kernel(const ProofDev* proofs)
{
    __shared__ uint64_t red[33];
    __shared__ uint64_t off[2];
    pdl_launch_dependents();
    const ProofDev pr = proofs[blockIdx.y];                // (the header is not written by the kernel before)
    const int n0 = 1 << pr.b;
    const int nblk = (n0 + REDUCE_THREADS - 1) / REDUCE_THREADS;
    const int tid = threadIdx.x;
    if ((int)blockIdx.x > nblk) return;
    if ((int)blockIdx.x == nblk) {
        // the claim; its offset needs only the challenges, so it is ready before the partial sums are
        uint64_t offset = 0;
        if (pr.c_offset) offset = gl::shl(offset_sums_closed_form(pr, off), 31);
        pdl_wait();
        uint64_t s = 0;
        int i = tid;
        for (; i + 7 * REDUCE_THREADS < pr.n_part_c; i += 8 * REDUCE_THREADS) {
            uint64_t v[8];
#pragma unroll
            for (int u = 0; u < 8; u++) v[u] = __ldcg(pr.part_c + i + u * REDUCE_THREADS);
#pragma unroll
            for (int u = 0; u < 8; u++) s = gl::add(s, v[u]);
        }
        for (; i < pr.n_part_c; i += REDUCE_THREADS) s = gl::add(s, __ldcg(pr.part_c + i));
        s = block_sum_fe(s, red);
        if (tid == 0) *pr.c0_ready = gl::sub(s, offset);
        return;
    }
    pdl_wait();
    const int y = blockIdx.x * REDUCE_THREADS + tid;
    if (y < n0) {
        const bool live = y < pr.k;                        // entries past k are the zero padding
        pr.tab[y] = live ? sum_parts_at(pr.part_a, pr.n_part_a, pr.k, y) : 0;
        pr.tab[n0 + y] = live ? sum_parts_at(pr.part_b, pr.n_part_b, pr.k, y) : 0;
    }
}

}  // namespace imm
