// Tensor-core contraction kernels (included by imm_kernels.cu after the shared device helpers).
//
// The eq-vector x matrix products are dense contractions once the 64-bit weight is cut into
// eight unsigned 8-bit limbs:  sum_q d[q] * W[q] = sum_l 2^(8l) * (sum_q d[q] * limb_l(W[q])).
// The inner sums are int8 x uint8 dot products with 32-bit accumulation, i.e. an integer MMA
// with the eight limbs as its N dimension (m16n8k32).  Each accumulator is rebuilt into a
// 128-bit integer and reduced mod p once per output.  Matrix bytes go global -> registers ->
// MMA with no shared-memory round trip; only the (tiny, reused) weight limbs are staged.
#pragma once

namespace imm {

// D += A(16x32, row) * B(32x8, col), 32-bit accumulators.  SIGNED_A: matrix bytes are int8,
// otherwise uint8; the weight limbs are always uint8.
template <bool SIGNED_A>
__device__ __forceinline__ void mma_m16n8k32(int32_t (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                             uint32_t a3, uint32_t b0, uint32_t b1)
{
    if constexpr (SIGNED_A) {
        asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    } else {
        asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                     : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                     : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    }
}

// A thread of the MMA holds limbs 2t and 2t+1 (t = lane % 4) of one output.  Rebuild
// 2^(16t) * (lo + 2^8 hi), add the four threads' shares; valid in all four lanes.
__device__ __forceinline__ uint64_t combine_limbs(int32_t lo, int32_t hi, int t)
{
    uint64_t v = gl::from_i64((int64_t)lo + ((int64_t)hi << 8));
    v = gl::shl(v, 16 * t);
    v = gl::add(v, shfl_xor_u64(v, 1));
    v = gl::add(v, shfl_xor_u64(v, 2));
    return v;
}

// ------------------------------------------------------------------------------------------
// eq tables of a batch and the limb tables of the weights, in fragment order
// ------------------------------------------------------------------------------------------
// W_COLS_*: weights of byte-columns.  Units of 256 byte-columns ("slabs"); a lane (4g + t) of
//   the byte-dot kernel owns bytes 64t..64t+63 of a slab, and its 64 weight bytes are limb g of
//   W[256s + 64t + 0..63].  They are stored as four 16-byte pieces, piece-major
//   ([slab][piece][lane]) so that a warp's 16-byte reads are conflict-free.
//   int8 matrix:  W[q] = eq[q].   int32 matrix seen as bytes: W[4j + b] = eq[j] * 2^(8b) mod p.
// W_ROWS: weights of rows for the transposed (row-binding) MMA.  Units of 32 rows; lane = 4g+t
//   holds 8 bytes: byte u of word h is limb g of eq[32G + 16h + 4t + u].
// Weights past the real extent are zero (the implicit zero padding).
//
// One block fills a slice of one table.  E[i] = hi[i >> nlo] * lo[i & (2^nlo - 1)] with the two
// small tables built per block straight from the product definition (no barriers beyond one).
// A thread produces four consecutive entries and, from the same registers, their words of the
// limb tables: byte g of four 32-bit halves is a 4x4 byte transpose.

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

// rows r0..r3 of a 4x4 byte block -> columns c0..c3
__device__ __forceinline__ void transpose4x4(uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3,
                                             uint32_t& c0, uint32_t& c1, uint32_t& c2, uint32_t& c3)
{
    const uint32_t x0 = prmt(r0, r1, 0x5140), x1 = prmt(r0, r1, 0x7362);
    const uint32_t y0 = prmt(r2, r3, 0x5140), y1 = prmt(r2, r3, 0x7362);
    c0 = prmt(x0, y0, 0x5410); c1 = prmt(x0, y0, 0x7632);
    c2 = prmt(x1, y1, 0x5410); c3 = prmt(x1, y1, 0x7632);
}

// limb[g], g = 0..7: byte v of limb[g] is byte g of w[v]
__device__ __forceinline__ void limbs_of4(const uint64_t (&w)[4], uint32_t (&limb)[8])
{
    transpose4x4((uint32_t)w[0], (uint32_t)w[1], (uint32_t)w[2], (uint32_t)w[3], limb[0], limb[1], limb[2], limb[3]);
    transpose4x4((uint32_t)(w[0] >> 32), (uint32_t)(w[1] >> 32), (uint32_t)(w[2] >> 32), (uint32_t)(w[3] >> 32),
                 limb[4], limb[5], limb[6], limb[7]);
}

// eq(r, x) over `cnt` variables r[0..cnt), variable 0 = top bit of x
__device__ __forceinline__ uint64_t eq_product(const uint64_t* r, const uint64_t* one_minus_r, int cnt, uint32_t x)
{
    uint64_t v = 1;
    for (int t = 0; t < cnt; t++) v = gl::mul(v, ((x >> (cnt - 1 - t)) & 1) ? r[t] : one_minus_r[t]);
    return v;
}

__global__ void __launch_bounds__(EQ_BATCH_THREADS) eq_batch_kernel(const EqTask* tasks)
{
    __shared__ uint64_t r_sh[MAX_EQ_VARS], omr_sh[MAX_EQ_VARS];
    __shared__ uint64_t lo_t[1024], hi_t[1024];
    const EqTask tk = tasks[blockIdx.y];
    const bool from_table = tk.given != nullptr;
    const int64_t total = from_table ? (int64_t)tk.extent : (int64_t)1 << tk.nvars;
    // entries this task has to cover: the table itself, and the limb tables' zero padding
    const int64_t pad = tk.w_rows ? 32 : 256;
    const int64_t cover = (tk.w_rows || tk.w_cols_i8 || tk.w_cols_i32)
                              ? max(total, ((int64_t)tk.extent + pad - 1) / pad * pad) : total;
    const int64_t q0 = (int64_t)blockIdx.x * EQ_SLICE_QUADS;
    if (4 * q0 >= cover) return;
    __shared__ uint64_t red[33];
    uint64_t slice_sum = 0;

    const int nlo = (tk.nvars + 1) / 2, nhi = tk.nvars - nlo;
    if (!from_table) {                                 // (uniform over the block)
        if ((int)threadIdx.x < tk.nvars) {
            const uint64_t r = tk.point ? tk.point[threadIdx.x]
                                        : gl::challenge(tk.seed, tk.proof_id, tk.domain, threadIdx.x);
            r_sh[threadIdx.x] = r;
            omr_sh[threadIdx.x] = gl::sub(1, r);
        }
        __syncthreads();
        for (int x = threadIdx.x; x < (1 << nhi); x += EQ_BATCH_THREADS) hi_t[x] = eq_product(r_sh, omr_sh, nhi, x);
        for (int x = threadIdx.x; x < (1 << nlo); x += EQ_BATCH_THREADS) lo_t[x] = eq_product(r_sh + nhi, omr_sh + nhi, nlo, x);
        __syncthreads();
    }
    const uint32_t mask = (1u << nlo) - 1;

    const int64_t q1 = min(q0 + EQ_SLICE_QUADS, (cover + 3) / 4);
    for (int64_t u = q0 + threadIdx.x; u < q1; u += EQ_BATCH_THREADS) {
        const int64_t i0 = 4 * u;
        uint64_t w[4];
#pragma unroll
        for (int v = 0; v < 4; v++) {
            const int64_t i = i0 + v;
            uint64_t e = 0;
            if (i < total) {
                if (from_table) e = tk.given[i];
                else { e = gl::mul(hi_t[i >> nlo], lo_t[(uint32_t)i & mask]); tk.out[i] = e; }
            }
            w[v] = i < tk.extent ? e : 0;
            slice_sum = gl::add(slice_sum, w[v]);
        }
        uint32_t limb[8];
        if (tk.w_rows && i0 < ((int64_t)tk.extent + 31) / 32 * 32) {
            limbs_of4(w, limb);
            const int64_t G = i0 >> 5;
            const int h = (int)(i0 >> 4) & 1, t = (int)(i0 >> 2) & 3;
#pragma unroll
            for (int g = 0; g < 8; g++) tk.w_rows[G * 64 + (4 * g + t) * 2 + h] = limb[g];
        }
        if (tk.w_cols_i8 && i0 < ((int64_t)tk.extent + 255) / 256 * 256) {
            limbs_of4(w, limb);
            const int64_t sl = i0 >> 8;
            const int t = (int)(i0 >> 6) & 3, piece = (int)(i0 >> 4) & 3, r = (int)(i0 >> 2) & 3;
#pragma unroll
            for (int g = 0; g < 8; g++) tk.w_cols_i8[((sl * 4 + piece) * 32 + 4 * g + t) * 4 + r] = limb[g];
        }
        if (tk.w_cols_i32 && i0 < ((int64_t)tk.extent + 63) / 64 * 64) {
            // column j = i0 + v weighs its four bytes by e, e 2^8, e 2^16, e 2^24; its words sit at
            // position v of a 16-byte piece, so the quad fills one piece per limb
            uint32_t word[8][4];
#pragma unroll
            for (int v = 0; v < 4; v++) {
                const uint64_t sh[4] = {w[v], gl::shl(w[v], 8), gl::shl(w[v], 16), gl::shl(w[v], 24)};
                limbs_of4(sh, limb);
#pragma unroll
                for (int g = 0; g < 8; g++) word[g][v] = limb[g];
            }
            const int64_t sl = i0 >> 6;
            const int t = (int)(i0 >> 4) & 3, piece = (int)(i0 >> 2) & 3;
            uint4* dst = reinterpret_cast<uint4*>(tk.w_cols_i32);
#pragma unroll
            for (int g = 0; g < 8; g++)
                dst[(sl * 4 + piece) * 32 + 4 * g + t] = make_uint4(word[g][0], word[g][1], word[g][2], word[g][3]);
        }
    }
    if (tk.slice_sums) {                       // (uniform over the block)
        slice_sum = block_sum_fe(slice_sum, red);
        if (threadIdx.x == 0) tk.slice_sums[blockIdx.x] = slice_sum;
    }
}

// ------------------------------------------------------------------------------------------
// byte-dot kernel:  u[i] = sum_q byte(M[i], q) * W[q]   (contraction along the contiguous index)
// ------------------------------------------------------------------------------------------
// Serves the column binding of int8 B (W = eq_col) and the claim on int32 C seen as an
// m x 4n byte matrix (W[4j+b] = eq_col[j] 2^(8b)).  For int32 the top byte of every word is
// flipped (x ^ 0x80000000) so that all four bytes are unsigned; every entry then reads 2^31 too
// high, which the consumer of the partial sums undoes once per matrix by subtracting
// 2^31 * (sum of the row weights) * (sum of the column weights).
//   POINT = false (int8 only): out[chunk][row] = u[row]      (partial over this column chunk)
//   POINT = true : out[tile][warp] = sum over the warp's rows of eq_row[row] * u[row]
// One tile = tile_rows rows x job.chunk byte-columns (chosen per batch: wide for large inputs, narrow
// so that small ones still spread over all SMs).  A warp sweeps 16*MT rows (MT MMA
// row tiles) across the chunk in slabs of 256 byte-columns; within a slab a thread owns 64
// CONTIGUOUS bytes of each of its 2*MT rows (two 256-bit loads), so four neighbouring lanes read
// 256 contiguous bytes of a row -- measured to stream at the rate of a linear read, where
// 64-byte pieces per row lose 15 %.  Which byte-column lands in which MMA k-slot is free as long
// as the weight limbs are laid out the same way (weights_kernel does that).

struct u32x8 { uint32_t v[8]; };

__device__ __forceinline__ u32x8 ld_stream_v8(const void* p)          // 256-bit streaming load, 32-byte aligned
{
    u32x8 r;
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]), "=r"(r.v[5]),
                   "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}

// 64 bytes of one row starting at p; `left` = bytes of the row from p on (may be <= 0).
// VL 2: rows 32-byte aligned, VL 1: 16-byte aligned, VL 0: element-wise loads.
template <typename T, int VL>
__device__ __forceinline__ void load64(const char* p, int64_t left, uint32_t (&d)[16])
{
    if (VL == 2 && left >= 64) {
        const u32x8 a = ld_stream_v8(p), b = ld_stream_v8(p + 32);
#pragma unroll
        for (int i = 0; i < 8; i++) { d[i] = a.v[i]; d[8 + i] = b.v[i]; }
        return;
    }
#pragma unroll
    for (int i = 0; i < 4; i++) {
        const int64_t l = left - 16 * i;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (l > 0) v = load_vec<T, (VL >= 1)>(p + 16 * i, l >= 16, (int)(min((int64_t)16, l) / (int64_t)sizeof(T)));
        d[4 * i] = v.x; d[4 * i + 1] = v.y; d[4 * i + 2] = v.z; d[4 * i + 3] = v.w;
    }
}

// Rows [r0, r1) of column chunk cci of one matrix, by one block: every warp takes 16*MT rows at a
// time across the chunk's slabs; sW holds the chunk's weight limbs.  POINT: returns this thread's
// share of sum_row row_weight(row) * u[row] (to be summed over the warp by the caller);
// otherwise writes u[row] to job.out[cci][row] and returns 0.
template <bool I32, bool POINT, int VL, int MT, int UNROLL = BYTEDOT_UNROLL, class RowWeight>
__device__ __forceinline__ uint64_t bytedot_rows(const MatJob& job, int cci, int r0, int r1, const uint4* sW, RowWeight row_weight)
{
    static_assert(POINT || !I32, "the int32 byte view is offset by 2^31 per entry: point evaluation only");
    using T = typename std::conditional<I32, int32_t, int8_t>::type;
    constexpr int ESZ = (int)sizeof(T);
    constexpr int NWARP = BYTEDOT_THREADS / 32;
    const int64_t row_bytes = (int64_t)job.cols * ESZ;
    const int64_t cb0 = (int64_t)cci * job.chunk;
    const int nslab = (int)min((int64_t)(job.chunk / 256), (row_bytes - cb0 + 255) / 256);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int64_t pitch = job.ld * (int64_t)ESZ;
    uint64_t part = 0;
    for (int rg = r0 + warp * (16 * MT); rg < r1; rg += NWARP * (16 * MT)) {
        int32_t acc[MT][4];
        const char* p[MT][2];
#pragma unroll
        for (int mt = 0; mt < MT; mt++) {
#pragma unroll
            for (int c = 0; c < 4; c++) acc[mt][c] = 0;
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const int row = min(rg + 16 * mt + g + 8 * h, r1 - 1);     // clamped: never out of bounds
                p[mt][h] = (const char*)job.mat + (int64_t)row * pitch + cb0 + 64 * t;
            }
        }
#pragma unroll UNROLL
        for (int s = 0; s < nslab; s++) {
            const int64_t left = row_bytes - (cb0 + 256 * s + 64 * t);    // bytes of the row from this thread's piece on
            uint32_t d[MT][2][16];
#pragma unroll
            for (int mt = 0; mt < MT; mt++)
#pragma unroll
                for (int h = 0; h < 2; h++) load64<T, VL>(p[mt][h] + 256 * s, left, d[mt][h]);
            uint4 w[4];
#pragma unroll
            for (int i = 0; i < 4; i++) w[i] = sW[(s * 4 + i) * 32 + lane];
#pragma unroll
            for (int mt = 0; mt < MT; mt++) {
                if (I32) {
#pragma unroll
                    for (int i = 0; i < 16; i++) { d[mt][0][i] ^= 0x80000000u; d[mt][1][i] ^= 0x80000000u; }
                }
#pragma unroll
                for (int i = 0; i < 4; i++) {        // 16-byte piece i feeds two MMAs
                    mma_m16n8k32<!I32>(acc[mt], d[mt][0][4 * i], d[mt][1][4 * i], d[mt][0][4 * i + 1],
                                       d[mt][1][4 * i + 1], w[i].x, w[i].y);
                    mma_m16n8k32<!I32>(acc[mt], d[mt][0][4 * i + 2], d[mt][1][4 * i + 2], d[mt][0][4 * i + 3],
                                       d[mt][1][4 * i + 3], w[i].z, w[i].w);
                }
            }
        }
        // every lane of a group of four holds u; the rows' products (or stores) are shared out over the four
#pragma unroll
        for (int mt = 0; mt < MT; mt++)
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const int row = rg + 16 * mt + g + 8 * h;
                uint64_t u = combine_limbs(acc[mt][2 * h], acc[mt][2 * h + 1], t);
                if (t == ((2 * mt + h) & 3) && row < r1) {
                    if (POINT) part = gl::add(part, gl::mul(row_weight(row), u));
                    else job.out[(int64_t)cci * job.rows + row] = u;
                }
            }
    }
    return part;
}

// One tile = rows [rbi * tile_rows, ...) of chunk cci: stages the chunk's weight limbs from job.wtab
// and takes the row weights from job.eq_row.
template <bool I32, bool POINT, int VL, int MT>
__device__ __forceinline__ void bytedot_tile(const MatJob& job, uint32_t local, uint4* sW)
{
    constexpr int ESZ = I32 ? 4 : 1;
    constexpr int NWARP = BYTEDOT_THREADS / 32;
    const int rbi = local / job.ncc, cci = local % job.ncc;
    const int r0 = rbi * job.tile_rows;
    const int r1 = min(r0 + job.tile_rows, job.rows);
    const int64_t row_bytes = (int64_t)job.cols * ESZ;
    const int64_t cb0 = (int64_t)cci * job.chunk;
    const int nslab = (int)min((int64_t)(job.chunk / 256), (row_bytes - cb0 + 255) / 256);
    const uint4* wsrc = reinterpret_cast<const uint4*>(job.wtab) + (cb0 / 256) * 128;
    for (int i = threadIdx.x; i < nslab * 128; i += BYTEDOT_THREADS) sW[i] = wsrc[i];
    __syncthreads();
    const imm_fe* erow = job.eq_row;
    uint64_t part = bytedot_rows<I32, POINT, VL, MT, BYTEDOT_UNROLL>(job, cci, r0, r1, sW, [erow](int row) { return erow[row]; });
    if (POINT) {                               // one partial per warp: no block barrier at the end of a tile
        part = warp_sum_fe(part);
        if ((threadIdx.x & 31) == 0) job.out[(int64_t)local * NWARP + (threadIdx.x >> 5)] = part;
    }
}

// MT = MMA row tiles (16 rows each) a warp carries per pass: more rows in flight per thread
// against more registers (three resident blocks per SM with one row tile, two with two).
template <bool I32, bool POINT, int MT>
__global__ void __launch_bounds__(BYTEDOT_THREADS, MT == 1 ? 3 : 2) bytedot_kernel(const MatJob* jobs, int njobs)
{
    __shared__ uint4 sW[(BYTEDOT_MAX_CHUNK_BYTES / 256) * 128];     // up to 32 KiB of weight limbs
    const MatJob job = jobs[find_job(jobs, njobs, blockIdx.x)];
    const uint32_t local = blockIdx.x - job.tile0;
    if (job.vec == 2) bytedot_tile<I32, POINT, 2, MT>(job, local, sW);
    else if (job.vec == 1) bytedot_tile<I32, POINT, 1, MT>(job, local, sW);
    else bytedot_tile<I32, POINT, 0, MT>(job, local, sW);
}

// ------------------------------------------------------------------------------------------
// row-binding MMA kernel (int8):  out[y] = sum_i eq_row[i] * M[i,y]
// ------------------------------------------------------------------------------------------
// The contraction runs along the strided index, so the MMA's K dimension is the row index and
// its M dimension the column index: each thread loads 16 columns of 8 rows (coalesced 16-byte
// loads, a warp reads 128 contiguous bytes of each row) and transposes 4x4 byte blocks in
// registers with byte permutes so that every register holds one column at four consecutive
// rows.  One tile = tile_rows rows x (128 columns per warp of the block); the block size is chosen
// per batch (8 warps for large inputs, fewer so that small ones still spread over all SMs).

// STAGE: copy the tile's weight limbs from job.wtab into sR; otherwise the caller has filled sR
// (and synchronised).
// SPLIT: a tile narrower than the block (k below 128 columns per warp, e.g. an attention head's Q) leaves
// warps without columns; they then share the rows instead -- warp w takes column group w % ncw and every
// (8 / ncw)-th group of 32 rows -- and the partial column sums meet in shared memory (sR, once the loop is done).
template <bool VEC, bool STAGE = true, bool SPLIT = false>
__device__ __forceinline__ void rowmma_tile(const MatJob& job, uint32_t local, uint2* sR)
{
    const int rbi = local / job.ncc, cci = local % job.ncc;
    const int r0 = rbi * job.tile_rows;                         // multiple of 32
    const int r1 = min(r0 + job.tile_rows, job.rows);
    const int ngroups = (r1 - r0 + 31) / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;

    if (STAGE) {
        const uint2* wsrc = reinterpret_cast<const uint2*>(job.wtab) + (int64_t)(r0 / 32) * 32;
        for (int i = threadIdx.x; i < ngroups * 32; i += blockDim.x) sR[i] = wsrc[i];
        __syncthreads();
    }

    const int tile_cols = (int)blockDim.x * 4;                    // 128 columns per warp
    int cw = warp, rw = 0, rs = 1, ncw = (int)blockDim.x >> 5;
    if (SPLIT) {
        const int need = (min(tile_cols, job.cols - cci * tile_cols) + 127) >> 7;     // warps that have columns
        ncw = 1;
        while (ncw < need) ncw <<= 1;
        rs = ((int)blockDim.x >> 5) / ncw;
        cw = warp % ncw;
        rw = warp / ncw;
    }
    const int col = cci * tile_cols + cw * 128 + 16 * g;          // this thread's 16 columns
    const int nvalid = min(16, job.cols - col);
    const bool full = nvalid == 16;
    int32_t acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
        for (int c = 0; c < 4; c++) acc[i][c] = 0;

    if (cw * 128 + cci * tile_cols < job.cols) {                // whole warp in or out
        for (int G = rw; G < ngroups; G += rs) {
            uint4 d[2][4];
#pragma unroll
            for (int h = 0; h < 2; h++)
#pragma unroll
                for (int u = 0; u < 4; u++) {
                    const int row = min(r0 + 32 * G + 16 * h + 4 * t + u, r1 - 1);   // clamped; its weight is 0 past r1
                    const char* p = (const char*)job.mat + (int64_t)row * job.ld + col;
                    d[h][u] = nvalid > 0 ? load_vec<int8_t, VEC>(p, full, nvalid) : make_uint4(0, 0, 0, 0);
                }
            const uint2 wb = sR[G * 32 + lane];
            uint32_t T[2][16];
#pragma unroll
            for (int h = 0; h < 2; h++) {
                transpose4x4(d[h][0].x, d[h][1].x, d[h][2].x, d[h][3].x, T[h][0], T[h][1], T[h][2], T[h][3]);
                transpose4x4(d[h][0].y, d[h][1].y, d[h][2].y, d[h][3].y, T[h][4], T[h][5], T[h][6], T[h][7]);
                transpose4x4(d[h][0].z, d[h][1].z, d[h][2].z, d[h][3].z, T[h][8], T[h][9], T[h][10], T[h][11]);
                transpose4x4(d[h][0].w, d[h][1].w, d[h][2].w, d[h][3].w, T[h][12], T[h][13], T[h][14], T[h][15]);
            }
#pragma unroll
            for (int i = 0; i < 8; i++)
                mma_m16n8k32<true>(acc[i], T[0][2 * i], T[0][2 * i + 1], T[1][2 * i], T[1][2 * i + 1], wb.x, wb.y);
        }
    }
    // MMA i: row-slot g is column col + 2i, row-slot g+8 is column col + 2i + 1
    if (SPLIT && rs > 1) {
        __syncthreads();                                        // every warp is done with the weights in sR
        uint64_t* red = reinterpret_cast<uint64_t*>(sR);        // [warp][128 columns]: 8 KiB, the size of sR
#pragma unroll
        for (int i = 0; i < 8; i++)
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const uint64_t v = combine_limbs(acc[i][2 * h], acc[i][2 * h + 1], t);
                if (t == 0) red[warp * 128 + 16 * g + 2 * i + h] = v;
            }
        __syncthreads();
        if (rw == 0 && t == 0) {
#pragma unroll
            for (int i = 0; i < 8; i++)
#pragma unroll
                for (int h = 0; h < 2; h++) {
                    const int c = col + 2 * i + h;
                    if (c < job.cols) {
                        uint64_t v = 0;
                        for (int r = 0; r < rs; r++) v = gl::add(v, red[(r * ncw + cw) * 128 + 16 * g + 2 * i + h]);
                        job.out[(int64_t)rbi * job.cols + c] = v;
                    }
                }
        }
        return;                                                 // (the caller synchronises before it refills sR)
    }
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
        for (int h = 0; h < 2; h++) {
            uint64_t v = combine_limbs(acc[i][2 * h], acc[i][2 * h + 1], t);
            const int c = col + 2 * i + h;
            if (t == 0 && c < job.cols) job.out[(int64_t)rbi * job.cols + c] = v;
        }
}

// Aligned rows: the byte transpose moves from the integer pipe (64 byte-permutes per 128 loaded
// bytes: the kernel above is bound by them) into the load path.  A warp streams its 128 columns
// through a ring of shared-memory stages with 16-byte asynchronous copies (a stage = 32 rows x
// 128 bytes, rows padded to 144 bytes so that ldmatrix is conflict-free); `ldmatrix ... .trans .b8`
// then delivers 16 x 16 byte blocks transposed, i.e. every register holds one column at four
// consecutive rows -- exactly the MMA's A fragment with K = rows:
//   lane 4g+t gets {M[4t..4t+3][g]}, {M[4t..4t+3][g+8]} of rows 0-15 and of rows 16-31  ->  a0..a3.
// MMA j of a group covers columns 16j..16j+15 of the warp; accumulator rows g / g+8 are columns
// 16j+g / 16j+g+8.  The ring belongs to the warp, so the loop needs warp barriers only.

__device__ __forceinline__ void cp_async_16(uint32_t smem_dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(smem_dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x2_trans_b8(uint32_t (&r)[4], uint32_t smem_row)
{
    asm volatile("ldmatrix.sync.aligned.m16n16.x2.trans.shared.b8 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_row));
}

__device__ __forceinline__ void rowldm_tile(const MatJob& job, uint32_t local, uint2* sR, char* ring_base)
{
    const int rbi = local / job.ncc, cci = local % job.ncc;
    const int r0 = rbi * job.tile_rows;                         // multiple of 32
    const int r1 = min(r0 + job.tile_rows, job.rows);
    const int ngroups = (r1 - r0 + 31) / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;

    const uint2* wsrc = reinterpret_cast<const uint2*>(job.wtab) + (int64_t)(r0 / 32) * 32;
    for (int i = threadIdx.x; i < ngroups * 32; i += blockDim.x) sR[i] = wsrc[i];
    __syncthreads();

    const int tile_cols = (int)blockDim.x * 4;                    // 128 columns per warp
    const int col0 = cci * tile_cols + warp * 128;                // this warp's first column
    int32_t acc[8][4];
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
        for (int c = 0; c < 4; c++) acc[i][c] = 0;

    if (col0 < job.cols) {                                        // whole warp in or out
        const uint32_t ring = (uint32_t)__cvta_generic_to_shared(ring_base) + (uint32_t)warp * ROWLDM_STAGES * ROWLDM_STAGE_BYTES;
        // this lane's eight 16-byte pieces of a group: piece p = lane + 32 i  ->  row p / 8, bytes 16 (p % 8) ...
        const int piece_col = col0 + 16 * (lane & 7);
        const int src_bytes = max(0, min(16, job.cols - piece_col));       // bytes past the last column arrive as zeros
        const char* src_col = (const char*)job.mat + (src_bytes > 0 ? piece_col : 0);
        auto issue = [&](int G) {
            if (G < ngroups) {
                const uint32_t stage = ring + (uint32_t)(G % ROWLDM_STAGES) * ROWLDM_STAGE_BYTES;
#pragma unroll
                for (int i = 0; i < 8; i++) {
                    const int rr = (lane >> 3) + 4 * i;                              // row of the group
                    const int row = min(r0 + 32 * G + rr, r1 - 1);                    // clamped; its weight is 0 past r1
                    cp_async_16(stage + (uint32_t)rr * ROWLDM_PITCH + 16u * (lane & 7), src_col + (int64_t)row * job.ld, src_bytes);
                }
            }
            cp_async_commit();                                        // (an empty group keeps the count uniform)
        };
#pragma unroll
        for (int s = 0; s < ROWLDM_STAGES - 1; s++) issue(s);
        // ldmatrix row address of this lane: matrix lane / 16 (rows 0-15 / 16-31), row lane % 16
        const uint32_t lrow = (uint32_t)(16 * (lane >> 4) + (lane & 15)) * ROWLDM_PITCH;
        for (int G = 0; G < ngroups; G++) {
            issue(G + ROWLDM_STAGES - 1);
            cp_async_wait<ROWLDM_STAGES - 1>();                       // this lane's pieces of group G have landed
            __syncwarp();                                             // ... and every other lane's
            const uint32_t stage = ring + (uint32_t)(G % ROWLDM_STAGES) * ROWLDM_STAGE_BYTES;
            const uint2 wb = sR[G * 32 + lane];
#pragma unroll
            for (int jb = 0; jb < 8; jb++) {
                uint32_t a[4];
                ldmatrix_x2_trans_b8(a, stage + lrow + 16u * jb);
                mma_m16n8k32<true>(acc[jb], a[0], a[1], a[2], a[3], wb.x, wb.y);
            }
            __syncwarp();                                             // the stage may be refilled from the next iteration on
        }
    }
#pragma unroll
    for (int jb = 0; jb < 8; jb++)
#pragma unroll
        for (int h = 0; h < 2; h++) {
            uint64_t v = combine_limbs(acc[jb][2 * h], acc[jb][2 * h + 1], t);
            const int c = col0 + 16 * jb + g + 8 * h;
            if (t == 0 && c < job.cols) job.out[(int64_t)rbi * job.cols + c] = v;
        }
}

__global__ void __launch_bounds__(ROWMMA_MAX_WARPS * 32) rowmma_kernel(const MatJob* jobs, int njobs)
{
    __shared__ uint2 sR[MAX_TILE_ROWS];                             // (MAX_TILE_ROWS / 32) groups x 32 lanes
    extern __shared__ __align__(128) char ring[];                   // warps x stages x (32 rows x 144 bytes)
    const MatJob job = jobs[find_job(jobs, njobs, blockIdx.x)];
    const uint32_t local = blockIdx.x - job.tile0;
    if (job.vec) rowldm_tile(job, local, sR, ring);
    else rowmma_tile<false>(job, local, sR);
}

}  // namespace imm
