// Internal structures shared by the host planner and the kernels of libimm (not part of the ABI).
#pragma once
#include <stdint.h>

typedef uint64_t imm_fe;

namespace imm {

// Contraction tile geometry (elements).  A thread of the row-binding kernels owns one 16-byte
// vector of columns; a warp of the column-binding kernel sweeps a chunk of columns for a few
// rows at a time.
constexpr int ROWBIND_THREADS = 128;           // -> 2048 int8 / 512 int32 columns per tile
constexpr int COLBIND_THREADS = 256;           // 8 warps
constexpr int COLBIND_VECS = 128;              // 16-byte vectors per column chunk (2048 int8 / 512 int32)
constexpr int COLBIND_ROWS_PER_WARP = 4;
constexpr int MAX_TILE_ROWS = 1024;            // eq entries staged per tile by the row-binding kernels
// Tensor-core (int8 MMA) contraction kernels.
#ifndef IMM_BYTEDOT_THREADS
#define IMM_BYTEDOT_THREADS 256
#endif
#ifndef IMM_BYTEDOT_MAX_CHUNK_BYTES
#define IMM_BYTEDOT_MAX_CHUNK_BYTES 4096
#endif
#ifndef IMM_BYTEDOT_UNROLL
#define IMM_BYTEDOT_UNROLL 1
#endif
constexpr int BYTEDOT_THREADS = IMM_BYTEDOT_THREADS;          // warps sweep 16 or 32 rows at a time
constexpr int BYTEDOT_MAX_CHUNK_BYTES = IMM_BYTEDOT_MAX_CHUNK_BYTES;  // most byte-columns per tile; a job's own
                                                                     // chunk is a multiple of 256 up to this
constexpr int BYTEDOT_UNROLL = IMM_BYTEDOT_UNROLL;            // slabs of 256 byte-columns in flight per warp
constexpr int ROWMMA_MAX_WARPS = 8;            // a block of w warps covers w x 128 int8 columns
constexpr int ROWLDM_STAGES = 4;               // shared-memory stages per warp of the row-binding kernel
constexpr int ROWLDM_PITCH = 144;              // bytes per staged row: 128 of data, 16 of padding
constexpr int ROWLDM_STAGE_BYTES = 32 * ROWLDM_PITCH;
#ifndef IMM_FUSED_BLOCKS
#define IMM_FUSED_BLOCKS 3
#endif
constexpr int FUSED_BLOCKS_PER_SM = IMM_FUSED_BLOCKS;         // resident blocks per SM of the fused contraction launch
constexpr int EQ_BATCH_THREADS = 256;
constexpr int EQ_SLICE_QUADS = 512;           // groups of four table entries per block of eq_batch_kernel
constexpr int SUMCHECK_THREADS = 512;
constexpr int COMBINE_THREADS = 128;        // threads of a block of the batched-transcript kernel
constexpr int SUMCHECK_MAX_CLUSTER = 16;    // most blocks per proof (a power of two dividing 256)
constexpr int MAX_EQ_VARS = 20;
constexpr int MAX_K_VARS = 17;

enum JobKind { JOB_ROWBIND = 0, JOB_COLBIND = 1, JOB_POINT = 2 };

// One matrix contraction: tiles [tile0, tile0 + nrb*ncc) of a launch belong to it.
struct MatJob {
    const void* mat;
    const imm_fe* eq_row;      // ROWBIND / POINT: weights of the rows
    const imm_fe* eq_col;      // COLBIND / POINT: weights of the columns
    imm_fe* out;               // ROWBIND: [nrb][cols]; COLBIND: [ncc][rows]; POINT: [nrb*ncc]
    const uint32_t* wtab;      // tensor-core kernels: limb table of the weights in fragment order
    int64_t ld;                // elements
    int32_t rows, cols;
    int32_t tile_rows;         // rows per tile
    int32_t nrb, ncc;          // row blocks, column chunks
    int32_t vec;               // 2: rows 32-byte aligned, 1: 16-byte aligned, 0: element-wise loads
    uint32_t tile0;            // first tile of this job in the launch
    int32_t chunk;             // byte-dot kernel: byte-columns per tile (multiple of 256)
};

// Fused launch (small batches): one persistent grid over all three matrix kinds.  The work is a
// sequence of segments -- a tile of A, or rows [r0, r1) of one column chunk of B or C -- cut on the
// host into one contiguous run per block with equal bytes, so that all blocks finish together.  The
// blocks build the eq weights they need from the challenges: no eq table or limb table is in memory.
struct FusedJob {
    MatJob mj;                 // matrix, geometry, output (wtab / eq_row / eq_col unused).  A: tile_rows x 1024-column
                               // tiles, out[nrb][cols]; B: chunk, ncc, out[ncc][rows]; C: chunk, ncc, out[segments * 8]
    uint64_t seed, proof_id;   // r_row = challenge(seed, proof_id, 1, .), r_col = challenge(seed, proof_id, 2, .)
    const imm_fe* pt_row;      // non-null: r_row is read from here (a variables) instead of the generator
    const imm_fe* pt_col;      // non-null: r_col likewise (c variables)
    int32_t kind;              // JobKind: ROWBIND = A (int8), COLBIND = B (int8), POINT = C (int32)
    int32_t a, c;              // variables of this matrix's row / column index
    int32_t seg0;              // C: its first segment (a segment's eight warp partials go to out[(seg - seg0) * 8 ..])
};

struct FusedSeg {
    int32_t job;               // index into the FusedJob list
    int32_t cci;               // B, C: column chunk;  A: tile index within the job (row block * ncc + column block)
    int32_t r0, r1;            // B, C: rows [r0, r1)
};

// Per-proof state of the round kernel.
struct ProofDev {
    imm_fe* e_row;             // 2^a entries
    imm_fe* e_col;             // 2^c entries
    const imm_fe* part_a;      // [n_part_a][k]   partial avec (one per row block of A)
    const imm_fe* part_b;      // [n_part_b][k]   partial bvec (one per column chunk of B)
    const imm_fe* part_c;      // [n_part_c]      partial c0 (one per tile, or per warp of a tile, of C)
    const imm_fe* sum_row;     // [n_sum_row] slice sums of E_row over the real rows    } only when the claim
    const imm_fe* sum_col;     // [n_sum_col] slice sums of E_col over the real columns } kernel leaves the
                               //             2^31 offset of its unsigned bytes in part_c (c_offset != 0)
    uint64_t round_id;         // id the round challenges are drawn under: the proof's own, or its batch's
    int32_t m, k, n;
    int32_t a, b, c;           // ceil(log2 m), ceil(log2 k), ceil(log2 n)
    int32_t n_part_a, n_part_b, n_part_c;
    int32_t c_offset;          // 1: c0 = sum(part_c) - 2^31 * (sum of E_row over the real rows) * (sum of E_col over the
                               //    real columns); the two sums come from sum_row / sum_col, or, where those are
                               //    null, from the challenges in closed form
    int32_t n_sum_row, n_sum_col;
    uint64_t seed, proof_id;   // the proof's own coins (r_row, r_col), for the closed form
    const imm_fe* pt_row;      // non-null: r_row / r_col are read from here instead of the generator
    const imm_fe* pt_col;
    imm_fe* tab;               // non-null: [2][2^b] both round tables, summed over the partial vectors and zero-padded
                               //           by reduce_parts_kernel, which also leaves the claim in c0_ready
    imm_fe* c0_ready;
};

// One eq table of a batch: r is derived in-kernel from (seed, proof_id, domain).  The same pass
// can emit the table's limb tables for the tensor-core kernels (null = not wanted): weights of
// entries at or past `extent` are zero.  Layouts: see eq_batch_kernel.
struct EqTask {
    imm_fe* out;               // 2^nvars entries
    uint64_t seed, proof_id;
    uint32_t domain;
    int32_t nvars;
    uint32_t* w_rows;          // ceil(extent / 32) * 64 words
    uint32_t* w_cols_i8;       // ceil(extent / 256) * 512 words
    uint32_t* w_cols_i32;      // ceil(4 * extent / 256) * 512 words
    int32_t extent;
    int32_t pad_;
    imm_fe* slice_sums;        // one entry per block of the task: sum of its entries below `extent` (or null)
    const imm_fe* given;       // non-null: the table exists already (`extent` entries are read from here, nothing
                               // is derived or written to `out`); only the limb tables and slice sums are produced
    const imm_fe* point;       // non-null: r is read from here (nvars entries) instead of the generator
};

// Per proof of a non-interactive (Fiat-Shamir) batch: where its statement and hashed challenges live.
constexpr int FS_POINT_SLOTS = 32;          // slots per point: r_row at [0, a), r_col at [FS_POINT_SLOTS, FS_POINT_SLOTS + c)
constexpr int FS_THREADS = 1024;            // threads of the round kernel's block (one block per proof)
struct FsProof {
    const uint8_t* com;        // 96 bytes: the commitments to A, B, C
    imm_fe* points;            // [2 * FS_POINT_SLOTS]
    uint32_t* state;           // [8]: s_0, the hash of the statement
    imm_fe* ta;                // [2^b] the round kernel's tables
    imm_fe* tb;
    uint64_t proof_id;
    uint32_t one;              // 1 (the multiplier of the multiply-add form of SHA-256's adds)
    uint32_t pad_;
};

// One batched non-interactive proof: where its coins and per-round exchange live (device pointers).
constexpr int FS_BATCH_MAX = 1024;          // members of one batched non-interactive proof (one block folds their statements)
struct FsBatch {
    uint32_t* T;               // [8]  the batch seed: hash of the tree over the member statements, the id, the count
    uint32_t* state;           // [8]  the transcript state
    imm_fe* rho;               // [P]  combination coefficients
    imm_fe* c0;                // [P]  the members' claims
    imm_fe* partial;           // [P][3] rho_p times the current round's three sums of member p
    imm_fe* r;                 // [MAX_K_VARS] round challenges as they become known
    uint64_t batch_id;
    int32_t nproofs, b;
    uint32_t one, pad_;
};

// Per proof of a verifier's pass: the eq table of the round challenges, E_k[y] = eq(r_k, y).
constexpr int VERIFY_POINT_SLOTS = 3 * FS_POINT_SLOTS;      // caller-given points per proof: r_row, r_col, r_k
struct ExpectDev {
    const imm_fe* e_k;         // 2^b entries, b the proof's round count (the batch's for a batched proof)
};

// A single eq table with r supplied by the caller (passed by value to the kernel).
struct EqDirect {
    imm_fe r[MAX_EQ_VARS];
};

}  // namespace imm
