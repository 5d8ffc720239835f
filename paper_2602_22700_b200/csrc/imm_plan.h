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
#ifndef IMM_BYTEDOT_CHUNK_BYTES
#define IMM_BYTEDOT_CHUNK_BYTES 4096
#endif
#ifndef IMM_BYTEDOT_UNROLL
#define IMM_BYTEDOT_UNROLL 1
#endif
constexpr int BYTEDOT_THREADS = IMM_BYTEDOT_THREADS;          // warps sweep 16 or 32 rows at a time
constexpr int BYTEDOT_CHUNK_BYTES = IMM_BYTEDOT_CHUNK_BYTES;  // byte-columns per tile (multiple of 256)
constexpr int BYTEDOT_UNROLL = IMM_BYTEDOT_UNROLL;            // slabs of 256 byte-columns in flight per warp
constexpr int ROWMMA_THREADS = 256;            // 8 warps x 128 columns
constexpr int ROWMMA_COLS = 1024;              // int8 columns per tile
constexpr int SUMCHECK_THREADS = 1024;
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
    uint32_t pad_;
};

// Per-proof state of the round kernel.
struct ProofDev {
    imm_fe* e_row;             // 2^a entries
    imm_fe* e_col;             // 2^c entries
    const imm_fe* part_a;      // [n_part_a][k]   partial avec (one per row block of A)
    const imm_fe* part_b;      // [n_part_b][k]   partial bvec (one per column chunk of B)
    const imm_fe* part_c;      // [n_part_c]      partial c0 (one per tile of C)
    imm_fe* tab;               // 2 * 2^b entries: avec then bvec, padded with zeros
    uint64_t proof_id;
    int32_t m, k, n;
    int32_t a, b, c;           // ceil(log2 m), ceil(log2 k), ceil(log2 n)
    int32_t n_part_a, n_part_b, n_part_c;
    int32_t pad_;
};

// One limb table of eq weights in MMA fragment order (see weights_kernel).
enum WeightMode { W_COLS_I8 = 0, W_COLS_I32 = 1, W_ROWS = 2 };
struct WeightTask {
    const imm_fe* eq;          // eq table
    uint32_t* out;             // nwords 32-bit words
    int32_t extent;            // real extent (columns or rows); weights past it are zero
    int32_t nwords;
    int32_t mode;
    int32_t pad_;
};

// One eq table of a batch: r is derived in-kernel from (seed, proof_id, domain).
struct EqTask {
    imm_fe* out;
    uint64_t seed, proof_id;
    uint32_t domain;
    int32_t nvars;
};

// A single eq table with r supplied by the caller (passed by value to the kernel).
struct EqDirect {
    imm_fe r[MAX_EQ_VARS];
};

}  // namespace imm
