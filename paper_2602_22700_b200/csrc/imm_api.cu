// C ABI of libimm: argument validation, workspace planning and launch sequencing.
// All arithmetic on matrix data happens in the kernels (imm_kernels.cu); the only field
// arithmetic done on the host is the verifier, which is host-side by definition.
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/imm.h"
#include "gl64.cuh"
#include "imm_kernels.h"
#include "imm_plan.h"
#include "sha256.cuh"

namespace {

using namespace imm;

thread_local std::string g_cuda_err;

int cuda_fail(cudaError_t e)
{
    g_cuda_err = std::string(cudaGetErrorName(e)) + ": " + cudaGetErrorString(e);
    return IMM_ERR_CUDA;
}
#define CU(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return cuda_fail(e_); } while (0)

constexpr int64_t MAX_EXTENT = (int64_t)1 << 20;
constexpr int64_t MAX_K = (int64_t)1 << MAX_K_VARS;
constexpr size_t ALIGN = 256;
static_assert(FS_BATCH_MAX == IMM_FS_BATCH_MAX, "the header's limit is the kernels'");

size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }

int ceil_log2(int64_t d)
{
    int n = 0;
    while (((int64_t)1 << n) < d) n++;
    return n;
}

size_t elem_size(int dtype) { return dtype == IMM_I8 ? 1 : 4; }

bool rows_vectorisable(const void* p, int64_t ld, int dtype)
{
    return ((uintptr_t)p % 16 == 0) && ((ld * (int64_t)elem_size(dtype)) % 16 == 0);
}

// Tile-geometry overrides for sweeps exist only in a library built with -DIMM_TUNING; the shipped
// library reads one environment variable, IMM_CONTRACT (documented in imm.h).
#ifdef IMM_TUNING
int env_int(const char* name, int dflt)
{
    const char* s = getenv(name);
    if (!s || !*s) return dflt;
    int v = atoi(s);
    return v > 0 ? v : dflt;
}
bool env_set(const char* name) { return getenv(name) != nullptr; }
#else
int env_int(const char*, int dflt) { return dflt; }
bool env_set(const char*) { return false; }
#endif

// Columns per tile of each kernel family.
int rowbind_cols(int dtype) { return ROWBIND_THREADS * (dtype == IMM_I8 ? 16 : 4); }
int colbind_cols(int dtype) { return COLBIND_VECS * (dtype == IMM_I8 ? 16 : 4); }

// Contraction back end of the prover: tensor-core (int8 MMA over 8-bit limbs of the weights) unless
// IMM_CONTRACT=alu selects the integer-pipe kernels.
bool use_mma()
{
    const char* s = getenv("IMM_CONTRACT");
    return !(s && strcmp(s, "alu") == 0);
}
struct Shape { int64_t rows, cols; };

// Rows per tile: the largest candidate that still yields enough tiles to fill the GPU several
// times over (the tail of the last wave is then a small fraction of the launch).
int pick_tile_rows(const std::vector<Shape>& mats, int cols_per_tile, const char* env_name,
                   int max_rows = MAX_TILE_ROWS)
{
    const int forced = env_int(env_name, 0);
    if (forced) {
        int v = forced < 32 ? 32 : forced > MAX_TILE_ROWS ? MAX_TILE_ROWS : forced;
        return v / 32 * 32;
    }
    const int64_t target = (int64_t)sm_count() * env_int("IMM_TILES_PER_SM", 24);
    const int cand[] = {1024, 512, 256, 128, 64, 32};
    for (int c : cand) {
        if (c > max_rows) continue;
        int64_t tiles = 0;
        for (const Shape& s : mats)
            tiles += ((s.rows + c - 1) / c) * ((s.cols + cols_per_tile - 1) / cols_per_tile);
        if (tiles >= target) return c;
    }
    return 32;
}

// Tile geometry of a tensor-core contraction: rows x width, width in the kernel's own unit
// (byte-columns for the byte-dot kernel, int8 columns for the row-binding kernel).
struct Geom { int rows, width; };

int64_t count_tiles(const std::vector<Shape>& mats, int rows, int width)
{
    int64_t tiles = 0;
    for (const Shape& s : mats) tiles += ((s.rows + rows - 1) / rows) * ((s.cols + width - 1) / width);
    return tiles;
}

// The largest tile among rows x widths that still cuts the batch into enough tiles to fill the GPU
// several times over (the last wave is then a small fraction of the launch); for a batch too small
// for that, the smallest tile, i.e. the most parallelism there is.  Large tiles amortise the
// per-tile set-up (weight limbs staged in shared memory) and keep DRAM pages open longer.
Geom pick_geom_for(const std::vector<Shape>& mats, const int* rows, int nrows, const int* widths, int nwidths,
                   int64_t target, const char* env_rows, const char* env_width);

Geom pick_geom(const std::vector<Shape>& mats, const int* rows, int nrows, const int* widths, int nwidths,
               int tiles_per_sm, const char* env_rows, const char* env_width)
{
    return pick_geom_for(mats, rows, nrows, widths, nwidths,
                         (int64_t)sm_count() * env_int("IMM_TILES_PER_SM", tiles_per_sm), env_rows, env_width);
}

Geom pick_geom_for(const std::vector<Shape>& mats, const int* rows, int nrows, const int* widths, int nwidths,
                   int64_t target, const char* env_rows, const char* env_width)
{
    Geom best{rows[nrows - 1], widths[nwidths - 1]};          // candidates are listed largest first
    int64_t best_area = -1;
    for (int i = 0; i < nrows; i++)
        for (int k = 0; k < nwidths; k++) {
            const int64_t area = (int64_t)rows[i] * widths[k];
            if (area > best_area && count_tiles(mats, rows[i], widths[k]) >= target) {
                best = Geom{rows[i], widths[k]};
                best_area = area;
            }
        }
    // overrides for sweeps; snapped to the candidate lists' ranges
    const int fr = env_int(env_rows, 0), fw = env_int(env_width, 0);
    if (fr) { int v = fr < rows[nrows - 1] ? rows[nrows - 1] : fr > rows[0] ? rows[0] : fr; best.rows = v / rows[nrows - 1] * rows[nrows - 1]; }
    if (fw) { int v = fw < widths[nwidths - 1] ? widths[nwidths - 1] : fw > widths[0] ? widths[0] : fw; best.width = v / widths[nwidths - 1] * widths[nwidths - 1]; }
    return best;
}

// candidate tile heights and widths of the tensor-core kernels, largest first
const int rows_a[] = {1024, 512, 256, 128, 64, 32}, widths_a[] = {1024, 512, 256, 128};
const int rows_b[] = {256}, rows_c[] = {1024, 512, 256, 128};
const int chunks[] = {4096, 2048, 1024, 512, 256};
// fused launch (small batches): one persistent grid, a run of equal bytes per block
// Which batches take the fused contraction launch (measured on expert, decoder-block and attention batches):
// it saves about 40 us of launches and dependencies but streams a little slower than the three tuned
// kernels, and its per-job set-up weighs on batches of many small proofs.  Fused: every batch under 4 GiB;
// up to 16 GiB when a proof averages 32 MiB or more (decoder projections, experts), where it wins by 15 % at
// 2 GiB and 1 % at 13 GiB; attention-sized proofs (11 MiB each) win by 9 % at 0.7 and 7 % at 2.7 GiB and
// lose by 3 % at 5.4 GiB.
constexpr int64_t FUSE_ALWAYS_BELOW_BYTES = (int64_t)4 << 30;
constexpr int64_t FUSE_BELOW_BYTES = (int64_t)16 << 30;
constexpr int64_t FUSE_MIN_BYTES_PER_PROOF = (int64_t)32 << 20;
constexpr int FUSED_A_TILE_COLS = 1024;                      // 8 warps x 128 columns
constexpr int64_t FUSED_MIN_RUN_BYTES = 32 << 10;            // below this a run is all set-up
constexpr int FUSED_JOB_SETUP_KB = 160, FUSED_CHUNK_SETUP_KB = 24;  // a job's and a chunk's set-up in bytes a block streams meanwhile (from sweeps over expert, FFN and attention batches)
constexpr int FUSED_COST_A = 250, FUSED_COST_C = 180;        // time per byte of A and of C relative to B, per cent (measured)
// rows one pass of a block's eight warps covers: row ranges are cut at multiples of it, so that no pass runs
// on a few warps only (16 rows per warp and pass)
constexpr int FUSED_PASS_ROWS_C = 128, FUSED_PASS_ROWS_B = 128;

void fill_job(MatJob& j, const void* mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
              int tile_rows, int cols_per_tile)
{
    memset(&j, 0, sizeof(j));
    j.mat = mat;
    j.ld = ld;
    j.rows = (int32_t)rows;
    j.cols = (int32_t)cols;
    j.tile_rows = tile_rows;
    j.nrb = (int32_t)((rows + tile_rows - 1) / tile_rows);
    j.ncc = (int32_t)((cols + cols_per_tile - 1) / cols_per_tile);
    // 2: rows 32-byte aligned (256-bit loads), 1: 16-byte aligned (128-bit loads), 0: element-wise
    const int64_t pitch = ld * (int64_t)elem_size(dtype);
    j.vec = ((uintptr_t)mat % 32 == 0 && pitch % 32 == 0) ? 2 : rows_vectorisable(mat, ld, dtype) ? 1 : 0;
}

int check_matrix_args(const void* d_mat, int dtype, int64_t rows, int64_t cols, int64_t ld)
{
    if (!d_mat || (dtype != IMM_I8 && dtype != IMM_I32)) return IMM_ERR_ARG;
    if (rows <= 0 || cols <= 0 || rows > MAX_EXTENT || cols > MAX_EXTENT || ld < cols) return IMM_ERR_SHAPE;
    return IMM_OK;
}

// ------------------------------------------------------------------ single-matrix calls ---
// imm_mle_partial_eval / imm_mle_eval_point on the tensor-core kernels: the workspace holds the job,
// two eq tasks (limb tables and slice sums from the caller's eq tables), the limb table, the slice
// sums and the partial results.  int32 partial evaluations have no tensor-core kernel and stay on
// the integer-pipe kernels, as does everything under IMM_CONTRACT=alu.
enum MleOp { OP_ROWS = 0, OP_COLS = 1, OP_POINT = 2 };

struct MlePlan {
    bool mma = false;
    Geom g{0, 0};
    int64_t nrb = 0, ncc = 0, nparts = 0;
    int nw = 0, n_sr = 0, n_sc = 0;
    size_t off_tasks = 0, off_w = 0, off_sr = 0, off_sc = 0, off_parts = 0, total = 0;
};

MlePlan plan_mle(int dtype, int64_t rows, int64_t cols, MleOp op)
{
    MlePlan p;
    p.mma = use_mma() && (op == OP_POINT || dtype == IMM_I8);
    if (!p.mma) return p;
    const int64_t slice = 4 * (int64_t)EQ_SLICE_QUADS;
    if (op == OP_ROWS) {
        std::vector<Shape> m{{rows, cols}};
        p.g = pick_geom(m, rows_a, 6, widths_a, 4, 12, "IMM_TILE_ROWS_A", "IMM_TILE_COLS_A");
        p.nw = (int)((rows + 31) / 32) * 64;
    } else if (op == OP_COLS) {
        std::vector<Shape> m{{rows, cols}};
        p.g = pick_geom(m, rows_b, 1, chunks, 5, 24, "IMM_TILE_ROWS_B", "IMM_CHUNK_B");
        p.nw = (int)((cols + 255) / 256) * 512;
    } else {
        const int64_t bytes = cols * (int64_t)elem_size(dtype);
        std::vector<Shape> m{{rows, bytes}};
        p.g = pick_geom(m, rows_c, 4, chunks, 5, 24, "IMM_TILE_ROWS_C", "IMM_CHUNK_C");
        p.nw = (int)((bytes + 255) / 256) * 512;
        if (dtype == IMM_I32) {
            p.n_sr = (int)((rows + slice - 1) / slice);
            p.n_sc = (int)(((cols + 255) / 256 * 256 + slice - 1) / slice);
        }
    }
    const int64_t width_elems = op == OP_POINT ? p.g.width / (int64_t)elem_size(dtype) : p.g.width;
    p.nrb = (rows + p.g.rows - 1) / p.g.rows;
    p.ncc = (cols + width_elems - 1) / width_elems;
    p.nparts = op == OP_ROWS ? p.nrb * cols : op == OP_COLS ? p.ncc * rows : p.nrb * p.ncc * (BYTEDOT_THREADS / 32);
    size_t off = ALIGN;                                   // the job
    p.off_tasks = off; off = align_up(off + 2 * sizeof(EqTask));
    p.off_w = off;     off = align_up(off + 4 * (size_t)p.nw);
    p.off_sr = off;    off = align_up(off + sizeof(imm_fe) * (size_t)p.n_sr);
    p.off_sc = off;    off = align_up(off + sizeof(imm_fe) * (size_t)p.n_sc);
    p.off_parts = off; off = align_up(off + sizeof(imm_fe) * (size_t)p.nparts);
    p.total = off;
    return p;
}

// ------------------------------------------------------------------ batch plan ------------

struct Plan {
    int status = IMM_OK;
    int nproofs = 0;
    int max_b = 0;
    bool mma = true;
    bool fused = false;                        // one contraction launch with the eq weights built in the tiles
    int64_t max_cover = 0;                     // most entries an eq task covers (table or padded limb tables)
    int rows_a = 0, rows_b = 0, rows_c = 0;
    int cols_a = 0, cols_b = 0, cols_c = 0;    // columns (elements) per tile of the three contractions
    int mt_b = 2, mt_c = 1;                    // MMA row tiles per warp pass of the byte-dot kernels
    uint32_t tiles_a = 0, tiles_b = 0, tiles_c = 0;
    // byte offsets from the workspace base
    size_t off_proofs = 0, off_jobs_a = 0, off_jobs_b = 0, off_jobs_c = 0, off_eq = 0, off_fjobs = 0, header_bytes = 0;
    struct PerProof {
        size_t e_row, e_col, part_a, part_b, part_c, sum_row, sum_col, tab, c0_ready;
        int n_sum_row, n_sum_col;
        size_t w_rows, w_cols_b, w_cols_c;          // limb tables (tensor-core back end)
        int nw_rows, nw_cols_b, nw_cols_c;          // their sizes in 32-bit words
        int a, b, c, n_part_a, n_part_b, n_part_c;
    };
    std::vector<PerProof> pp;
    size_t total_bytes = 0;
    // fused launch: per-proof geometry, the segment list and each block's first segment
    struct FusedGeom { int rows_a, nrb_a, ncc_a, chunk_b, ncc_b, chunk_c, ncc_c, seg0_c, nseg_c; };
    std::vector<FusedGeom> fg;
    std::vector<FusedSeg> segs;
    std::vector<uint32_t> block_first;          // blocks + 1 entries
    size_t off_segs = 0, off_block_first = 0;
};

int pow2_ceil_clamped(int64_t v, int lo, int hi)
{
    int c = lo;
    while (c < hi && c < v) c *= 2;
    return c;
}

int pow2_floor_clamped(int64_t v, int lo, int hi)
{
    int c = lo;
    while (2 * c <= hi && 2 * c <= v) c *= 2;
    return c;
}

// The fused launch's partition: every block of the persistent grid gets one contiguous run of the
// sequence [tiles of every A][row ranges of every column chunk of every C][the same for every B],
// cut so that all runs hold (almost) the same number of matrix bytes.
// Lays the sequence out for runs of `run` cost units (bytes of B); returns the cost of the whole sequence.
// A job's set-up (challenges, eq tables: some 6 us) and a chunk's or tile's (weight limbs: 1-2 us) are
// charged as the bytes a block would stream meanwhile, so that a run of many small matrices is not
// taken for a short one.
int64_t plan_fused_runs(Plan& p, const imm_matmul_desc* descs, int nproofs, int64_t blocks, int64_t run)
{
    // cost of a byte of each kind relative to B, in per cent (measured: see FUSED_COST_*)
    const int64_t cost_a = env_int("IMM_FUSED_COST_A", FUSED_COST_A), cost_c = env_int("IMM_FUSED_COST_C", FUSED_COST_C);
    const int64_t job_cost = (int64_t)env_int("IMM_FUSED_JOB_KB", FUSED_JOB_SETUP_KB) << 10;
    const int64_t chunk_cost = (int64_t)env_int("IMM_FUSED_CHUNK_KB", FUSED_CHUNK_SETUP_KB) << 10;
    p.segs.clear();
    // widest column chunk that still cuts a run into several passes of all eight warps (the cuts fall on pass
    // boundaries, so the passes per run set how evenly the runs can be sized)
    const int passes = env_int("IMM_FUSED_PASSES", 4);
    const int pass_c = env_int("IMM_FUSED_PASS_C", FUSED_PASS_ROWS_C), pass_b = env_int("IMM_FUSED_PASS_B", FUSED_PASS_ROWS_B);
    const int cap = env_int("IMM_FUSED_CHUNK", BYTEDOT_MAX_CHUNK_BYTES);
    p.fg.resize(nproofs);
    std::vector<int32_t> seg_block;
    int64_t cum = 0;
    auto block_of = [&](int64_t pos) { return (int32_t)std::min<int64_t>(blocks - 1, pos / run); };
    // A: whole tiles of about half a run
    for (int i = 0; i < nproofs; i++) {
        const imm_matmul_desc& d = descs[i];
        Plan::FusedGeom& g = p.fg[i];
        cum += job_cost;
        const int64_t width = std::min<int64_t>(FUSED_A_TILE_COLS, d.k);
        int64_t rows = (run * 100 / cost_a / 2 / width) / 32 * 32;
        rows = rows < 32 ? 32 : rows > MAX_TILE_ROWS ? MAX_TILE_ROWS : rows;
        g.nrb_a = (int)((d.m + rows - 1) / rows);
        rows = ((d.m + g.nrb_a - 1) / g.nrb_a + 31) / 32 * 32;                // even row blocks
        g.rows_a = (int)rows;
        g.nrb_a = (int)((d.m + rows - 1) / rows);
        g.ncc_a = (int)((d.k + FUSED_A_TILE_COLS - 1) / FUSED_A_TILE_COLS);
        for (int rb = 0; rb < g.nrb_a; rb++)
            for (int cc = 0; cc < g.ncc_a; cc++) {
                const int64_t tr = std::min<int64_t>(rows, d.m - (int64_t)rb * rows);
                const int64_t tc = std::min<int64_t>(FUSED_A_TILE_COLS, d.k - (int64_t)cc * FUSED_A_TILE_COLS);
                p.segs.push_back(FusedSeg{i, rb * g.ncc_a + cc, 0, 0});
                seg_block.push_back(block_of(cum));
                cum += tr * tc * cost_a / 100 + chunk_cost / 2;
            }
    }
    // C then B: row ranges of column chunks
    for (int kind = 1; kind < 3; kind++)
        for (int i = 0; i < nproofs; i++) {
            const imm_matmul_desc& d = descs[i];
            Plan::FusedGeom& g = p.fg[i];
            const int64_t rows = kind == 1 ? d.m : d.k;
            const int64_t row_bytes = kind == 1 ? 4 * d.n : d.n;
            const int64_t cost = kind == 1 ? cost_c : 100;
            const int64_t step = kind == 1 ? pass_c : pass_b;
            const int chunk = pow2_ceil_clamped(row_bytes, 256, pow2_floor_clamped(run * 100 / cost / (passes * step), 256, cap));
            const int ncc = (int)((row_bytes + chunk - 1) / chunk);
            if (kind == 1) { g.chunk_c = chunk; g.ncc_c = ncc; g.seg0_c = (int)p.segs.size(); }
            else { g.chunk_b = chunk; g.ncc_b = ncc; }
            cum += job_cost;
            for (int cc = 0; cc < ncc; cc++) {
                if (kind == 1 && cc == 0) g.nseg_c = 0;
                cum += chunk_cost;
                // (a row piece costs whole slabs of 256 bytes: a 128-byte row of an attention head's V fills half of one)
                const int64_t w = std::max<int64_t>(1, (std::min<int64_t>(chunk, row_bytes - (int64_t)cc * chunk) + 255) / 256 * 256 * cost / 100);
                int64_t r = 0;
                while (r < rows) {
                    const int32_t b = block_of(cum);
                    int64_t nr = rows - r;
                    if (b < blocks - 1) {
                        const int64_t room = (int64_t)(b + 1) * run - cum;
                        int64_t want = ((room + w / 2) / w + step / 2) / step * step;           // to the nearest pass boundary
                        if (want < step) want = step;
                        if (r + want + step <= rows) nr = want;                  // (a remainder under one pass joins this range)
                    }
                    p.segs.push_back(FusedSeg{kind * nproofs + i, cc, (int32_t)r, (int32_t)(r + nr)});
                    seg_block.push_back(b);
                    if (kind == 1) g.nseg_c++;
                    cum += nr * w;
                    r += nr;
                }
            }
        }
    const int used = seg_block.empty() ? 0 : seg_block.back() + 1;
    p.block_first.assign(used + 1, 0);
    size_t si = 0;
    for (int b = 0; b <= used; b++) {
        while (si < seg_block.size() && seg_block[si] < b) si++;
        p.block_first[b] = (uint32_t)si;
    }
    return cum;
}

void plan_fused(Plan& p, const imm_matmul_desc* descs, int nproofs)
{
    const int64_t blocks = (int64_t)sm_count() * FUSED_BLOCKS_PER_SM;
    const int64_t cost_a = env_int("IMM_FUSED_COST_A", FUSED_COST_A), cost_c = env_int("IMM_FUSED_COST_C", FUSED_COST_C);
    int64_t total = 0;
    for (int i = 0; i < nproofs; i++)
        total += descs[i].m * descs[i].k * cost_a / 100 + descs[i].k * descs[i].n + 4 * descs[i].m * descs[i].n * cost_c / 100;
    // the set-up charges depend on the chunk widths, which depend on the run: lay out once to learn the
    // sequence's cost, then again with the run that cost gives
    int64_t run = std::max<int64_t>((total + blocks - 1) / blocks, FUSED_MIN_RUN_BYTES);
    const int64_t cost = plan_fused_runs(p, descs, nproofs, blocks, run);
    run = std::max<int64_t>((cost + blocks - 1) / blocks, FUSED_MIN_RUN_BYTES);
    plan_fused_runs(p, descs, nproofs, blocks, run);
}


int check_desc(const imm_matmul_desc& d)
{
    if (!d.A || !d.B || !d.C) return IMM_ERR_ARG;
    if (d.m <= 0 || d.k <= 0 || d.n <= 0 || d.m > MAX_EXTENT || d.n > MAX_EXTENT || d.k > MAX_K)
        return IMM_ERR_SHAPE;
    if (d.lda < d.k || d.ldb < d.n || d.ldc < d.n) return IMM_ERR_SHAPE;
    return IMM_OK;
}

Plan make_plan(const imm_matmul_desc* descs, int nproofs)
{
    Plan p;
    if (!descs || nproofs <= 0) { p.status = IMM_ERR_ARG; return p; }
    p.nproofs = nproofs;
    std::vector<Shape> sa, sb, sc;
    for (int i = 0; i < nproofs; i++) {
        int rc = check_desc(descs[i]);
        if (rc != IMM_OK) { p.status = rc; return p; }
        sa.push_back({descs[i].m, descs[i].k});
        sb.push_back({descs[i].k, descs[i].n});
        sc.push_back({descs[i].m, descs[i].n});
    }
    p.mma = use_mma();
    int64_t batch_bytes = 0;
    for (int i = 0; i < nproofs; i++)
        batch_bytes += descs[i].m * descs[i].k + descs[i].k * descs[i].n + 4 * descs[i].m * descs[i].n;
    const int64_t fuse_below = (int64_t)env_int("IMM_FUSE_BELOW_MB", (int)(FUSE_BELOW_BYTES >> 20)) << 20;
    p.fused = p.mma && !env_set("IMM_NO_FUSE") &&
              (batch_bytes < std::min(fuse_below, FUSE_ALWAYS_BELOW_BYTES) ||
               (batch_bytes < fuse_below &&
                batch_bytes / nproofs >= (int64_t)env_int("IMM_FUSE_MIN_PROOF_MB", (int)(FUSE_MIN_BYTES_PER_PROOF >> 20)) << 20));
    if (p.fused) {
        plan_fused(p, descs, nproofs);
    } else if (p.mma) {
        // A: rows x (128 columns per warp).  B, C: rows x byte-columns; a block pass covers
        // 128 rows per MMA row tile, so shorter tiles would leave warps idle.  Measured on the
        // decoder-block workload: B (two row tiles per warp) is best at 256 rows per tile, C (one) at
        // 512-1024.
        p.mt_b = env_int("IMM_BYTEDOT_MT_B", 2) == 1 ? 1 : 2;
        p.mt_c = env_int("IMM_BYTEDOT_MT_C", 1) == 2 ? 2 : 1;
        std::vector<Shape> scb;                               // C as a byte matrix
        for (const Shape& s : sc) scb.push_back({s.rows, 4 * s.cols});
        // tiles per SM aimed at, from sweeps over 1024...16384 tokens: the row-binding kernel (a
        // warp streams its own 128 columns) needs fewer, larger tiles than the byte-dot kernels
        const Geom ga = pick_geom(sa, rows_a, 6, widths_a, 4, 12, "IMM_TILE_ROWS_A", "IMM_TILE_COLS_A");
        // ... and a short launch (a few hundred MB) runs best on few, larger tiles: 4 per SM below
        // 256 MB, one more per 64 MB, 24 from 1.5 GB on
        int64_t bytes_b = 0, bytes_c = 0;
        for (const Shape& s : sb) bytes_b += s.rows * s.cols;
        for (const Shape& s : scb) bytes_c += s.rows * s.cols;
        auto per_sm = [](int64_t bytes) { int64_t t = bytes >> 26; return (int)(t < 4 ? 4 : t > 24 ? 24 : t); };
        const Geom gb = pick_geom(sb, rows_b, 1, chunks, 5, per_sm(bytes_b), "IMM_TILE_ROWS_B", "IMM_CHUNK_B");
        const Geom gc = pick_geom(scb, rows_c, 4, chunks, 5, per_sm(bytes_c), "IMM_TILE_ROWS_C", "IMM_CHUNK_C");
        p.rows_a = ga.rows; p.cols_a = ga.width;
        p.rows_b = gb.rows; p.cols_b = gb.width;
        p.rows_c = gc.rows; p.cols_c = gc.width / 4;
    } else {
        p.cols_a = rowbind_cols(IMM_I8); p.cols_b = colbind_cols(IMM_I8); p.cols_c = rowbind_cols(IMM_I32);
        p.rows_a = pick_tile_rows(sa, p.cols_a, "IMM_TILE_ROWS_A");
        p.rows_b = pick_tile_rows(sb, p.cols_b, "IMM_TILE_ROWS_B");
        p.rows_c = pick_tile_rows(sc, p.cols_c, "IMM_TILE_ROWS_C");
    }
    const int acols = p.cols_a, bcols = p.cols_b, ccols = p.cols_c;

    size_t off = 0;
    p.off_proofs = off; off = align_up(off + sizeof(ProofDev) * nproofs);
    p.off_jobs_a = off; off = align_up(off + sizeof(MatJob) * nproofs);
    p.off_jobs_b = off; off = align_up(off + sizeof(MatJob) * nproofs);
    p.off_jobs_c = off; off = align_up(off + sizeof(MatJob) * nproofs);
    p.off_eq = off;     off = align_up(off + sizeof(EqTask) * 2 * nproofs);
    p.off_fjobs = off;  off = align_up(off + (p.fused ? sizeof(FusedJob) * 3 * (size_t)nproofs : 0));
    p.off_segs = off;   off = align_up(off + sizeof(FusedSeg) * p.segs.size());
    p.off_block_first = off; off = align_up(off + sizeof(uint32_t) * p.block_first.size());
    p.header_bytes = off;

    uint64_t ta = 0, tb = 0, tc = 0;
    p.pp.resize(nproofs);
    for (int i = 0; i < nproofs; i++) {
        const imm_matmul_desc& d = descs[i];
        Plan::PerProof& q = p.pp[i];
        q.a = ceil_log2(d.m); q.b = ceil_log2(d.k); q.c = ceil_log2(d.n);
        if (q.b > p.max_b) p.max_b = q.b;
        int64_t c_nrb = 0, c_ncc = 0;
        if (p.fused) {
            // one partial avec per row block of A, one partial bvec per column chunk of B, eight warp
            // partials per segment of C
            const Plan::FusedGeom& g = p.fg[i];
            q.n_part_a = g.nrb_a;
            q.n_part_b = g.ncc_b;
            q.n_part_c = g.nseg_c * (BYTEDOT_THREADS / 32);
        } else {
            q.n_part_a = (int)((d.m + p.rows_a - 1) / p.rows_a);
            q.n_part_b = (int)((d.n + bcols - 1) / bcols);
            c_nrb = (d.m + p.rows_c - 1) / p.rows_c;
            c_ncc = (d.n + ccols - 1) / ccols;
            q.n_part_c = (int)(c_nrb * c_ncc) * (p.mma ? BYTEDOT_THREADS / 32 : 1);   // tensor-core kernel: one per warp
        }
        const int64_t slice = 4 * (int64_t)EQ_SLICE_QUADS;                  // entries per block of the eq kernel
        q.n_sum_row = (int)((std::max<int64_t>((int64_t)1 << q.a, (d.m + 31) / 32 * 32) + slice - 1) / slice);
        q.n_sum_col = (int)((std::max<int64_t>((int64_t)1 << q.c, (d.n + 255) / 256 * 256) + slice - 1) / slice);
        if (((int64_t)1 << q.a) > p.max_cover) p.max_cover = (int64_t)1 << q.a;
        if (((int64_t)1 << q.c) > p.max_cover) p.max_cover = (int64_t)1 << q.c;
        if (p.fused) { q.n_sum_row = q.n_sum_col = 0; }
        q.e_row = off;  off = align_up(off + (p.fused ? 0 : sizeof(imm_fe) * ((size_t)1 << q.a)));
        q.e_col = off;  off = align_up(off + (p.fused ? 0 : sizeof(imm_fe) * ((size_t)1 << q.c)));
        q.part_a = off; off = align_up(off + sizeof(imm_fe) * (size_t)q.n_part_a * d.k);
        q.part_b = off; off = align_up(off + sizeof(imm_fe) * (size_t)q.n_part_b * d.k);
        q.part_c = off; off = align_up(off + sizeof(imm_fe) * (size_t)q.n_part_c);
        q.sum_row = off; off = align_up(off + sizeof(imm_fe) * (size_t)q.n_sum_row);
        q.sum_col = off; off = align_up(off + sizeof(imm_fe) * (size_t)q.n_sum_col);
        q.nw_rows = q.nw_cols_b = q.nw_cols_c = 0;
        q.w_rows = q.w_cols_b = q.w_cols_c = 0;
        if (p.mma && !p.fused) {
            q.nw_rows = (int)((d.m + 31) / 32) * 64;
            q.nw_cols_b = (int)((d.n + 255) / 256) * 512;
            q.nw_cols_c = (int)((4 * d.n + 255) / 256) * 512;
            q.w_rows = off;   off = align_up(off + 4 * (size_t)q.nw_rows);
            q.w_cols_b = off; off = align_up(off + 4 * (size_t)q.nw_cols_b);
            q.w_cols_c = off; off = align_up(off + 4 * (size_t)q.nw_cols_c);
            const int64_t cover_rows = (d.m + 31) / 32 * 32, cover_cols = (d.n + 255) / 256 * 256;
            if (cover_rows > p.max_cover) p.max_cover = cover_rows;
            if (cover_cols > p.max_cover) p.max_cover = cover_cols;
        }
        if (!p.fused) {
            ta += (uint64_t)q.n_part_a * ((d.k + acols - 1) / acols);
            tb += (uint64_t)((d.k + p.rows_b - 1) / p.rows_b) * q.n_part_b;
            tc += (uint64_t)(c_nrb * c_ncc);
        }
    }
    if (ta > 0x7FFFFFFFu || tb > 0x7FFFFFFFu || tc > 0x7FFFFFFFu || ta + tb + tc > 0x7FFFFFFFu) { p.status = IMM_ERR_SHAPE; return p; }
    p.tiles_a = (uint32_t)ta; p.tiles_b = (uint32_t)tb; p.tiles_c = (uint32_t)tc;
    if (p.fused)                                 // both round tables (2^max_b entries each: a batched proof pads every k) and the claim
        for (int i = 0; i < nproofs; i++) {
            p.pp[i].tab = off;      off = align_up(off + 2 * (sizeof(imm_fe) << p.max_b));
            p.pp[i].c0_ready = off; off = align_up(off + sizeof(imm_fe));
        }
    p.total_bytes = off;
    return p;
}

// phase-timing events (see imm_profile_enable)
constexpr int PROF_EV = 2 * IMM_PROFILE_PHASES;    // a (start, end) pair per phase
std::vector<cudaEvent_t> g_prof_ev;        // capacity * PROF_EV events, empty when profiling is off
int64_t g_prof_calls = 0;

int check_stride(const imm_matmul_desc* descs, int nproofs, int64_t stride)
{
    for (int i = 0; i < nproofs; i++)
        if (stride < 3 * ceil_log2(descs[i].k) + 3) return IMM_ERR_SHAPE;
    return IMM_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// exported functions
// ---------------------------------------------------------------------------------------------

extern "C" {

int imm_version(void) { return 100; }

const char* imm_last_cuda_error(void) { return g_cuda_err.c_str(); }

imm_fe imm_challenge(uint64_t seed, uint64_t proof_id, uint32_t domain, uint32_t index)
{
    return gl::challenge(seed, proof_id, domain, index);
}

int imm_field_binop(int op, const imm_fe* d_x, const imm_fe* d_y, imm_fe* d_out, int64_t count,
                    void* stream)
{
    if (op < IMM_FIELD_ADD || op > IMM_FIELD_MUL || count < 0) return IMM_ERR_ARG;
    if (count == 0) return IMM_OK;
    if (!d_x || !d_y || !d_out) return IMM_ERR_ARG;
    CU(launch_field_binop(op, d_x, d_y, d_out, count, (cudaStream_t)stream));
    return IMM_OK;
}

int imm_eq_table(const imm_fe* r_host, int nvars, imm_fe* d_out, void* stream)
{
    if (!d_out || (nvars > 0 && !r_host)) return IMM_ERR_ARG;
    if (nvars < 0 || nvars > MAX_EQ_VARS) return IMM_ERR_SHAPE;
    if ((uintptr_t)d_out % 16 != 0) return IMM_ERR_ALIGN;
    EqDirect r;
    memset(&r, 0, sizeof(r));
    for (int t = 0; t < nvars; t++) {
        if (r_host[t] >= IMM_P) return IMM_ERR_NONCANONICAL;
        r.r[t] = r_host[t];
    }
    CU(launch_eq_direct(r, nvars, d_out, (cudaStream_t)stream));
    return IMM_OK;
}

size_t imm_mle_workspace(int dtype, int64_t rows, int64_t cols, int bind)
{
    if ((dtype != IMM_I8 && dtype != IMM_I32) || rows <= 0 || cols <= 0 || rows > MAX_EXTENT ||
        cols > MAX_EXTENT || (bind != IMM_BIND_ROWS && bind != IMM_BIND_COLS))
        return 0;
    std::vector<Shape> one{{rows, cols}};
    size_t parts;
    if (bind == IMM_BIND_ROWS) {
        int tr = pick_tile_rows(one, rowbind_cols(dtype), "IMM_TILE_ROWS_A");
        int64_t nrb = (rows + tr - 1) / tr, ncc = (cols + rowbind_cols(dtype) - 1) / rowbind_cols(dtype);
        size_t vec_parts = (size_t)nrb * cols, pt_parts = (size_t)(nrb * ncc);   // partial_eval / eval_point
        parts = vec_parts > pt_parts ? vec_parts : pt_parts;
    } else {
        int64_t ncc = (cols + colbind_cols(dtype) - 1) / colbind_cols(dtype);
        parts = (size_t)ncc * rows;
    }
    size_t need = ALIGN + align_up(parts * sizeof(imm_fe));       // the integer-pipe kernels
    const MlePlan a = plan_mle(dtype, rows, cols, bind == IMM_BIND_ROWS ? OP_ROWS : OP_COLS);
    if (a.mma && a.total > need) need = a.total;
    if (bind == IMM_BIND_ROWS) {                                    // imm_mle_eval_point sizes itself with BIND_ROWS
        const MlePlan b = plan_mle(dtype, rows, cols, OP_POINT);
        if (b.mma && b.total > need) need = b.total;
    }
    return need;
}

int imm_mle_partial_eval(const void* d_mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
                         int bind, const imm_fe* d_eq, imm_fe* d_out,
                         void* d_ws, size_t ws_bytes, void* stream)
{
    int rc = check_matrix_args(d_mat, dtype, rows, cols, ld);
    if (rc != IMM_OK) return rc;
    if (!d_eq || !d_out || !d_ws || (bind != IMM_BIND_ROWS && bind != IMM_BIND_COLS)) return IMM_ERR_ARG;
    if ((uintptr_t)d_ws % 16 != 0 || (uintptr_t)d_out % 16 != 0 || (uintptr_t)d_eq % 8 != 0) return IMM_ERR_ALIGN;
    if (ws_bytes < imm_mle_workspace(dtype, rows, cols, bind)) return IMM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    std::vector<Shape> one{{rows, cols}};
    MatJob* d_job = (MatJob*)d_ws;
    MatJob j;
    const MlePlan mp = plan_mle(dtype, rows, cols, bind == IMM_BIND_ROWS ? OP_ROWS : OP_COLS);
    if (mp.mma) {
        // tensor-core path: limb table of the caller's eq weights, then the contraction
        char* base = (char*)d_ws;
        uint32_t* wtab = (uint32_t*)(base + mp.off_w);
        imm_fe* parts = (imm_fe*)(base + mp.off_parts);
        const bool by_rows = bind == IMM_BIND_ROWS;
        const int64_t extent = by_rows ? rows : cols;
        char hdr[ALIGN + 2 * sizeof(EqTask)];
        memset(hdr, 0, sizeof(hdr));
        fill_job(j, d_mat, dtype, rows, cols, ld, mp.g.rows, mp.g.width);
        j.wtab = wtab;
        j.chunk = mp.g.width;
        const bool direct = (by_rows ? mp.nrb : mp.ncc) == 1;
        j.out = direct ? d_out : parts;
        if (by_rows) j.eq_row = d_eq; else j.eq_col = d_eq;
        memcpy(hdr, &j, sizeof(j));
        EqTask t{nullptr, 0, 0, 0u, 0, by_rows ? wtab : nullptr, by_rows ? nullptr : wtab, nullptr, (int32_t)extent, 0,
                 nullptr, d_eq};
        memcpy(hdr + ALIGN, &t, sizeof(t));
        CU(cudaMemcpyAsync(base, hdr, sizeof(hdr), cudaMemcpyHostToDevice, st));
        const int64_t pad = by_rows ? 32 : 256;
        CU(launch_eq_batch((const EqTask*)(base + mp.off_tasks), 1, (extent + pad - 1) / pad * pad, st));
        const uint32_t ntiles = (uint32_t)(mp.nrb * mp.ncc);
        if (by_rows) {
            CU(launch_rowmma(d_job, 1, ntiles, mp.g.width / 128, st));
            if (!direct) CU(launch_sum_parts(parts, (int)mp.nrb, cols, d_out, st));
        } else {
            CU(launch_bytedot(false, false, 2, d_job, 1, ntiles, st));
            if (!direct) CU(launch_sum_parts(parts, (int)mp.ncc, rows, d_out, st));
        }
        return IMM_OK;
    }
    imm_fe* d_parts = (imm_fe*)((char*)d_ws + ALIGN);
    if (bind == IMM_BIND_ROWS) {
        int tr = pick_tile_rows(one, rowbind_cols(dtype), "IMM_TILE_ROWS_A");
        fill_job(j, d_mat, dtype, rows, cols, ld, tr, rowbind_cols(dtype));
        j.eq_row = d_eq;
        j.out = j.nrb == 1 ? d_out : d_parts;
        CU(cudaMemcpyAsync(d_job, &j, sizeof(j), cudaMemcpyHostToDevice, st));
        CU(launch_rowbind(dtype, false, d_job, 1, (uint32_t)(j.nrb * j.ncc), st));
        if (j.nrb > 1) CU(launch_sum_parts(d_parts, j.nrb, cols, d_out, st));
    } else {
        int tr = pick_tile_rows(one, colbind_cols(dtype), "IMM_TILE_ROWS_B");
        fill_job(j, d_mat, dtype, rows, cols, ld, tr, colbind_cols(dtype));
        j.eq_col = d_eq;
        j.out = j.ncc == 1 ? d_out : d_parts;
        CU(cudaMemcpyAsync(d_job, &j, sizeof(j), cudaMemcpyHostToDevice, st));
        CU(launch_colbind(dtype, d_job, 1, (uint32_t)(j.nrb * j.ncc), st));
        if (j.ncc > 1) CU(launch_sum_parts(d_parts, j.ncc, rows, d_out, st));
    }
    return IMM_OK;
}

int imm_mle_eval_point(const void* d_mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
                       const imm_fe* d_eq_row, const imm_fe* d_eq_col, imm_fe* d_out,
                       void* d_ws, size_t ws_bytes, void* stream)
{
    int rc = check_matrix_args(d_mat, dtype, rows, cols, ld);
    if (rc != IMM_OK) return rc;
    if (!d_eq_row || !d_eq_col || !d_out || !d_ws) return IMM_ERR_ARG;
    if ((uintptr_t)d_ws % 16 != 0 || (uintptr_t)d_out % 8 != 0) return IMM_ERR_ALIGN;
    if (ws_bytes < imm_mle_workspace(dtype, rows, cols, IMM_BIND_ROWS)) return IMM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    std::vector<Shape> one{{rows, cols}};
    MatJob* d_job = (MatJob*)d_ws;
    MatJob j;
    const MlePlan mp = plan_mle(dtype, rows, cols, OP_POINT);
    if (mp.mma) {
        // tensor-core path: limb table of eq_col (and, for int32, the sums of both eq tables for the
        // 2^31 offset of the unsigned byte view), the point contraction, the final sum
        char* base = (char*)d_ws;
        uint32_t* wtab = (uint32_t*)(base + mp.off_w);
        imm_fe* parts = (imm_fe*)(base + mp.off_parts);
        imm_fe* sr = (imm_fe*)(base + mp.off_sr);
        imm_fe* sc = (imm_fe*)(base + mp.off_sc);
        const bool i32 = dtype == IMM_I32;
        char hdr[ALIGN + 2 * sizeof(EqTask)];
        memset(hdr, 0, sizeof(hdr));
        const int width_elems = mp.g.width / (int)elem_size(dtype);
        fill_job(j, d_mat, dtype, rows, cols, ld, mp.g.rows, width_elems);
        j.wtab = wtab;
        j.chunk = mp.g.width;
        j.eq_row = d_eq_row;
        j.eq_col = d_eq_col;
        j.out = parts;
        memcpy(hdr, &j, sizeof(j));
        EqTask tc{nullptr, 0, 0, 0u, 0, nullptr, i32 ? nullptr : wtab, i32 ? wtab : nullptr, (int32_t)cols, 0,
                  i32 ? sc : nullptr, d_eq_col};
        EqTask tr_{nullptr, 0, 0, 0u, 0, nullptr, nullptr, nullptr, (int32_t)rows, 0, sr, d_eq_row};
        memcpy(hdr + ALIGN, &tc, sizeof(tc));
        memcpy(hdr + ALIGN + sizeof(EqTask), &tr_, sizeof(tr_));
        CU(cudaMemcpyAsync(base, hdr, sizeof(hdr), cudaMemcpyHostToDevice, st));
        int64_t cover = (cols + 255) / 256 * 256;
        if (i32 && rows > cover) cover = rows;
        CU(launch_eq_batch((const EqTask*)(base + mp.off_tasks), i32 ? 2 : 1, cover, st));
        CU(launch_bytedot(i32, true, 1, d_job, 1, (uint32_t)(mp.nrb * mp.ncc), st));
        CU(launch_point_finish(parts, mp.nparts, sr, mp.n_sr, sc, mp.n_sc, d_out, st));
        return IMM_OK;
    }
    imm_fe* d_parts = (imm_fe*)((char*)d_ws + ALIGN);
    int tr = pick_tile_rows(one, rowbind_cols(dtype), "IMM_TILE_ROWS_A");
    fill_job(j, d_mat, dtype, rows, cols, ld, tr, rowbind_cols(dtype));
    j.eq_row = d_eq_row;
    j.eq_col = d_eq_col;
    j.out = d_parts;
    CU(cudaMemcpyAsync(d_job, &j, sizeof(j), cudaMemcpyHostToDevice, st));
    CU(launch_rowbind(dtype, true, d_job, 1, (uint32_t)(j.nrb * j.ncc), st));
    CU(launch_sum_all(d_parts, (int64_t)j.nrb * j.ncc, d_out, st));
    return IMM_OK;
}

int imm_profile_enable(int capacity)
{
    if (capacity < 0 || capacity > 4096) return IMM_ERR_ARG;
    for (cudaEvent_t e : g_prof_ev) cudaEventDestroy(e);
    g_prof_ev.clear();
    g_prof_calls = 0;
    if (capacity == 0) return IMM_OK;
    std::vector<cudaEvent_t> ev((size_t)capacity * PROF_EV);
    for (size_t i = 0; i < ev.size(); i++) {
        cudaError_t e = cudaEventCreate(&ev[i]);
        if (e != cudaSuccess) {
            for (size_t j = 0; j < i; j++) cudaEventDestroy(ev[j]);
            return cuda_fail(e);
        }
    }
    g_prof_ev.swap(ev);
    return IMM_OK;
}

int64_t imm_profile_calls(void) { return g_prof_calls; }

int imm_profile_read(int64_t call, float* ms_host, int count)
{
    if (!ms_host || count != IMM_PROFILE_PHASES || g_prof_ev.empty()) return IMM_ERR_ARG;
    const int64_t cap = (int64_t)(g_prof_ev.size() / PROF_EV);
    if (call < 0 || call >= g_prof_calls || call < g_prof_calls - cap) return IMM_ERR_ARG;
    cudaEvent_t* ev = &g_prof_ev[(size_t)(call % cap) * PROF_EV];
    CU(cudaEventSynchronize(ev[PROF_EV - 1]));                  // the end of the last phase: everything before it is done
    for (int i = 0; i < IMM_PROFILE_PHASES; i++) CU(cudaEventElapsedTime(&ms_host[i], ev[2 * i], ev[2 * i + 1]));
    return IMM_OK;
}

size_t imm_sumcheck_matmul_workspace(const imm_matmul_desc* descs_host, int nproofs)
{
    Plan p = make_plan(descs_host, nproofs);
    return p.status == IMM_OK ? p.total_bytes : 0;
}

int imm_sumcheck_matmul_launches(const imm_matmul_desc* descs_host, int nproofs)
{
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return 0;
    return p.fused ? 3 : 5;
}

// The launch sequence of a batch.  shared_round_id: null = every proof draws its round challenges
// under its own proof_id and runs its own ceil(log2 k) rounds; else all proofs draw them under that
// one id and run the rounds of the largest k (a batched proof).
// fs: null = public coins from the generator; else the challenges are hashed from the commitments
// and the transcript (non-interactive proof) and fs describes the extra device arrays.
struct FsArgs {
    const uint8_t* d_com;      // nproofs x 96 bytes
    char* ext;                 // device region laid out by fs_layout
    bool batched;              // one proof for all members (shared_round_id carries the batch id)
};

struct FsLayout {
    size_t off_fs = 0, off_points = 0, off_state = 0, bytes = 0;
    std::vector<size_t> off_tabs;
    size_t off_T = 0, off_bstate = 0, off_rho = 0, off_c0 = 0, off_partial = 0, off_r = 0;   // batched proof only
};

static FsLayout fs_layout(const imm_matmul_desc* descs, int nproofs, int shared_b /* 0: per proof */)
{
    FsLayout L;
    size_t off = align_up((size_t)nproofs * sizeof(FsProof));
    L.off_points = off; off = align_up(off + (size_t)nproofs * 2 * FS_POINT_SLOTS * sizeof(imm_fe));
    L.off_state = off;  off = align_up(off + (size_t)nproofs * 8 * sizeof(uint32_t));
    L.off_tabs.resize(nproofs);
    for (int i = 0; i < nproofs; i++) {
        L.off_tabs[i] = off;
        off = align_up(off + 2 * (sizeof(imm_fe) << (shared_b ? shared_b : ceil_log2(descs[i].k))));
    }
    L.off_T = off;       off = align_up(off + 8 * sizeof(uint32_t));
    L.off_bstate = off;  off = align_up(off + 8 * sizeof(uint32_t));
    L.off_rho = off;     off = align_up(off + (size_t)nproofs * sizeof(imm_fe));
    L.off_c0 = off;      off = align_up(off + (size_t)nproofs * sizeof(imm_fe));
    L.off_partial = off; off = align_up(off + (size_t)nproofs * 3 * sizeof(imm_fe));
    L.off_r = off;       off = align_up(off + MAX_K_VARS * sizeof(imm_fe));
    L.bytes = off;
    return L;
}

// vf: non-null = the verifier's pass: the rounds are replaced by the inner products with E_k and
// d_transcripts receives three words per proof (stride 3): its own c0, a_fin, b_fin.
struct VerifyArgs {
    char* ext;                 // device region laid out by verify_layout
    const imm_fe* points_host; // null: challenges from the generator; else nproofs x VERIFY_POINT_SLOTS given values
};

struct VerifyLayout {
    size_t off_ex = 0, off_tasks = 0, off_points = 0, bytes = 0;
    std::vector<size_t> off_ek;
};

static VerifyLayout verify_layout(const imm_matmul_desc* descs, int nproofs, int shared_b /* 0: per proof */)
{
    VerifyLayout L;
    size_t off = align_up((size_t)nproofs * sizeof(ExpectDev));
    L.off_tasks = off;  off = align_up(off + (size_t)nproofs * sizeof(EqTask));
    L.off_points = off; off = align_up(off + (size_t)nproofs * VERIFY_POINT_SLOTS * sizeof(imm_fe));
    L.off_ek.resize(nproofs);
    for (int i = 0; i < nproofs; i++) {
        L.off_ek[i] = off;
        off = align_up(off + (sizeof(imm_fe) << (shared_b ? shared_b : ceil_log2(descs[i].k))));
    }
    L.bytes = off;
    return L;
}

static int prove_batch(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed,
                       const uint64_t* shared_round_id, const FsArgs* fs, const VerifyArgs* vf,
                       imm_fe* d_transcripts, int64_t stride,
                       int32_t* d_status, void* d_ws, size_t ws_bytes, void* stream)
{
    if (!d_transcripts || !d_status || !d_ws) return IMM_ERR_ARG;
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return p.status;
    int rc = vf ? IMM_OK : check_stride(descs_host, nproofs, stride);
    if (rc != IMM_OK) return rc;
    if ((uintptr_t)d_ws % 16 != 0 || (uintptr_t)d_transcripts % 8 != 0 || (uintptr_t)d_status % 4 != 0)
        return IMM_ERR_ALIGN;
    if (ws_bytes < p.total_bytes) return IMM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)d_ws;

    // header image: per-proof state, the three job lists, the eq tasks
    std::vector<char> hdr(p.header_bytes, 0);
    ProofDev* pd = (ProofDev*)(hdr.data() + p.off_proofs);
    MatJob* ja = (MatJob*)(hdr.data() + p.off_jobs_a);
    MatJob* jb = (MatJob*)(hdr.data() + p.off_jobs_b);
    MatJob* jc = (MatJob*)(hdr.data() + p.off_jobs_c);
    EqTask* eq = (EqTask*)(hdr.data() + p.off_eq);
    FusedJob* fj = p.fused ? (FusedJob*)(hdr.data() + p.off_fjobs) : nullptr;
    const bool tables_ready = p.fused && !fs && !vf;            // reduce_parts_kernel finishes the round tables
    const int acols = p.cols_a, bcols = p.cols_b, ccols = p.cols_c;
    FsLayout fsl;
    std::vector<FsProof> fsp;
    if (fs) {
        fsl = fs_layout(descs_host, nproofs, fs->batched ? p.max_b : 0);
        fsp.assign(nproofs, FsProof{});
    }
    VerifyLayout vl;
    std::vector<ExpectDev> exd;
    std::vector<EqTask> ekt;
    if (vf) {
        vl = verify_layout(descs_host, nproofs, shared_round_id ? p.max_b : 0);
        exd.assign(nproofs, ExpectDev{});
        ekt.assign(nproofs, EqTask{});
    }
    uint32_t ta = 0, tb = 0, tc = 0;
    for (int i = 0; i < nproofs; i++) {
        const imm_matmul_desc& d = descs_host[i];
        const Plan::PerProof& q = p.pp[i];
        ProofDev& P = pd[i];
        P.e_row = (imm_fe*)(base + q.e_row);
        P.e_col = (imm_fe*)(base + q.e_col);
        P.part_a = (imm_fe*)(base + q.part_a);
        P.part_b = (imm_fe*)(base + q.part_b);
        P.part_c = (imm_fe*)(base + q.part_c);
        P.round_id = shared_round_id ? *shared_round_id : d.proof_id;
        P.m = (int32_t)d.m; P.k = (int32_t)d.k; P.n = (int32_t)d.n;
        P.a = q.a; P.b = shared_round_id ? p.max_b : q.b; P.c = q.c;   // a batched proof pads every k to the largest 2^b
        P.n_part_a = q.n_part_a; P.n_part_b = q.n_part_b; P.n_part_c = q.n_part_c;
        P.sum_row = p.fused ? nullptr : (imm_fe*)(base + q.sum_row);
        P.sum_col = p.fused ? nullptr : (imm_fe*)(base + q.sum_col);
        P.n_sum_row = q.n_sum_row; P.n_sum_col = q.n_sum_col;
        P.c_offset = p.mma ? 1 : 0;
        P.seed = seed; P.proof_id = d.proof_id;
        P.pt_row = P.pt_col = nullptr;
        P.tab = tables_ready ? (imm_fe*)(base + q.tab) : nullptr;
        P.c0_ready = tables_ready ? (imm_fe*)(base + q.c0_ready) : nullptr;

        if (!p.fused) {
            fill_job(ja[i], d.A, IMM_I8, d.m, d.k, d.lda, p.rows_a, acols);
            ja[i].eq_row = P.e_row; ja[i].out = (imm_fe*)P.part_a; ja[i].tile0 = ta;
            ta += (uint32_t)(ja[i].nrb * ja[i].ncc);
            fill_job(jb[i], d.B, IMM_I8, d.k, d.n, d.ldb, p.rows_b, bcols);
            jb[i].eq_col = P.e_col; jb[i].out = (imm_fe*)P.part_b; jb[i].tile0 = tb; jb[i].chunk = bcols;
            tb += (uint32_t)(jb[i].nrb * jb[i].ncc);
            fill_job(jc[i], d.C, IMM_I32, d.m, d.n, d.ldc, p.rows_c, ccols);
            jc[i].eq_row = P.e_row; jc[i].eq_col = P.e_col; jc[i].out = (imm_fe*)P.part_c; jc[i].tile0 = tc;
            jc[i].chunk = 4 * ccols;
            tc += (uint32_t)(jc[i].nrb * jc[i].ncc);
        }

        if (p.mma && !p.fused) {
            ja[i].wtab = (const uint32_t*)(base + q.w_rows);
            jb[i].wtab = (const uint32_t*)(base + q.w_cols_b);
            jc[i].wtab = (const uint32_t*)(base + q.w_cols_c);
        }
        const imm_fe* pts = fs ? (const imm_fe*)(fs->ext + fsl.off_points) + (size_t)i * 2 * FS_POINT_SLOTS : nullptr;
        eq[2 * i] = EqTask{P.e_row, seed, d.proof_id, 1u, q.a,
                           p.mma ? (uint32_t*)(base + q.w_rows) : nullptr, nullptr, nullptr, (int32_t)d.m, 0,
                           p.mma ? (imm_fe*)(base + q.sum_row) : nullptr};
        eq[2 * i + 1] = EqTask{P.e_col, seed, d.proof_id, 2u, q.c, nullptr,
                               p.mma ? (uint32_t*)(base + q.w_cols_b) : nullptr,
                               p.mma ? (uint32_t*)(base + q.w_cols_c) : nullptr, (int32_t)d.n, 0,
                               p.mma ? (imm_fe*)(base + q.sum_col) : nullptr};
        if (vf) {
            const imm_fe* given = vf->points_host
                ? (const imm_fe*)(vf->ext + vl.off_points) + (size_t)i * VERIFY_POINT_SLOTS : nullptr;
            if (given) {
                eq[2 * i].point = given;
                eq[2 * i + 1].point = given + FS_POINT_SLOTS;
                P.pt_row = given; P.pt_col = given + FS_POINT_SLOTS;
            }
            imm_fe* e_k = (imm_fe*)(vf->ext + vl.off_ek[i]);
            ekt[i] = EqTask{e_k, seed, P.round_id, 3u, P.b, nullptr, nullptr, nullptr, (int32_t)d.k, 0, nullptr};
            if (given) ekt[i].point = given + 2 * FS_POINT_SLOTS;
            exd[i].e_k = e_k;
        }
        if (fs) {
            eq[2 * i].point = pts;
            eq[2 * i + 1].point = pts + FS_POINT_SLOTS;
            P.pt_row = pts; P.pt_col = pts + FS_POINT_SLOTS;
            FsProof& F = fsp[i];
            F.com = fs->d_com + (size_t)i * 96;
            F.points = (imm_fe*)pts;
            F.state = (uint32_t*)(fs->ext + fsl.off_state) + (size_t)i * 8;
            F.ta = (imm_fe*)(fs->ext + fsl.off_tabs[i]);
            F.tb = F.ta + ((size_t)1 << P.b);
            F.proof_id = d.proof_id;
            F.one = 1;
        }
    }
    if (!p.fused && (ta != p.tiles_a || tb != p.tiles_b || tc != p.tiles_c)) return IMM_ERR_ARG;   // planner invariant
    if (p.fused) {
        // the fused launch's job list, kind-major: every A, every C, every B (the order of the segments)
        for (int kind = 0; kind < 3; kind++)
            for (int i = 0; i < nproofs; i++) {
                const imm_matmul_desc& d = descs_host[i];
                const Plan::FusedGeom& g = p.fg[i];
                FusedJob& F = fj[kind * nproofs + i];
                memset(&F, 0, sizeof(F));
                if (kind == 0) {
                    fill_job(F.mj, d.A, IMM_I8, d.m, d.k, d.lda, g.rows_a, FUSED_A_TILE_COLS);
                    F.mj.out = (imm_fe*)pd[i].part_a;
                    F.kind = JOB_ROWBIND;
                } else if (kind == 1) {
                    fill_job(F.mj, d.C, IMM_I32, d.m, d.n, d.ldc, MAX_TILE_ROWS, g.chunk_c / 4);
                    F.mj.chunk = g.chunk_c;
                    F.mj.out = (imm_fe*)pd[i].part_c;
                    F.kind = JOB_POINT;
                    F.seg0 = g.seg0_c;
                } else {
                    fill_job(F.mj, d.B, IMM_I8, d.k, d.n, d.ldb, MAX_TILE_ROWS, g.chunk_b);
                    F.mj.chunk = g.chunk_b;
                    F.mj.out = (imm_fe*)pd[i].part_b;
                    F.kind = JOB_COLBIND;
                }
                F.seed = seed; F.proof_id = d.proof_id;
                F.pt_row = pd[i].pt_row; F.pt_col = pd[i].pt_col;
                F.a = p.pp[i].a; F.c = p.pp[i].c;
            }
        memcpy(hdr.data() + p.off_segs, p.segs.data(), sizeof(FusedSeg) * p.segs.size());
        memcpy(hdr.data() + p.off_block_first, p.block_first.data(), sizeof(uint32_t) * p.block_first.size());
    }

    const bool prof = !g_prof_ev.empty();
    cudaEvent_t* pev = prof ? &g_prof_ev[(size_t)(g_prof_calls % (int64_t)(g_prof_ev.size() / PROF_EV)) * PROF_EV]
                            : nullptr;
    // phase i is timed by events 2i (start) and 2i+1 (end), each on the stream its kernel runs on
#define PROF_MARK(i, stream_) do { if (prof) CU(cudaEventRecord(pev[i], stream_)); } while (0)
    CU(cudaMemcpyAsync(base, hdr.data(), hdr.size(), cudaMemcpyHostToDevice, st));
    if (fs) {
        CU(cudaMemcpyAsync(fs->ext + fsl.off_fs, fsp.data(), fsp.size() * sizeof(FsProof), cudaMemcpyHostToDevice, st));
        CU(launch_fs_points((const ProofDev*)(base + p.off_proofs), (const FsProof*)(fs->ext + fsl.off_fs), nproofs, st));
    }
    if (vf) {
        CU(cudaMemcpyAsync(vf->ext + vl.off_ex, exd.data(), exd.size() * sizeof(ExpectDev), cudaMemcpyHostToDevice, st));
        CU(cudaMemcpyAsync(vf->ext + vl.off_tasks, ekt.data(), ekt.size() * sizeof(EqTask), cudaMemcpyHostToDevice, st));
        if (vf->points_host)
            CU(cudaMemcpyAsync(vf->ext + vl.off_points, vf->points_host,
                               (size_t)nproofs * VERIFY_POINT_SLOTS * sizeof(imm_fe), cudaMemcpyHostToDevice, st));
    }
    // (While phase timing is on, the events recorded between the launches of a fused batch undo their
    // programmatic overlap: whole steps are timed with it off.)
    PROF_MARK(0, st);
    if (!p.fused) CU(launch_eq_batch((const EqTask*)(base + p.off_eq), 2 * nproofs, p.max_cover, st));
    if (vf) CU(launch_eq_batch((const EqTask*)(vf->ext + vl.off_tasks), nproofs, (int64_t)1 << p.max_b, st));
    PROF_MARK(1, st);
    PROF_MARK(2, st);
    if (p.fused)
        CU(launch_fused_contract((const FusedJob*)(base + p.off_fjobs), (const FusedSeg*)(base + p.off_segs),
                                 (const uint32_t*)(base + p.off_block_first), (uint32_t)p.block_first.size() - 1, st));
    else if (p.mma) CU(launch_bytedot(true, true, p.mt_c, (const MatJob*)(base + p.off_jobs_c), nproofs, p.tiles_c, st));
    else CU(launch_rowbind(IMM_I32, true, (const MatJob*)(base + p.off_jobs_c), nproofs, p.tiles_c, st));
    PROF_MARK(3, st);
    PROF_MARK(4, st);
    if (p.fused) {}
    else if (p.mma) CU(launch_rowmma((const MatJob*)(base + p.off_jobs_a), nproofs, p.tiles_a, p.cols_a / 128, st));
    else CU(launch_rowbind(IMM_I8, false, (const MatJob*)(base + p.off_jobs_a), nproofs, p.tiles_a, st));
    PROF_MARK(5, st);
    PROF_MARK(6, st);
    if (p.fused) {}
    else if (p.mma) CU(launch_bytedot(false, false, p.mt_b, (const MatJob*)(base + p.off_jobs_b), nproofs, p.tiles_b, st));
    else CU(launch_colbind(IMM_I8, (const MatJob*)(base + p.off_jobs_b), nproofs, p.tiles_b, st));
    PROF_MARK(7, st);
    PROF_MARK(8, st);
    if (vf)
        CU(launch_expected((const ProofDev*)(base + p.off_proofs), (const ExpectDev*)(vf->ext + vl.off_ex), nproofs,
                           d_transcripts, d_status, st));
    else if (fs && fs->batched) {
        FsBatch fb{};
        fb.T = (uint32_t*)(fs->ext + fsl.off_T);
        fb.state = (uint32_t*)(fs->ext + fsl.off_bstate);
        fb.rho = (imm_fe*)(fs->ext + fsl.off_rho);
        fb.c0 = (imm_fe*)(fs->ext + fsl.off_c0);
        fb.partial = (imm_fe*)(fs->ext + fsl.off_partial);
        fb.r = (imm_fe*)(fs->ext + fsl.off_r);
        fb.batch_id = *shared_round_id;
        fb.nproofs = nproofs;
        fb.b = p.max_b;
        fb.one = 1;
        CU(launch_fs_batched_rounds((const ProofDev*)(base + p.off_proofs), (const FsProof*)(fs->ext + fsl.off_fs), fb,
                                    d_transcripts, d_status, st));
    } else if (fs)
        CU(launch_sumcheck_fs((const ProofDev*)(base + p.off_proofs), (const FsProof*)(fs->ext + fsl.off_fs), nproofs,
                              d_transcripts, stride, d_status, st));
    else {
        if (tables_ready) CU(launch_reduce_parts((const ProofDev*)(base + p.off_proofs), nproofs, p.max_b, st));
        CU(launch_sumcheck((const ProofDev*)(base + p.off_proofs), nproofs, seed, d_transcripts, stride,
                           d_status, p.max_b, env_int("IMM_SC_CLUSTER", 0), tables_ready, st));
    }
    PROF_MARK(9, st);
#undef PROF_MARK
    if (prof) g_prof_calls++;
    return IMM_OK;
}

int imm_sumcheck_matmul_prove(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed,
                              imm_fe* d_transcripts, int64_t stride, int32_t* d_status,
                              void* d_ws, size_t ws_bytes, void* stream)
{
    return prove_batch(descs_host, nproofs, seed, nullptr, nullptr, nullptr, d_transcripts, stride, d_status, d_ws,
                       ws_bytes, stream);
}

// Batched proof: the per-proof transcripts (shared round challenges) go to the head of the
// workspace, the prover's own workspace follows, and one more launch combines them.
static int batched_layout(const imm_matmul_desc* descs_host, int nproofs, int* b, size_t* rows_bytes, size_t* total)
{
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return p.status;
    if (nproofs > IMM_BATCH_MAX_PROOFS) return IMM_ERR_LIMIT;
    *b = p.max_b;
    *rows_bytes = align_up((size_t)nproofs * (size_t)(3 * *b + 3) * sizeof(imm_fe));
    *total = *rows_bytes + p.total_bytes;
    return IMM_OK;
}

size_t imm_sumcheck_matmul_batched_workspace(const imm_matmul_desc* descs_host, int nproofs)
{
    int b;
    size_t rows, total;
    return batched_layout(descs_host, nproofs, &b, &rows, &total) == IMM_OK ? total : 0;
}

int64_t imm_sumcheck_batched_transcript_len(int nrounds, int nproofs)
{
    if (nrounds < 0 || nrounds > 64 || nproofs <= 0 || nproofs > IMM_BATCH_MAX_PROOFS) return 0;
    return 1 + 3 * (int64_t)nrounds + 3 * (int64_t)nproofs;
}

int imm_sumcheck_matmul_prove_batched(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed,
                                      uint64_t batch_id, imm_fe* d_transcript, int32_t* d_status,
                                      void* d_ws, size_t ws_bytes, void* stream)
{
    if (!d_transcript || !d_status || !d_ws) return IMM_ERR_ARG;
    int b;
    size_t rows, total;
    int rc = batched_layout(descs_host, nproofs, &b, &rows, &total);
    if (rc != IMM_OK) return rc;
    if ((uintptr_t)d_ws % ALIGN != 0 || (uintptr_t)d_transcript % 8 != 0) return IMM_ERR_ALIGN;
    if (ws_bytes < total) return IMM_ERR_WORKSPACE;
    imm_fe* d_rows = (imm_fe*)d_ws;
    const int64_t stride = 3 * b + 3;
    rc = prove_batch(descs_host, nproofs, seed, &batch_id, nullptr, nullptr, d_rows, stride, d_status,
                     (char*)d_ws + rows, ws_bytes - rows, stream);
    if (rc != IMM_OK) return rc;
    CU(launch_combine(d_rows, stride, nproofs, b, seed, batch_id, d_transcript, (cudaStream_t)stream));
    return IMM_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ the verifier's pass -----

extern "C" {

size_t imm_sumcheck_expected_workspace(const imm_matmul_desc* descs_host, int nproofs, int batched)
{
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return 0;
    return verify_layout(descs_host, nproofs, batched ? p.max_b : 0).bytes + p.total_bytes;
}

int imm_sumcheck_expected(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed, const uint64_t* batch_id,
                          const imm_fe* points_host, imm_fe* d_expected, int32_t* d_status,
                          void* d_ws, size_t ws_bytes, void* stream)
{
    if (!d_expected || !d_status || !d_ws) return IMM_ERR_ARG;
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return p.status;
    if ((uintptr_t)d_ws % ALIGN != 0 || (uintptr_t)d_expected % 8 != 0) return IMM_ERR_ALIGN;
    if (points_host)
        for (int64_t i = 0; i < (int64_t)nproofs * VERIFY_POINT_SLOTS; i++)
            if (points_host[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
    const size_t ext = verify_layout(descs_host, nproofs, batch_id ? p.max_b : 0).bytes;
    if (ws_bytes < ext + p.total_bytes) return IMM_ERR_WORKSPACE;
    // a pageable copy: its upload is staged before the call returns, whatever memory the caller's array is in
    std::vector<imm_fe> points;
    if (points_host) points.assign(points_host, points_host + (size_t)nproofs * VERIFY_POINT_SLOTS);
    VerifyArgs vf{(char*)d_ws, points_host ? points.data() : nullptr};
    return prove_batch(descs_host, nproofs, seed, batch_id, nullptr, &vf, d_expected, 3, d_status,
                       (char*)d_ws + ext, ws_bytes - ext, stream);
}

}  // extern "C"

// ------------------------------------------------------------------ non-interactive proof ---

extern "C" {

size_t imm_sumcheck_matmul_fs_workspace(const imm_matmul_desc* descs_host, int nproofs)
{
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return 0;
    return fs_layout(descs_host, nproofs, 0).bytes + p.total_bytes;
}

int imm_sumcheck_matmul_prove_fs(const imm_matmul_desc* descs_host, int nproofs, const uint8_t* d_commitments,
                                 imm_fe* d_transcripts, int64_t stride, int32_t* d_status,
                                 void* d_ws, size_t ws_bytes, void* stream)
{
    if (!d_commitments || !d_ws) return IMM_ERR_ARG;
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return p.status;
    if ((uintptr_t)d_ws % ALIGN != 0) return IMM_ERR_ALIGN;
    const size_t ext = fs_layout(descs_host, nproofs, 0).bytes;
    if (ws_bytes < ext + p.total_bytes) return IMM_ERR_WORKSPACE;
    FsArgs fs{d_commitments, (char*)d_ws, false};
    return prove_batch(descs_host, nproofs, 0, nullptr, &fs, nullptr, d_transcripts, stride, d_status,
                       (char*)d_ws + ext, ws_bytes - ext, stream);
}

size_t imm_sumcheck_matmul_fs_batched_workspace(const imm_matmul_desc* descs_host, int nproofs)
{
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK || nproofs > FS_BATCH_MAX) return 0;
    return fs_layout(descs_host, nproofs, p.max_b).bytes + p.total_bytes;
}

int imm_sumcheck_matmul_prove_fs_batched(const imm_matmul_desc* descs_host, int nproofs, const uint8_t* d_commitments,
                                         uint64_t batch_id, imm_fe* d_transcript, int32_t* d_status,
                                         void* d_ws, size_t ws_bytes, void* stream)
{
    if (!d_commitments || !d_ws) return IMM_ERR_ARG;
    Plan p = make_plan(descs_host, nproofs);
    if (p.status != IMM_OK) return p.status;
    if (nproofs > FS_BATCH_MAX) return IMM_ERR_LIMIT;
    if ((uintptr_t)d_ws % ALIGN != 0) return IMM_ERR_ALIGN;
    const size_t ext = fs_layout(descs_host, nproofs, p.max_b).bytes;
    if (ws_bytes < ext + p.total_bytes) return IMM_ERR_WORKSPACE;
    FsArgs fs{d_commitments, (char*)d_ws, true};
    return prove_batch(descs_host, nproofs, 0, &batch_id, &fs, nullptr, d_transcript, 3 * p.max_b + 3, d_status,
                       (char*)d_ws + ext, ws_bytes - ext, stream);
}

}  // extern "C"

namespace {

// host side of the transcript hashing (the same byte strings as the kernels')
uint64_t fs_fe_host(const uint32_t (&h)[8])
{
    const uint64_t v = ((uint64_t)h[0] << 32) | h[1];
    return v >= IMM_P ? v - IMM_P : v;
}

void put_le(uint8_t* dst, uint64_t v, int nbytes)
{
    for (int q = 0; q < nbytes; q++) dst[q] = (uint8_t)(v >> (8 * q));
}

void fs_absorb_host(uint32_t (&s)[8], uint8_t tag, const uint64_t* vals, int nvals)
{
    uint8_t m[64];
    m[0] = tag;
    imm_sha::digest_bytes(s, m + 1);
    for (int i = 0; i < nvals; i++) put_le(m + 33 + 8 * i, vals[i], 8);
    imm_sha::sha256_short(m, 33 + 8 * (uint32_t)nvals, s, 1);
}

void fs_statement_host(const uint8_t* com, int64_t m_, int64_t k, int64_t n, uint64_t proof_id, uint32_t (&s0)[8])
{
    uint8_t m[136];
    m[0] = 0x10;
    memcpy(m + 1, com, 96);
    put_le(m + 97, (uint64_t)m_, 8);
    put_le(m + 105, (uint64_t)k, 8);
    put_le(m + 113, (uint64_t)n, 8);
    put_le(m + 121, proof_id, 8);
    imm_sha::sha256_short(m, 129, s0, 1);
}

uint64_t fs_point_host(const uint32_t (&s0)[8], uint32_t domain, uint32_t t)
{
    uint8_t m[48];
    uint32_t h[8];
    m[0] = 0x11;
    imm_sha::digest_bytes(s0, m + 1);
    put_le(m + 33, domain, 4);
    put_le(m + 37, t, 4);
    imm_sha::sha256_short(m, 41, h, 1);
    return fs_fe_host(h);
}

// Merkle tree hash (RFC 6962) over 32-byte leaves given as state words; neighbours pair level by level,
// an unpaired last node moves up unchanged.
void merkle_root_host(std::vector<imm_sha::Digest> level, uint32_t (&root)[8])
{
    for (imm_sha::Digest& d : level) {
        uint8_t m[40];
        m[0] = 0x00;
        imm_sha::digest_bytes(d.h, m + 1);
        imm_sha::sha256_short(m, 33, d.h, 1);
    }
    while (level.size() > 1) {
        std::vector<imm_sha::Digest> next;
        for (size_t i = 0; i + 1 < level.size(); i += 2) {
            uint8_t m[72];
            m[0] = 0x01;
            imm_sha::digest_bytes(level[i].h, m + 1);
            imm_sha::digest_bytes(level[i + 1].h, m + 33);
            imm_sha::Digest d;
            imm_sha::sha256_short(m, 65, d.h, 1);
            next.push_back(d);
        }
        if (level.size() % 2) next.push_back(level.back());
        level.swap(next);
    }
    for (int i = 0; i < 8; i++) root[i] = level[0].h[i];
}

int fs_check_shape(int64_t m, int64_t k, int64_t n, int nrounds)
{
    if (m <= 0 || k <= 0 || n <= 0 || m > MAX_EXTENT || n > MAX_EXTENT || k > MAX_K) return IMM_ERR_SHAPE;
    if (nrounds != ceil_log2(k)) return IMM_ERR_SHAPE;
    return IMM_OK;
}

}  // namespace

extern "C" {

int imm_fs_challenges(const imm_fe* transcript_host, int nrounds, const uint8_t* commitments_host,
                      int64_t m, int64_t k, int64_t n, uint64_t proof_id,
                      imm_fe* r_row_host, imm_fe* r_col_host, imm_fe* r_k_host)
{
    if (!commitments_host) return IMM_ERR_ARG;
    int rc = fs_check_shape(m, k, n, nrounds);
    if (rc != IMM_OK) return rc;
    uint32_t s[8];
    fs_statement_host(commitments_host, m, k, n, proof_id, s);
    if (r_row_host)
        for (int t = 0; t < ceil_log2(m); t++) r_row_host[t] = fs_point_host(s, 1, (uint32_t)t);
    if (r_col_host)
        for (int t = 0; t < ceil_log2(n); t++) r_col_host[t] = fs_point_host(s, 2, (uint32_t)t);
    if (r_k_host) {
        if (!transcript_host) return IMM_ERR_ARG;
        for (int i = 0; i < 3 * nrounds + 1; i++)
            if (transcript_host[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
        fs_absorb_host(s, 0x12, transcript_host, 1);
        for (int j = 0; j < nrounds; j++) {
            const uint64_t hashed[2] = {transcript_host[1 + 3 * j], transcript_host[3 + 3 * j]};     // g_j(0), g_j(2)
            fs_absorb_host(s, 0x13, hashed, 2);
            r_k_host[j] = fs_fe_host(s);
        }
    }
    return IMM_OK;
}

int imm_fs_batched_challenges(const imm_fe* transcript_host, int nrounds, const imm_matmul_desc* descs_host,
                              int nproofs, const uint8_t* commitments_host, uint64_t batch_id,
                              imm_fe* rho_host, imm_fe* r_k_host)
{
    if (!descs_host || !commitments_host || nproofs <= 0 || nproofs > FS_BATCH_MAX || nrounds < 0 ||
        nrounds > MAX_K_VARS)
        return IMM_ERR_ARG;
    int b = 0;
    std::vector<imm_sha::Digest> stmts(nproofs);
    for (int i = 0; i < nproofs; i++) {
        const imm_matmul_desc& d = descs_host[i];
        int rc = fs_check_shape(d.m, d.k, d.n, ceil_log2(d.k));
        if (rc != IMM_OK) return rc;
        if (ceil_log2(d.k) > b) b = ceil_log2(d.k);
        fs_statement_host(commitments_host + (size_t)i * 96, d.m, d.k, d.n, d.proof_id, stmts[i].h);
    }
    if (nrounds != b) return IMM_ERR_SHAPE;
    uint32_t T[8];
    merkle_root_host(stmts, T);
    {
        uint8_t m[48];
        m[0] = 0x14;
        imm_sha::digest_bytes(T, m + 1);
        put_le(m + 33, batch_id, 8);
        put_le(m + 41, (uint64_t)nproofs, 4);
        imm_sha::sha256_short(m, 45, T, 1);
    }
    if (rho_host)
        for (int p = 0; p < nproofs; p++) {
            uint8_t m[40];
            uint32_t h[8];
            m[0] = 0x15;
            imm_sha::digest_bytes(T, m + 1);
            put_le(m + 33, (uint64_t)p, 4);
            imm_sha::sha256_short(m, 37, h, 1);
            rho_host[p] = fs_fe_host(h);
        }
    if (r_k_host) {
        if (!transcript_host) return IMM_ERR_ARG;
        for (int i = 0; i < 3 * nrounds + 1; i++)
            if (transcript_host[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
        fs_absorb_host(T, 0x12, transcript_host, 1);
        for (int j = 0; j < nrounds; j++) {
            const uint64_t hashed[2] = {transcript_host[1 + 3 * j], transcript_host[3 + 3 * j]};
            fs_absorb_host(T, 0x13, hashed, 2);
            r_k_host[j] = fs_fe_host(T);
        }
    }
    return IMM_OK;
}

int imm_sumcheck_verify_fs_batched(const imm_fe* transcript_host, int nrounds, const imm_matmul_desc* descs_host,
                                   int nproofs, const uint8_t* commitments_host, uint64_t batch_id,
                                   const imm_fe* expect_host, int* fail_at)
{
    if (!transcript_host || !fail_at) return IMM_ERR_ARG;
    std::vector<uint64_t> rho((size_t)(nproofs > 0 ? nproofs : 1));
    uint64_t r_k[64];
    int rc = imm_fs_batched_challenges(transcript_host, nrounds, descs_host, nproofs, commitments_host, batch_id,
                                       rho.data(), r_k);
    if (rc != IMM_OK) return rc;
    const imm_fe* t = transcript_host;
    const int64_t len = 1 + 3 * (int64_t)nrounds + 3 * (int64_t)nproofs;
    for (int64_t i = 0; i < len; i++)
        if (t[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
    if (expect_host)
        for (int64_t i = 0; i < 3 * (int64_t)nproofs; i++)
            if (expect_host[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
    const imm_fe* tail = t + 1 + 3 * nrounds;
    uint64_t combo = 0, fin = 0;
    for (int p = 0; p < nproofs; p++) {
        combo = gl::add(combo, gl::mul(rho[p], tail[3 * (int64_t)p]));
        fin = gl::add(fin, gl::mul(rho[p], gl::mul(tail[3 * (int64_t)p + 1], tail[3 * (int64_t)p + 2])));
    }
    uint64_t claim = t[0];
    if (claim != combo) { *fail_at = nrounds + 1; return IMM_REJECT; }
    const uint64_t inv2 = 0x7FFFFFFF80000001ULL;
    for (int j = 0; j < nrounds; j++) {
        const uint64_t g0 = t[1 + 3 * j], g1 = t[2 + 3 * j], g2 = t[3 + 3 * j];
        if (gl::add(g0, g1) != claim) { *fail_at = j; return IMM_REJECT; }
        const uint64_t r = r_k[j];
        const uint64_t d1 = gl::sub(g1, g0);
        const uint64_t d2 = gl::sub(gl::sub(g2, g1), d1);
        const uint64_t c2 = gl::mul(gl::mul(r, gl::sub(r, 1)), inv2);
        claim = gl::add(g0, gl::add(gl::mul(r, d1), gl::mul(c2, d2)));
    }
    if (fin != claim) { *fail_at = nrounds; return IMM_REJECT; }
    if (expect_host)
        for (int64_t i = 0; i < 3 * (int64_t)nproofs; i++)
            if (expect_host[i] != tail[i]) { *fail_at = nrounds + 2 + (int)i; return IMM_REJECT; }
    *fail_at = -1;
    return IMM_OK;
}

int imm_sumcheck_verify_fs(const imm_fe* transcript_host, int nrounds, const uint8_t* commitments_host,
                           int64_t m, int64_t k, int64_t n, uint64_t proof_id, const imm_fe* expect_c0,
                           const imm_fe* expect_a_fin, const imm_fe* expect_b_fin, int* fail_at)
{
    if (!transcript_host || !commitments_host || !fail_at) return IMM_ERR_ARG;
    int rc = fs_check_shape(m, k, n, nrounds);
    if (rc != IMM_OK) return rc;
    const imm_fe* t = transcript_host;
    for (int i = 0; i < 3 * nrounds + 3; i++)
        if (t[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
    if ((expect_c0 && *expect_c0 >= IMM_P) || (expect_a_fin && *expect_a_fin >= IMM_P) ||
        (expect_b_fin && *expect_b_fin >= IMM_P))
        return IMM_ERR_NONCANONICAL;
    uint64_t r_k[64];
    rc = imm_fs_challenges(t, nrounds, commitments_host, m, k, n, proof_id, nullptr, nullptr, r_k);
    if (rc != IMM_OK) return rc;
    const uint64_t inv2 = 0x7FFFFFFF80000001ULL;
    uint64_t claim = t[0];
    for (int j = 0; j < nrounds; j++) {
        const uint64_t g0 = t[1 + 3 * j], g1 = t[2 + 3 * j], g2 = t[3 + 3 * j];
        if (gl::add(g0, g1) != claim) { *fail_at = j; return IMM_REJECT; }
        const uint64_t r = r_k[j];
        const uint64_t d1 = gl::sub(g1, g0);
        const uint64_t d2 = gl::sub(gl::sub(g2, g1), d1);
        const uint64_t c2 = gl::mul(gl::mul(r, gl::sub(r, 1)), inv2);
        claim = gl::add(g0, gl::add(gl::mul(r, d1), gl::mul(c2, d2)));
    }
    const uint64_t a_fin = t[3 * nrounds + 1], b_fin = t[3 * nrounds + 2];
    if (gl::mul(a_fin, b_fin) != claim) { *fail_at = nrounds; return IMM_REJECT; }
    if (expect_c0 && *expect_c0 != t[0]) { *fail_at = nrounds + 1; return IMM_REJECT; }
    if (expect_a_fin && *expect_a_fin != a_fin) { *fail_at = nrounds + 2; return IMM_REJECT; }
    if (expect_b_fin && *expect_b_fin != b_fin) { *fail_at = nrounds + 3; return IMM_REJECT; }
    *fail_at = -1;
    return IMM_OK;
}

}  // extern "C"

// ------------------------------------------------------------------ host-buffer variant ---

namespace {

struct ArenaPlan {
    int status = IMM_OK;
    struct M { size_t a, b, c; int64_t lda, ldb, ldc; };
    std::vector<M> mats;
    size_t off_tr = 0, off_status = 0, off_ws = 0, ws_bytes = 0, total = 0;
};

int64_t pad16(int64_t cols, int elem) { int per = 16 / elem; return (cols + per - 1) / per * per; }

ArenaPlan make_arena(const imm_matmul_desc* descs, int nproofs, int64_t stride)
{
    ArenaPlan ap;
    Plan p = make_plan(descs, nproofs);
    if (p.status != IMM_OK) { ap.status = p.status; return ap; }
    size_t off = 0;
    ap.mats.resize(nproofs);
    for (int i = 0; i < nproofs; i++) {
        const imm_matmul_desc& d = descs[i];
        ArenaPlan::M& m = ap.mats[i];
        m.lda = pad16(d.k, 1); m.ldb = pad16(d.n, 1); m.ldc = pad16(d.n, 4);
        m.a = off; off = align_up(off + (size_t)d.m * m.lda);
        m.b = off; off = align_up(off + (size_t)d.k * m.ldb);
        m.c = off; off = align_up(off + (size_t)d.m * m.ldc * 4);
    }
    ap.off_tr = off;     off = align_up(off + (size_t)nproofs * (size_t)stride * sizeof(imm_fe));
    ap.off_status = off; off = align_up(off + (size_t)nproofs * sizeof(int32_t));
    ap.off_ws = off;
    ap.ws_bytes = p.total_bytes;
    ap.total = off + p.total_bytes;
    return ap;
}

int64_t max_transcript_len(const imm_matmul_desc* descs, int nproofs)
{
    int64_t len = 3;
    for (int i = 0; i < nproofs; i++) {
        int64_t l = 3 * ceil_log2(descs[i].k) + 3;
        if (l > len) len = l;
    }
    return len;
}

cudaError_t copy_in(void* dst, int64_t dld, const void* src, int64_t sld, int64_t rows, int64_t cols,
                    int elem, cudaStream_t st)
{
    if (dld == sld)
        return cudaMemcpyAsync(dst, src, (size_t)((rows - 1) * sld + cols) * elem, cudaMemcpyHostToDevice, st);
    return cudaMemcpy2DAsync(dst, (size_t)dld * elem, src, (size_t)sld * elem, (size_t)cols * elem,
                             (size_t)rows, cudaMemcpyHostToDevice, st);
}

}  // namespace

extern "C" {

size_t imm_sumcheck_matmul_host_arena(const imm_matmul_desc* descs_host, int nproofs)
{
    if (!descs_host || nproofs <= 0) return 0;
    for (int i = 0; i < nproofs; i++)
        if (check_desc(descs_host[i]) != IMM_OK) return 0;
    ArenaPlan ap = make_arena(descs_host, nproofs, max_transcript_len(descs_host, nproofs));
    return ap.status == IMM_OK ? ap.total : 0;
}

int imm_sumcheck_matmul_prove_host(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed,
                                   imm_fe* transcripts_host, int64_t stride, int32_t* status_host,
                                   void* d_arena, size_t arena_bytes, void* stream)
{
    if (!descs_host || nproofs <= 0 || !transcripts_host || !status_host || !d_arena) return IMM_ERR_ARG;
    for (int i = 0; i < nproofs; i++) {
        int rc = check_desc(descs_host[i]);
        if (rc != IMM_OK) return rc;
    }
    int rc = check_stride(descs_host, nproofs, stride);
    if (rc != IMM_OK) return rc;
    if ((uintptr_t)d_arena % ALIGN != 0) return IMM_ERR_ALIGN;
    // the arena is sized for the tightest stride; a wider one only grows the transcript block
    ArenaPlan ap = make_arena(descs_host, nproofs, stride);
    if (ap.status != IMM_OK) return ap.status;
    if (arena_bytes < ap.total) return IMM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)d_arena;

    std::vector<imm_matmul_desc> dev(descs_host, descs_host + nproofs);
    for (int i = 0; i < nproofs; i++) {
        const imm_matmul_desc& d = descs_host[i];
        const ArenaPlan::M& m = ap.mats[i];
        CU(copy_in(base + m.a, m.lda, d.A, d.lda, d.m, d.k, 1, st));
        CU(copy_in(base + m.b, m.ldb, d.B, d.ldb, d.k, d.n, 1, st));
        CU(copy_in(base + m.c, m.ldc, d.C, d.ldc, d.m, d.n, 4, st));
        dev[i].A = (const int8_t*)(base + m.a); dev[i].lda = m.lda;
        dev[i].B = (const int8_t*)(base + m.b); dev[i].ldb = m.ldb;
        dev[i].C = (const int32_t*)(base + m.c); dev[i].ldc = m.ldc;
    }
    imm_fe* d_tr = (imm_fe*)(base + ap.off_tr);
    int32_t* d_status = (int32_t*)(base + ap.off_status);
    rc = imm_sumcheck_matmul_prove(dev.data(), nproofs, seed, d_tr, stride, d_status,
                                   base + ap.off_ws, ap.ws_bytes, stream);
    if (rc != IMM_OK) return rc;
    CU(cudaMemcpyAsync(transcripts_host, d_tr, (size_t)nproofs * (size_t)stride * sizeof(imm_fe),
                       cudaMemcpyDeviceToHost, st));
    CU(cudaMemcpyAsync(status_host, d_status, (size_t)nproofs * sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return IMM_OK;
}

// ------------------------------------------------------------------ verifier (host) -------

int imm_sumcheck_verify(const imm_fe* transcript_host, int nrounds, uint64_t seed,
                        uint64_t proof_id, const imm_fe* expect_c0, const imm_fe* expect_a_fin,
                        const imm_fe* expect_b_fin, int* fail_at)
{
    if (!transcript_host || !fail_at || nrounds < 0 || nrounds > 64) return IMM_ERR_ARG;
    const imm_fe* t = transcript_host;
    for (int i = 0; i < 3 * nrounds + 3; i++)
        if (t[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
    if ((expect_c0 && *expect_c0 >= IMM_P) || (expect_a_fin && *expect_a_fin >= IMM_P) ||
        (expect_b_fin && *expect_b_fin >= IMM_P))
        return IMM_ERR_NONCANONICAL;
    const uint64_t inv2 = 0x7FFFFFFF80000001ULL;
    uint64_t claim = t[0];
    for (int j = 0; j < nrounds; j++) {
        const uint64_t g0 = t[1 + 3 * j], g1 = t[2 + 3 * j], g2 = t[3 + 3 * j];
        if (gl::add(g0, g1) != claim) { *fail_at = j; return IMM_REJECT; }
        // Newton form on the nodes 0,1,2: g(r) = g0 + r*d1 + r(r-1)/2 * d2
        const uint64_t r = gl::challenge(seed, proof_id, 3, (uint32_t)j);
        const uint64_t d1 = gl::sub(g1, g0);
        const uint64_t d2 = gl::sub(gl::sub(g2, g1), d1);
        const uint64_t c2 = gl::mul(gl::mul(r, gl::sub(r, 1)), inv2);
        claim = gl::add(g0, gl::add(gl::mul(r, d1), gl::mul(c2, d2)));
    }
    const uint64_t a_fin = t[3 * nrounds + 1], b_fin = t[3 * nrounds + 2];
    if (gl::mul(a_fin, b_fin) != claim) { *fail_at = nrounds; return IMM_REJECT; }
    if (expect_c0 && *expect_c0 != t[0]) { *fail_at = nrounds + 1; return IMM_REJECT; }
    if (expect_a_fin && *expect_a_fin != a_fin) { *fail_at = nrounds + 2; return IMM_REJECT; }
    if (expect_b_fin && *expect_b_fin != b_fin) { *fail_at = nrounds + 3; return IMM_REJECT; }
    *fail_at = -1;
    return IMM_OK;
}

int imm_sumcheck_verify_batched(const imm_fe* transcript_host, int nrounds, int nproofs, uint64_t seed,
                                uint64_t batch_id, const imm_fe* expect_host, int* fail_at)
{
    if (!transcript_host || !fail_at || nrounds < 0 || nrounds > 64 || nproofs <= 0 ||
        nproofs > IMM_BATCH_MAX_PROOFS)
        return IMM_ERR_ARG;
    const imm_fe* t = transcript_host;
    const int64_t len = 1 + 3 * (int64_t)nrounds + 3 * (int64_t)nproofs;
    for (int64_t i = 0; i < len; i++)
        if (t[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
    if (expect_host)
        for (int64_t i = 0; i < 3 * (int64_t)nproofs; i++)
            if (expect_host[i] >= IMM_P) return IMM_ERR_NONCANONICAL;
    const imm_fe* tail = t + 1 + 3 * nrounds;
    uint64_t combo = 0, fin = 0;
    for (int p = 0; p < nproofs; p++) {
        const uint64_t rho = gl::challenge(seed, batch_id, 4, (uint32_t)p);
        combo = gl::add(combo, gl::mul(rho, tail[3 * (int64_t)p]));
        fin = gl::add(fin, gl::mul(rho, gl::mul(tail[3 * (int64_t)p + 1], tail[3 * (int64_t)p + 2])));
    }
    uint64_t claim = t[0];
    if (claim != combo) { *fail_at = nrounds + 1; return IMM_REJECT; }
    const uint64_t inv2 = 0x7FFFFFFF80000001ULL;
    for (int j = 0; j < nrounds; j++) {
        const uint64_t g0 = t[1 + 3 * j], g1 = t[2 + 3 * j], g2 = t[3 + 3 * j];
        if (gl::add(g0, g1) != claim) { *fail_at = j; return IMM_REJECT; }
        const uint64_t r = gl::challenge(seed, batch_id, 3, (uint32_t)j);
        const uint64_t d1 = gl::sub(g1, g0);
        const uint64_t d2 = gl::sub(gl::sub(g2, g1), d1);
        const uint64_t c2 = gl::mul(gl::mul(r, gl::sub(r, 1)), inv2);
        claim = gl::add(g0, gl::add(gl::mul(r, d1), gl::mul(c2, d2)));
    }
    if (fin != claim) { *fail_at = nrounds; return IMM_REJECT; }
    if (expect_host)
        for (int64_t i = 0; i < 3 * (int64_t)nproofs; i++)
            if (expect_host[i] != tail[i]) {
                *fail_at = nrounds + 2 + (int)i;
                return IMM_REJECT;
            }
    *fail_at = -1;
    return IMM_OK;
}

}  // extern "C"
