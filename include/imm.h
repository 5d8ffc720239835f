/*
 * imm.h -- C ABI of the B200 (sm_100a) prover for sumcheck proofs of int8 matrix products
 * over the Goldilocks field p = 2^64 - 2^32 + 1, and of what the same audit needs around it.
 * Sections, in this order: field and eq-table helpers; multilinear evaluations; the interactive
 * proof (prover, phase timing, host-buffer variant, host verifier); the batched proof; hash
 * commitments; the verifier's pass over the opened matrices; the element-wise links between
 * products; the non-interactive (Fiat-Shamir) proof, per product and per batch; the logit
 * distance statistics.
 *
 * Background.  The audited-inference protocol this library serves has the server prove, for an
 * audited request, that the "continuous transformations" of the reference model -- its
 * attention and MLP matrix products -- were computed as claimed (paper Section 5.2, item 2;
 * Algorithm 3, the F_theta* step), through a verifiable-computation pair (Prove, Vrfy)
 * (Section 2.2).  The paper leaves the proof system open.  This library instantiates it for one
 * claimed product C = A*B of int8 matrices (C int32) with the classic sumcheck over
 *     sum_y A~(r_row, y) * B~(y, r_col) = C~(r_row, r_col),
 * where M~ is the multilinear extension of M lifted into the field.
 *
 * Conventions
 *   - imm_fe is a canonical field element: a uint64 in [0, p).  Inputs must be canonical;
 *     outputs are.
 *   - lift(v) of a signed integer v is v mod p.
 *   - An index of n bits has variables z_0..z_{n-1}, z_0 the MOST significant bit;
 *     eq(r, i) = prod_t (bit_t(i) ? r_t : 1 - r_t).
 *   - A dimension d is zero-padded (implicitly) at the high end to 2^ceil(log2 d).
 *   - Challenges are public coins of an interactive verifier, drawn from a counter-based
 *     generator (SplitMix64 mixer) keyed by (seed, proof_id); they do not depend on the
 *     prover's messages.  domain 1 = r_row, 2 = r_col, 3 = sumcheck rounds, 4 = the
 *     coefficients of a batched proof (keyed by the batch's id).  The non-interactive proofs
 *     hash their challenges from the commitments and the transcript instead (their section).
 *   - Transcript of one proof: [c0, g_0(0), g_0(1), g_0(2), ..., g_{b-1}(0), g_{b-1}(1),
 *     g_{b-1}(2), a_fin, b_fin], b = ceil(log2 k), 3b+3 words.
 *
 * General rules
 *   - Every call returns an int status (IMM_OK or a negative IMM_ERR_*; imm_sumcheck_verify may
 *     also return IMM_REJECT).  Nothing throws or aborts across this boundary.
 *   - The caller owns every buffer.  The library allocates no device memory: scratch comes from
 *     a caller-provided device workspace whose size a query call returns.  Workspace and output
 *     pointers must be 16-byte aligned.  What the library does keep, per process: the event
 *     ring of imm_profile_enable (while enabled) and the 64 KiB device array of
 *     imm_mle_eval_point_noalloc.  It creates no streams and launches only on the caller's.
 *   - One environment variable is read, on every prove / evaluation call: IMM_CONTRACT=alu selects
 *     the integer-pipe contraction kernels instead of the tensor-core ones (same results; meant for
 *     A/B measurements).  Anything else, or unset, is the default.
 *   - Pointers named d_* are DEVICE pointers, *_host are HOST pointers.
 *   - Device calls enqueue work on the given CUDA stream (a cudaStream_t passed as void*; NULL =
 *     the legacy default stream) and return without synchronising, unless stated otherwise.
 *     Host descriptor arrays are read before the call returns.
 *   - Matrices are row-major with a leading dimension ld in ELEMENTS (ld >= cols).  Rows that
 *     are 16-byte aligned (base pointer and ld*sizeof(element) multiples of 16) take the
 *     vectorised kernels; anything else takes an element-wise path with the same results.
 *   - Limits: 1 <= rows, cols <= 2^20 for the matrix calls; for proofs 1 <= m, n <= 2^20 and
 *     1 <= k <= 2^17.  A zero extent is IMM_ERR_SHAPE.
 *   - There is no CPU fallback: without a CUDA device every device call returns IMM_ERR_CUDA.
 */
#ifndef IMM_H_
#define IMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef uint64_t imm_fe;

#define IMM_P 0xFFFFFFFF00000001ULL

enum {
    IMM_OK = 0,
    IMM_REJECT = 1,              /* imm_sumcheck_verify only: the proof is rejected        */
    IMM_ERR_ARG = -1,            /* null pointer, bad enum value, negative count           */
    IMM_ERR_SHAPE = -2,          /* zero or too large extent, ld < cols                    */
    IMM_ERR_ALIGN = -3,          /* workspace / output pointer not 16-byte aligned         */
    IMM_ERR_WORKSPACE = -4,      /* workspace smaller than the query call asks for         */
    IMM_ERR_NONCANONICAL = -5,   /* a field element >= p on input                          */
    IMM_ERR_CUDA = -6,           /* a CUDA runtime call failed (see imm_last_cuda_error)   */
    IMM_ERR_TIMEOUT = -7,        /* reserved: a bounded device-side wait ran out.  No kernel
                                    of this library waits on a flag, so nothing returns it */
    IMM_ERR_LIMIT = -8           /* beyond a fixed capacity stated with the call           */
};
enum { IMM_I8 = 0, IMM_I32 = 1 };
enum { IMM_BIND_ROWS = 0, IMM_BIND_COLS = 1 };
enum { IMM_FIELD_ADD = 0, IMM_FIELD_SUB = 1, IMM_FIELD_MUL = 2 };

/* Library version (major*100 + minor). */
int imm_version(void);

/* Text of the last CUDA runtime error seen by the calling thread's device calls ("" if none).
 * The pointer stays valid until the thread's next failing call. */
const char* imm_last_cuda_error(void);

/* HOST.  Challenge `index` of `domain` (1 = r_row, 2 = r_col, 3 = sumcheck round, 4 = batching coefficient) for
 * (seed, proof_id): canon(mix64(key + G*(ctr+1))) with key = mix64(mix64(seed+G) + G*(proof_id+1)),
 * ctr = domain<<32 | index, G = 0x9E3779B97F4A7C15, canon(x) = x >= p ? x-p : x.  These are the
 * verifier's public coins (Section 2.2's Vrfy side). */
imm_fe imm_challenge(uint64_t seed, uint64_t proof_id, uint32_t domain, uint32_t index);

/* Element-wise field arithmetic on device arrays: d_out[i] = d_x[i] (op) d_y[i], i < count.
 * Exists so the device field arithmetic can be tested in isolation.  Inputs must be canonical
 * (not checked).  count == 0 is a no-op. */
int imm_field_binop(int op, const imm_fe* d_x, const imm_fe* d_y, imm_fe* d_out, int64_t count,
                    void* stream);

/* eq table (the Lagrange basis of the Boolean cube at r; multilinear-extension definition
 * used by every step of the proof).  d_out[i] = eq(r, i) for i < 2^nvars.
 *   r_host : HOST array of nvars canonical field elements (read before return)
 *   nvars  : 0..20
 *   d_out  : DEVICE array of 2^nvars elements, 16-byte aligned
 * Errors: IMM_ERR_ARG, IMM_ERR_SHAPE (nvars out of range), IMM_ERR_NONCANONICAL, IMM_ERR_ALIGN. */
int imm_eq_table(const imm_fe* r_host, int nvars, imm_fe* d_out, void* stream);

/* Workspace bytes needed by imm_mle_partial_eval / imm_mle_eval_point for this matrix. */
size_t imm_mle_workspace(int dtype, int64_t rows, int64_t cols, int bind);

/* Partial evaluation of a matrix's multilinear extension: binds one index with an eq table.
 *   IMM_BIND_ROWS: d_out[y] = sum_{i<rows} d_eq[i] * lift(M[i,y]),  y < cols  (A~(r_row, .))
 *   IMM_BIND_COLS: d_out[i] = sum_{j<cols} lift(M[i,j]) * d_eq[j],  i < rows  (B~(., r_col))
 *   d_mat   : DEVICE matrix, dtype IMM_I8 (int8) or IMM_I32 (int32), rows x cols, leading dim ld
 *   d_eq    : DEVICE eq table with at least rows (BIND_ROWS) / cols (BIND_COLS) entries; entries
 *             past the real extent are ignored, which is the implicit zero padding
 *   d_out   : DEVICE array of cols (BIND_ROWS) / rows (BIND_COLS) elements
 *   d_ws    : DEVICE workspace of at least imm_mle_workspace(dtype, rows, cols, bind) bytes
 * Errors: IMM_ERR_ARG, IMM_ERR_SHAPE, IMM_ERR_ALIGN, IMM_ERR_WORKSPACE, IMM_ERR_CUDA. */
int imm_mle_partial_eval(const void* d_mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
                         int bind, const imm_fe* d_eq, imm_fe* d_out,
                         void* d_ws, size_t ws_bytes, void* stream);

/* Full evaluation at a point given as two eq tables (the verifier's claim C~(r_row, r_col), and
 * the checks of a_fin, b_fin):  d_out[0] = sum_{i,j} d_eq_row[i] * lift(M[i,j]) * d_eq_col[j].
 * Workspace: imm_mle_workspace(dtype, rows, cols, IMM_BIND_ROWS) bytes.  Same errors. */
int imm_mle_eval_point(const void* d_mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
                       const imm_fe* d_eq_row, const imm_fe* d_eq_col, imm_fe* d_out,
                       void* d_ws, size_t ws_bytes, void* stream);

/* Point evaluation for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a deployment convenience of this library.)
 *
 * Same result as imm_mle_eval_point, but without a workspace argument: the per-tile partial sums
 * live in a fixed 64 KiB array that is part of the library's device image, so every GPU that
 * loads the library holds that array until the process exits.  It is meant for code that runs
 * inside a serving engine's step -- an audit hook called between decode steps, say -- where all
 * device memory already belongs to the engine's pool, so a cudaMalloc would fail under the
 * memory cap or stall every stream with its implicit device-wide synchronisation, and where no
 * spare buffer can be threaded through to the call site.  The call itself performs no
 * cudaMalloc / cudaFree and uses no allocating library routine; it enqueues two kernels on
 * `stream` and returns.
 *
 * Capacity: the matrix is cut into tiles of up to 1024 rows x 512 int32 (2048 int8) columns and at
 * most IMM_NOALLOC_MAX_TILES tiles fit the array (about 16 GiB of matrix); anything larger returns
 * IMM_ERR_LIMIT before any device work.  Other errors as imm_mle_eval_point (no workspace ones).
 *
 * The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 * that device current); make that first call outside any stream capture.  All calls on one
 * device share the array: it keeps the previous call's partial sums, which is harmless because
 * every slot a call reads is first overwritten by that call (nothing needs to start at zero), but
 * two calls whose kernels overlap on the GPU (different streams, or different host threads
 * without ordering) race on it and return garbage.  Order such calls on one stream. */
#define IMM_NOALLOC_MAX_TILES 8192
int imm_mle_eval_point_noalloc(const void* d_mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
                               const imm_fe* d_eq_row, const imm_fe* d_eq_col, imm_fe* d_out,
                               void* stream);

/* One claimed product C = A*B.  A: m x k int8, B: k x n int8, C: m x n int32 -- the CLAIMED
 * matrix, used as given (the prover never recomputes A*B).  DEVICE pointers for
 * imm_sumcheck_matmul_prove, HOST pointers for imm_sumcheck_matmul_prove_host. */
typedef struct {
    const int8_t* A;
    const int8_t* B;
    const int32_t* C;
    int64_t m, k, n;
    int64_t lda, ldb, ldc;      /* leading dimensions in elements */
    uint64_t proof_id;
} imm_matmul_desc;

/* Workspace bytes imm_sumcheck_matmul_prove needs for this batch (0 on invalid input). */
size_t imm_sumcheck_matmul_workspace(const imm_matmul_desc* descs_host, int nproofs);

/* Prover (Prove of Section 2.2, for the matrix products of Algorithm 3's F_theta* step).  For
 * every proof of the batch: derives r_row, r_col, r_k from (seed, proof_id); builds both eq
 * tables; evaluates avec = A~(r_row, .), bvec = B~(., r_col) and c0 = C~(r_row, r_col); runs
 * the ceil(log2 k) sumcheck rounds (each round's g(0), g(1), g(2), then the fold of both
 * tables with that round's challenge); writes the transcript.
 *   descs_host    : HOST array of nproofs descriptors with DEVICE matrix pointers
 *   d_transcripts : DEVICE array, nproofs rows of `stride` words, stride >= 3*ceil(log2(max k))+3;
 *                   row p holds proof p's transcript, words past its length are set to zero
 *   d_status      : DEVICE array of nproofs int32, set to IMM_OK per proof (reserved for
 *                   device-detected conditions)
 *   d_ws          : DEVICE workspace, >= imm_sumcheck_matmul_workspace(...) bytes
 * The whole batch is one small host-to-device copy (the job lists) and a fixed sequence of kernel
 * launches on `stream`, ordered after the work already there; results are valid once the stream has
 * been synchronised.  A large batch takes five launches: eq tables and weight limb tables, the
 * claim, the row binding, the column binding, the rounds.  A batch under 4 GiB of matrices, or
 * under 16 GiB whose proofs average 32 MiB or more, is held back by launch latency and the gaps
 * between kernels more than by bandwidth and takes three, chained by programmatic dependent
 * launch: one contraction launch for all three matrix kinds, whose tiles build their own slice of
 * the eq tables from the challenges (no table reaches memory); a reduction of the partial vectors
 * into the round tables; the rounds.  Same transcripts either way.
 * Errors: IMM_ERR_ARG, IMM_ERR_SHAPE, IMM_ERR_ALIGN, IMM_ERR_WORKSPACE, IMM_ERR_CUDA. */
int imm_sumcheck_matmul_prove(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed,
                              imm_fe* d_transcripts, int64_t stride, int32_t* d_status,
                              void* d_ws, size_t ws_bytes, void* stream);

/* Kernel launches imm_sumcheck_matmul_prove enqueues for this batch: 5, or 3 for a batch that takes
 * the fused contraction launch (0 on invalid input). */
int imm_sumcheck_matmul_launches(const imm_matmul_desc* descs_host, int nproofs);

/* Phase timing of imm_sumcheck_matmul_prove, for measurement.  While enabled, every prove call
 * records a pair of CUDA events around each of its launches, into the next of `capacity` event sets
 * (a ring), without synchronising.  Phases:
 *   [0] eq tables, [1] claim C~ (int32 point contraction), [2] A~ row binding,
 *   [3] B~ column binding, [4] sumcheck rounds.
 * A batch that takes the fused contraction launch (see imm_sumcheck_matmul_prove) reports that launch
 * as phase [1], phases [0], [2], [3] as (almost) zero, and the reduction plus the rounds as [4]; the
 * events between its launches undo their programmatic overlap, so whole steps are best timed with
 * phase timing off.
 * The event ring is per process; profiled calls must not overlap on different host threads.
 * imm_profile_enable(capacity): capacity in 1..4096 creates the ring and resets the call count
 *   (needs a CUDA device); capacity 0 destroys it.
 * imm_profile_calls(): profiled prove calls since the ring was created.
 * imm_profile_read(call, ms_host, count): waits for profiled call number `call` (0-based) to
 *   finish and writes its elapsed milliseconds per phase; count must be IMM_PROFILE_PHASES.
 *   IMM_ERR_ARG if profiling is off or the call is not (or no longer) in the ring. */
#define IMM_PROFILE_PHASES 5
int imm_profile_enable(int capacity);
int64_t imm_profile_calls(void);
int imm_profile_read(int64_t call, float* ms_host, int count);

/* Device arena bytes imm_sumcheck_matmul_prove_host needs: staged copies of all matrices, the
 * transcripts and status words, and the prover workspace (0 on invalid input). */
size_t imm_sumcheck_matmul_host_arena(const imm_matmul_desc* descs_host, int nproofs);

/* End-to-end variant with HOST matrices: copies every A, B, C to the device arena, proves,
 * copies transcripts and status back, and SYNCHRONISES the stream before returning.
 *   descs_host       : HOST descriptors with HOST matrix pointers (pinned memory copies fastest)
 *   transcripts_host : HOST array, nproofs x stride words
 *   status_host      : HOST array of nproofs int32
 *   d_arena          : DEVICE arena of >= imm_sumcheck_matmul_host_arena(...) bytes, 256-byte aligned
 * Same errors as imm_sumcheck_matmul_prove. */
int imm_sumcheck_matmul_prove_host(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed,
                                   imm_fe* transcripts_host, int64_t stride, int32_t* status_host,
                                   void* d_arena, size_t arena_bytes, void* stream);

/* HOST verifier (Vrfy of Section 2.2).  claim <- c0; for each round j require
 * g_j(0) + g_j(1) = claim and set claim <- g_j(r_j) by interpolation on the nodes {0,1,2};
 * finally require claim = a_fin * b_fin.  When an expect_* pointer is non-NULL the
 * corresponding transcript word must also equal the pointed-to value (the verifier's own
 * evaluation of C~, A~ or B~).
 *   transcript_host : HOST array of 3*nrounds+3 canonical words
 *   fail_at         : HOST out.  -1 accepted; j in [0,nrounds) = round j's sum check failed;
 *                     nrounds = final product check failed; nrounds+1 / +2 / +3 = c0 / a_fin /
 *                     b_fin differs from the expected value
 * Returns IMM_OK, IMM_REJECT, IMM_ERR_ARG or IMM_ERR_NONCANONICAL. */
int imm_sumcheck_verify(const imm_fe* transcript_host, int nrounds, uint64_t seed,
                        uint64_t proof_id, const imm_fe* expect_c0, const imm_fe* expect_a_fin,
                        const imm_fe* expect_b_fin, int* fail_at);

/* ---------------------------------------------------------------------------------------------
 * Batched proof: one sumcheck for a random linear combination of product claims
 * ---------------------------------------------------------------------------------------------
 * The products a proof of the reference execution must cover are many (the attention and MLP
 * products of every layer, Section 4.1).  They can share one sumcheck over b = max_p ceil(log2 k_p)
 * variables (a smaller k is zero-padded to 2^b like any other, which changes neither the product
 * nor the claim): with public coins rho_p = imm_challenge(seed, batch_id, 4, p) the prover shows
 *   sum_p rho_p * sum_y A_p~(r_row_p, y) B_p~(y, r_col_p) = sum_p rho_p C_p~(r_row_p, r_col_p),
 * all proofs folding with the same round challenges r_j = imm_challenge(seed, batch_id, 3, j);
 * r_row_p and r_col_p stay each proof's own (domains 1, 2 under its proof_id).  The verifier then
 * reads 1 + 3b + 3P words instead of P * (3b + 3).
 *
 * Batched transcript, imm_sumcheck_batched_transcript_len(b, P) = 1 + 3b + 3P words:
 *   [c0B, g_0(0), g_0(1), g_0(2), ..., g_{b-1}(0..2), (c0_0, a_fin_0, b_fin_0), ..., (c0_{P-1}, ..)]
 *   c0B = sum_p rho_p c0_p;  g_j = sum_p rho_p g_j^(p);  a_fin_p = A_p~(r_row_p, r),
 *   b_fin_p = B_p~(r, r_col_p) at the shared point r = (r_0..r_{b-1}).                          */
#define IMM_BATCH_MAX_PROOFS (1 << 24)

/* Transcript words of a batched proof (0 on invalid arguments). */
int64_t imm_sumcheck_batched_transcript_len(int nrounds, int nproofs);

/* Workspace bytes imm_sumcheck_matmul_prove_batched needs (0 on invalid input). */
size_t imm_sumcheck_matmul_batched_workspace(const imm_matmul_desc* descs_host, int nproofs);

/* Batched prover.  Runs the launch sequence of imm_sumcheck_matmul_prove with the shared round
 * challenges (per-proof transcripts go to the workspace), then one more launch forms the
 * batched transcript.
 *   descs_host   : HOST array of nproofs descriptors with DEVICE matrix pointers
 *   d_transcript : DEVICE array of imm_sumcheck_batched_transcript_len(b, nproofs) words,
 *                  b = ceil(log2 of the largest k)
 *   d_status     : DEVICE array of nproofs int32 (as imm_sumcheck_matmul_prove)
 *   d_ws         : DEVICE workspace, 256-byte aligned, >= imm_sumcheck_matmul_batched_workspace(...)
 * Errors: IMM_ERR_ARG, IMM_ERR_SHAPE, IMM_ERR_ALIGN, IMM_ERR_WORKSPACE, IMM_ERR_LIMIT (more than
 * IMM_BATCH_MAX_PROOFS proofs), IMM_ERR_CUDA. */
int imm_sumcheck_matmul_prove_batched(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed,
                                      uint64_t batch_id, imm_fe* d_transcript, int32_t* d_status,
                                      void* d_ws, size_t ws_bytes, void* stream);

/* HOST verifier of a batched transcript.  Requires c0B = sum_p rho_p c0_p; then, with
 * claim <- c0B, per round g_j(0) + g_j(1) = claim and claim <- g_j(r_j); finally
 * claim = sum_p rho_p a_fin_p b_fin_p.  expect_host, when non-NULL, holds the verifier's own
 * 3*nproofs values (c0_p, a_fin_p, b_fin_p in transcript order) and is compared word for word.
 *   fail_at : HOST out.  -1 accepted; j in [0,nrounds) = round j; nrounds = the final check;
 *             nrounds+1 = c0B is not the combination of the listed c0_p; nrounds+2+t = word t of
 *             the per-proof part differs from expect_host
 * Returns IMM_OK, IMM_REJECT, IMM_ERR_ARG or IMM_ERR_NONCANONICAL. */
int imm_sumcheck_verify_batched(const imm_fe* transcript_host, int nrounds, int nproofs, uint64_t seed,
                                uint64_t batch_id, const imm_fe* expect_host, int* fail_at);

/* ---------------------------------------------------------------------------------------------
 * Hash commitments
 * ---------------------------------------------------------------------------------------------
 * c = Hash(m || r) (Section 2.1, cryptographic commitment): the server's commitment to the model
 * and, under fresh randomness r, to the logits of a response (Algorithm 1); the auditor recomputes
 * both (first check of the auditing algorithm).  The paper names no hash; here
 *   Hash  = SHA-256 (FIPS 180-4) in a tree mode, so that a message of gigabytes hashes in parallel:
 *   root  = Merkle tree hash of RFC 6962, Section 2.1, over the message cut into
 *           IMM_COMMIT_LEAF-byte pieces (the last may be shorter; an empty message is one empty
 *           piece): leaf = SHA-256(0x00 || piece), node = SHA-256(0x01 || left || right), the split
 *           of n pieces at the largest power of two below n;
 *   c     = SHA-256(0x02 || root || le64(nbytes) || r), r = 32 bytes, or none for a commitment
 *           that hides nothing (the model's).
 * Digests are the usual 32-byte big-endian serialisation. */
#define IMM_COMMIT_LEAF 4096
#define IMM_COMMIT_MAX_MESSAGES (1 << 20)
#define IMM_COMMIT_MAX_BYTES (1ull << 40)

typedef struct {
    const void* msg;        /* DEVICE pointer to nbytes contiguous bytes (may be NULL when nbytes = 0) */
    uint64_t nbytes;
    uint8_t r[32];          /* the commitment's randomness (read when r_len = 32) */
    int32_t r_len;          /* 0 or 32 */
    int32_t reserved;       /* set to 0 */
} imm_commit_desc;

/* Workspace bytes imm_commit needs for this batch (0 on invalid input). */
size_t imm_commit_workspace(const imm_commit_desc* descs_host, int n);

/* Kernel launches imm_commit enqueues for this batch (0 on invalid input). */
int imm_commit_launches(const imm_commit_desc* descs_host, int n);

/* Commits to every message of the batch.
 *   descs_host : HOST array of n descriptors (at most IMM_COMMIT_MAX_MESSAGES, each message at
 *                most IMM_COMMIT_MAX_BYTES)
 *   d_digests  : DEVICE array of n x 32 bytes: the commitments c
 *   d_roots    : DEVICE array of n x 32 bytes for the tree roots, or NULL
 *   d_ws       : DEVICE workspace, 256-byte aligned, >= imm_commit_workspace(...) bytes
 * Messages whose pointer is 16-byte aligned are read with 128-bit loads, others byte by byte
 * (slow).  The batch is one leaf launch (one thread per leaf; the 128 to 512 leaves of a block fold
 * to a subtree root on chip), one launch per further factor of 1024 in the largest count of subtree
 * roots, and a final launch; all are enqueued on `stream`, nothing is synchronised or allocated.
 * Errors: IMM_ERR_ARG, IMM_ERR_LIMIT, IMM_ERR_ALIGN, IMM_ERR_WORKSPACE, IMM_ERR_CUDA. */
int imm_commit(const imm_commit_desc* descs_host, int n, uint8_t* d_digests, uint8_t* d_roots,
               void* d_ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * The verifier's pass
 * ---------------------------------------------------------------------------------------------
 * Vrfy of Section 2.2 accepts a transcript only if its c0, a_fin, b_fin are the verifier's OWN
 * evaluations C~(r_row, r_col), A~(r_row, r_k), B~(r_k, r_col) of the opened matrices (the expect_*
 * arguments of the host verifiers).  That is one pass over every matrix, like proving: the three
 * contractions are the prover's, and where the prover runs the rounds the verifier takes the
 * inner products of A~(r_row, .) and B~(., r_col) with E_k = eq(r_k, .). */

/* Workspace bytes imm_sumcheck_expected needs (0 on invalid input).  batched != 0: for the members
 * of a batched proof (every k padded to the largest 2^b). */
size_t imm_sumcheck_expected_workspace(const imm_matmul_desc* descs_host, int nproofs, int batched);

/* The verifier's own (c0, a_fin, b_fin) of every proof of a batch.
 *   descs_host  : HOST descriptors with DEVICE matrix pointers (the opened A, B and claimed C)
 *   seed        : the verifier's coins (interactive and batched proofs; ignored with points_host)
 *   batch_id    : HOST, NULL for proofs proved one by one (r_k under each proof_id, ceil(log2 k)
 *                 rounds); else the id of the batched proof (shared r_k, the batch's round count)
 *   points_host : HOST, NULL to draw r_row, r_col, r_k from the generator; else nproofs x 96 given
 *                 canonical values, per proof r_row at [0, 32), r_col at [32, 64), r_k at [64, 96)
 *                 (a non-interactive proof: imm_fs_challenges)
 *   d_expected  : DEVICE array of nproofs x 3 words: c0, a_fin, b_fin per proof
 *   d_status    : DEVICE array of nproofs int32, set to IMM_OK per proof
 *   d_ws        : DEVICE workspace, 256-byte aligned, >= imm_sumcheck_expected_workspace(...)
 * Launch sequence and errors as imm_sumcheck_matmul_prove (IMM_ERR_NONCANONICAL for a given point
 * not below p). */
int imm_sumcheck_expected(const imm_matmul_desc* descs_host, int nproofs, uint64_t seed, const uint64_t* batch_id,
                          const imm_fe* points_host, imm_fe* d_expected, int32_t* d_status,
                          void* d_ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Links between products
 * ---------------------------------------------------------------------------------------------
 * The reference execution is a chain of attention, MLP and normalisation steps (Section 4.1), and
 * the proof must cover the whole chain (Section 5.2, item 2).  The sumcheck proofs above cover its
 * matrix products one at a time; nothing in them says that the int8 input of one product is the
 * output of the one before.  In an int8-quantised execution the map between the two is the
 * requantisation of the int32 accumulators,
 *     H[i,j] = clamp( floor( (C[i,j] + rnd) / 2^shift ), lo, hi )
 * (round-half-up division by 2^shift when rnd = 2^(shift-1), then saturation; e.g. the FFN hidden
 * activations between the up and the down projection).  A verifier that holds the opened tensors
 * checks such a link by recomputing it: one streaming pass, 4 bytes of C and 1 byte of H per entry. */

/* d_result[0] = number of entries where H differs from the requantised C, d_result[1] = the row-major
 * position i*cols + j of the first such entry (UINT64_MAX if there is none).  The link holds iff
 * d_result[0] == 0.
 *   d_C      : DEVICE int32 matrix, rows x cols, leading dimension ldc (elements)
 *   d_H      : DEVICE int8 matrix, rows x cols, leading dimension ldh
 *   shift    : 0..30;  rnd : 0 <= rnd < 2^shift;  -128 <= lo <= hi <= 127
 *   d_result : DEVICE array of two uint64, 8-byte aligned; overwritten
 * Rows of C that are 32-byte (or 16-byte) aligned with rows of H 16-byte aligned are read with
 * 256-bit (128-bit) loads, anything else element by element.  Two memsets and one kernel are
 * enqueued on `stream`; nothing is allocated or synchronised.  A differing entry is an audit
 * finding, not an error: the call still returns IMM_OK.
 * Errors: IMM_ERR_ARG (null pointer, parameters out of range), IMM_ERR_SHAPE (zero or > 2^20
 * extent, ld < cols), IMM_ERR_ALIGN, IMM_ERR_CUDA. */
int imm_requant_check(const int32_t* d_C, const int8_t* d_H, int64_t rows, int64_t cols, int64_t ldc,
                      int64_t ldh, int shift, int32_t rnd, int32_t lo, int32_t hi, uint64_t* d_result,
                      void* stream);

/* The element-wise step of a gated feed-forward block (the MLP of the decoder models of Section 6.1;
 * one of the parts of the reference execution in Section 4.1): an activation of the gate projection
 * and its product with the up projection give the int8 input of the down projection,
 *     g[i,j] = act[ clamp(floor((G[i,j] + rnd) / 2^shift), -128, 127) + 128 ]
 *     u[i,j] =      clamp(floor((U[i,j] + rnd) / 2^shift), -128, 127)
 *     H[i,j] = clamp( floor( (g[i,j] * u[i,j] + rnd2) / 2^shift2 ), lo, hi )
 * with G, U the int32 outputs of the two products.  The activation is the committed model's own
 * int8 -> int8 table (the paper fixes no integer arithmetic).  d_U == NULL: the activation alone,
 * H = g (shift2, rnd2, lo, hi are then ignored).  Results as for imm_requant_check: d_result[0] the
 * number of entries of H that differ, d_result[1] the position of the first (UINT64_MAX if none).
 *   d_G, d_U : DEVICE int32 matrices, rows x cols, leading dimensions ldg, ldu (elements)
 *   d_H      : DEVICE int8 matrix, rows x cols, leading dimension ldh
 *   act_host : HOST array of 256 int8: act_host[v + 128] answers the value v; copied into the launch
 *   shift    : 0..30, 0 <= rnd < 2^shift;  shift2 : 0..14, 0 <= rnd2 < 2^shift2;  -128 <= lo <= hi <= 127
 * One streaming pass: 4 (+4) bytes of G (and U) and 1 byte of H per entry, each read once; 16-byte
 * aligned rows are read with 128-bit loads, anything else element by element.  Two memsets and one
 * kernel on `stream`; nothing allocated or synchronised; a differing entry is a finding, not an error.
 * Errors: IMM_ERR_ARG, IMM_ERR_SHAPE (zero or > 2^20 extent, ld < cols), IMM_ERR_ALIGN, IMM_ERR_CUDA. */
int imm_gated_link_check(const int32_t* d_G, const int32_t* d_U, const int8_t* d_H, int64_t rows, int64_t cols,
                         int64_t ldg, int64_t ldu, int64_t ldh, const int8_t* act_host, int shift, int32_t rnd,
                         int shift2, int32_t rnd2, int32_t lo, int32_t hi, uint64_t* d_result, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Non-interactive proof (Fiat-Shamir)
 * ---------------------------------------------------------------------------------------------
 * Algorithm 1 has the server attach a proof pi to its response: no verifier is on line to draw
 * coins, so the public coins of the proof above are replaced by hashes of everything sent so far.
 * H = SHA-256; integers are little-endian; a field element is the le64 of its canonical value;
 * fe(d) = the first 8 bytes of a digest as a big-endian integer, minus p if not below p.
 *   s_0      = H(0x10 || com_A || com_B || com_C || le64(m) || le64(k) || le64(n) || le64(proof_id)),
 *              com_X the 32-byte commitments to the three matrices (imm_commit);
 *   r_row[t] = fe(H(0x11 || s_0 || le32(1) || le32(t))),  r_col[t] the same with le32(2);
 *   s_1      = H(0x12 || s_0 || le64(c0));
 *   round j:   s_{j+2} = H(0x13 || s_{j+1} || le64(g_j(0)) || le64(g_j(2))),  r_j = fe(s_{j+2});
 *              g_j(1) is in the transcript but not in the hash: the verifier's check
 *              g_j(0) + g_j(1) = claim pins it, and the message stays one SHA-256 block.
 * The transcript has the layout of the interactive proof (3b+3 words). */

/* Workspace bytes imm_sumcheck_matmul_prove_fs needs (0 on invalid input). */
size_t imm_sumcheck_matmul_fs_workspace(const imm_matmul_desc* descs_host, int nproofs);

/* Non-interactive prover.  As imm_sumcheck_matmul_prove, but every challenge is hashed: one launch
 * hashes the statements and derives r_row, r_col, and the round kernel (one block per proof) hashes
 * each round's three values before it folds with the challenge they give.
 *   d_commitments : DEVICE array, nproofs x 96 bytes: com_A || com_B || com_C of each proof
 *   d_ws          : DEVICE workspace, 256-byte aligned, >= imm_sumcheck_matmul_fs_workspace(...)
 * Other arguments and errors as imm_sumcheck_matmul_prove. */
int imm_sumcheck_matmul_prove_fs(const imm_matmul_desc* descs_host, int nproofs, const uint8_t* d_commitments,
                                 imm_fe* d_transcripts, int64_t stride, int32_t* d_status,
                                 void* d_ws, size_t ws_bytes, void* stream);

/* HOST.  The challenges of a non-interactive proof, as the verifier derives them: r_row
 * (ceil(log2 m) values), r_col (ceil(log2 n)) from the statement, r_k (nrounds) from the statement
 * and the transcript's first 3*nrounds+1 words.  Any output pointer may be NULL (transcript_host
 * may be NULL when r_k_host is).  nrounds must equal ceil(log2 k).
 * Returns IMM_OK, IMM_ERR_ARG, IMM_ERR_SHAPE or IMM_ERR_NONCANONICAL. */
int imm_fs_challenges(const imm_fe* transcript_host, int nrounds, const uint8_t* commitments_host,
                      int64_t m, int64_t k, int64_t n, uint64_t proof_id,
                      imm_fe* r_row_host, imm_fe* r_col_host, imm_fe* r_k_host);

/* Batched non-interactive proof: ONE proof for all products of a batch, every coin hashed.  The
 * batched proof above with
 *   root  = Merkle tree hash (RFC 6962: leaf = H(0x00 || d), node = H(0x01 || l || r)) over the member
 *           statements s_0^(0), ..., s_0^(P-1) as 32-byte leaves,
 *   T     = H(0x14 || root || le64(batch_id) || le32(P)),   rho_p = fe(H(0x15 || T || le32(p))),
 *   s_1   = H(0x12 || T || le64(c0B)),  rounds as for the single proof on the combined values;
 * r_row, r_col of a member come from its own statement.  The member values c0_p are not hashed: with
 * binding commitments they are functions of the statements, and the verifier compares them with
 * its own.  At most IMM_FS_BATCH_MAX members.  Transcript layout: that of the batched proof. */
#define IMM_FS_BATCH_MAX 1024

size_t imm_sumcheck_matmul_fs_batched_workspace(const imm_matmul_desc* descs_host, int nproofs);

/* Prover.  Arguments as imm_sumcheck_matmul_prove_fs; d_transcript holds
 * imm_sumcheck_batched_transcript_len(b, nproofs) words, b = ceil(log2 of the largest k).  After the
 * contractions the rounds are a chain of 3 + 2b small launches (every round needs the sum over all
 * members before its challenge exists).  IMM_ERR_LIMIT for more than IMM_FS_BATCH_MAX members. */
int imm_sumcheck_matmul_prove_fs_batched(const imm_matmul_desc* descs_host, int nproofs, const uint8_t* d_commitments,
                                         uint64_t batch_id, imm_fe* d_transcript, int32_t* d_status,
                                         void* d_ws, size_t ws_bytes, void* stream);

/* HOST.  The coins of a batched non-interactive proof: rho (nproofs values) and r_k (nrounds values,
 * from the transcript's first 3*nrounds+1 words).  descs_host gives every member's m, k, n and
 * proof_id (matrix pointers are not read); commitments_host holds nproofs x 96 bytes.  Either
 * output may be NULL.  The members' r_row, r_col: imm_fs_challenges with a NULL transcript. */
int imm_fs_batched_challenges(const imm_fe* transcript_host, int nrounds, const imm_matmul_desc* descs_host,
                              int nproofs, const uint8_t* commitments_host, uint64_t batch_id,
                              imm_fe* rho_host, imm_fe* r_k_host);

/* HOST verifier of a batched non-interactive proof: the checks and fail_at of
 * imm_sumcheck_verify_batched with the hashed coins. */
int imm_sumcheck_verify_fs_batched(const imm_fe* transcript_host, int nrounds, const imm_matmul_desc* descs_host,
                                   int nproofs, const uint8_t* commitments_host, uint64_t batch_id,
                                   const imm_fe* expect_host, int* fail_at);

/* HOST verifier of a non-interactive proof: the checks of imm_sumcheck_verify with the hashed round
 * challenges; fail_at has the same meaning.  commitments_host: the 96 bytes of the statement.
 * Returns IMM_OK, IMM_REJECT, IMM_ERR_ARG, IMM_ERR_SHAPE or IMM_ERR_NONCANONICAL. */
int imm_sumcheck_verify_fs(const imm_fe* transcript_host, int nrounds, const uint8_t* commitments_host,
                           int64_t m, int64_t k, int64_t n, uint64_t proof_id, const imm_fe* expect_c0,
                           const imm_fe* expect_a_fin, const imm_fe* expect_b_fin, int* fail_at);

/* ---------------------------------------------------------------------------------------------
 * Logit distance distribution (LDD)
 * ---------------------------------------------------------------------------------------------
 * The auditing footprint of the paper: for every discrete decision of an audited request, the
 * distance between the logits the deployed execution committed to and the logits of the reference
 * execution (Section 4.2, definition of the logit distance distribution), the per-request tail
 * statistic built on it (Section 5.3), and the Top-K distance that lets a server commit K indices
 * instead of a whole logit vector (appendix on the verification of Top-K).
 *
 * Logit rows are float32, row-major: step i occupies entries [i*ld, i*ld + n) of its matrix
 * (ld >= n).  An entry may be -inf (a masked vocabulary entry: probability exactly 0); NaN and
 * +inf entries are not inputs (the row's results are then NaN, unchecked).  Rows that are 16-byte
 * aligned (base pointer and ld*4) are read with 128-bit loads, others element by element.  All pointers are DEVICE pointers; calls
 * enqueue on `stream` and do not synchronise; nothing is allocated.  The arithmetic is float32
 * per entry (exp2-based softmax) with the cross-thread sums in float64; the Top-K distance is
 * selected exactly and evaluated in float64.
 */
#define IMM_LDD_MAX_N (1 << 20)        /* entries per logit row                      */
#define IMM_LDD_MAX_K 64               /* size of a Top-K index set                  */
#define IMM_LDD_MAX_STEPS (1 << 27)    /* rows (or requests) per call                */

/* tv[i] = 1/2 * sum_v |p_v - q_v| and kl[i] = sum_v q_v (log q_v - log p_v), where
 * p = softmax(logits row i) (the deployed execution) and q = softmax(ref_logits row i) (the
 * reference), temperature 1.  The paper names "KL divergence or TV distance" without fixing the
 * KL direction: the reference distribution comes first here.  Masked entries: 0 log 0 = 0, so an
 * entry without reference mass adds nothing to kl; kl[i] = +inf when the reference gives mass to an
 * entry the deployed row masks; a row with no finite entry has no distribution and gives
 * tv[i] = kl[i] = NaN (which imm_ldd_tail_fraction counts as exceeding any threshold).
 * Errors: IMM_ERR_ARG (null pointer), IMM_ERR_SHAPE (n <= 0, ld < n, n or steps beyond the limits
 * above), IMM_ERR_ALIGN (pointers not aligned to their element size), IMM_ERR_CUDA. */
int imm_ldd_tv_kl(const float* d_logits, const float* d_ref_logits, int64_t steps, int64_t n, int64_t ld,
                  double* d_tv, double* d_kl, void* stream);

/* dist[i] = min over rows l' whose K largest entries are exactly the index set I_i of
 * ||l' - l_i||_1, with l_i = ref_logits row i and I_i = d_topk[i*k .. i*k + k) (k distinct
 * indices in [0, n)).  It is 0 iff I_i is a valid top-K set of the row.  Computed as the minimum
 * over finite thresholds t of  sum_{j not in I} max(l_j - t, 0) + sum_{i in I} max(t - l_i, 0):
 * a masked (-inf) entry outside I costs nothing, a masked member of I makes dist[i] = +inf.
 * status[i] = IMM_OK, IMM_ERR_ARG (an index out of range or repeated; dist[i] = NaN), or
 * IMM_ERR_LIMIT (after six refinements more than 256 entries of one 8192-entry slice still lie
 * above the bound on its K-th largest entry; dist[i] = NaN).
 * d_ws: DEVICE workspace of at least imm_ldd_topk_workspace(steps, n, k) bytes, 16-byte aligned;
 * the call overwrites it (a flag word and the K largest entries of every 8192-entry slice).
 * Errors of the call itself: as imm_ldd_tv_kl, plus IMM_ERR_SHAPE for k outside
 * 1..min(n, IMM_LDD_MAX_K) and IMM_ERR_WORKSPACE. */
size_t imm_ldd_topk_workspace(int64_t steps, int64_t n, int k);
int imm_ldd_topk_distance(const float* d_ref_logits, int64_t steps, int64_t n, int64_t ld,
                          const int32_t* d_topk, int k, double* d_dist, int32_t* d_status,
                          void* d_ws, size_t ws_bytes, void* stream);

/* Per-request tail statistic: request r owns the steps offsets[r] .. offsets[r+1]-1 of `dist`
 * (offsets: nrequests + 1 non-decreasing int64 values).  p[r] = (number of its steps with
 * dist > t1) / (number of its steps), 0 for an empty request; flag[r] = 1 if p[r] > t2 else 0
 * (d_flag may be null).  Both comparisons are strict, as the paper prints them.  A step whose
 * distance is NaN -- imm_ldd_topk_distance writes NaN for a malformed index set, imm_ldd_tv_kl for
 * a row without a finite logit -- counts as exceeding t1: what is not known to be within the
 * threshold never lowers p[r], so a server cannot escape the flag by committing garbage. */
int imm_ldd_tail_fraction(const double* d_dist, const int64_t* d_offsets, int64_t nrequests, double t1, double t2,
                          double* d_p, int32_t* d_flag, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* IMM_H_ */
