/*
 * imm_oracle.c -- plain, slow CPU oracle for the sumcheck proof of an int8 matrix product
 * over the Goldilocks field.  TEST INFRASTRUCTURE ONLY: nothing on the product path may call,
 * link or import this file; it shares no code, table or constant generator with the CUDA
 * library and is the authority the CUDA results are compared against, bit for bit.
 *
 * What it instantiates.  The paper treats verifiable computation as a black-box pair
 * (Prove, Vrfy) for a deterministic public function (Section 2.2) and asks that the proof
 * establish that "continuous transformations" -- the attention and MLP matrix products of the
 * reference model -- were computed as claimed (Section 5.2, item 2; Algorithm 3, the
 * F_theta* step).  The paper gives no proof system.  This oracle therefore writes out the
 * textbook definitions: the prime field, multilinear extensions, and the sumcheck protocol for
 * sum_y A~(r_row,y) * B~(y,r_col) = C~(r_row,r_col).  Every function below is the definition
 * itself (reduction with the % operator on 128-bit integers, plain loops, no blocking, no
 * fusion, no reordering).
 *
 * Conventions (fixed by this implementation; the paper is silent on all of them):
 *   field       p = 2^64 - 2^32 + 1; elements are canonical uint64 in [0, p).
 *   lift        signed integer v -> v mod p (negative v -> p - |v|).
 *   variables   an index of n bits has variables z_0..z_{n-1}, z_0 the MOST significant bit.
 *   eq          eq(r, i) = prod_t (bit_t(i) ? r_t : 1 - r_t).
 *   padding     a dimension d is padded with zeros at the high end to 2^ceil(log2 d).
 *   transcript  [c0, g_0(0), g_0(1), g_0(2), ..., g_{b-1}(0..2), a_fin, b_fin], 3b+3 words.
 *   challenges  public coins from a counter-based generator built on the SplitMix64 output
 *               mixer (Steele, Lea, Flood 2014): they do not depend on the prover's messages.
 *
 * Pins (tests/test_oracle_*.py): published SplitMix64 outputs, Goldilocks identities
 * (2^64 = 2^32-1, 2^96 = -1, the published 2^32-th root of unity), Python big-integer
 * arithmetic, MLE values at Boolean points, exhaustive hypercube sums for every round
 * polynomial on tiny shapes, closed forms (identity / all-ones matrices, extra padding
 * variable), g(0)+g(1) = running claim, accept honest / reject tampered; for the batched
 * proof: the exhaustive big-integer definition of the combined round polynomials, the
 * single-proof transcript at P = 1, linearity in the per-proof transcripts, soundness cases.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

#define ORC_P 0xFFFFFFFF00000001ULL

enum { ORC_I8 = 0, ORC_I32 = 1 };
enum { ORC_BIND_ROWS = 0, ORC_BIND_COLS = 1 };
enum { ORC_OK = 0, ORC_REJECT = 1, ORC_ERR_ARG = -1 };

/* ------------------------------------------------------------------ field ---------- */

uint64_t orc_add(uint64_t x, uint64_t y) { return (uint64_t)(((u128)x + (u128)y) % ORC_P); }
uint64_t orc_sub(uint64_t x, uint64_t y) { return (uint64_t)(((u128)x + ORC_P - (u128)y) % ORC_P); }
uint64_t orc_mul(uint64_t x, uint64_t y) { return (uint64_t)(((u128)x * (u128)y) % ORC_P); }

uint64_t orc_pow(uint64_t x, uint64_t e)
{
    uint64_t acc = 1;
    while (e) {
        if (e & 1) acc = orc_mul(acc, x);
        x = orc_mul(x, x);
        e >>= 1;
    }
    return acc;
}

/* signed integer -> field element */
uint64_t orc_lift(int64_t v)
{
    if (v >= 0) return (uint64_t)v % ORC_P;
    /* -v fits because callers pass int8/int32 values */
    uint64_t mag = (uint64_t)(-v) % ORC_P;
    return mag == 0 ? 0 : ORC_P - mag;
}

/* ------------------------------------------------------------------ challenges ----- */

#define ORC_GAMMA 0x9E3779B97F4A7C15ULL

/* SplitMix64 output mixer */
uint64_t orc_mix64(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

uint64_t orc_stream(uint64_t seed, uint64_t sid, uint64_t ctr)
{
    uint64_t key = orc_mix64(orc_mix64(seed + ORC_GAMMA) + ORC_GAMMA * (sid + 1));
    return orc_mix64(key + ORC_GAMMA * (ctr + 1));
}

/* domain 1 = r_row, 2 = r_col, 3 = sumcheck round */
uint64_t orc_challenge(uint64_t seed, uint64_t proof_id, uint32_t domain, uint32_t index)
{
    uint64_t x = orc_stream(seed, proof_id, ((uint64_t)domain << 32) | (uint64_t)index);
    return x >= ORC_P ? x - ORC_P : x;
}

/* ------------------------------------------------------------------ helpers -------- */

int orc_ceil_log2(int64_t d)
{
    int n = 0;
    while (((int64_t)1 << n) < d) n++;
    return n;
}

static int64_t mat_get(const void* mat, int dtype, int64_t ld, int64_t i, int64_t j)
{
    if (dtype == ORC_I8) return (int64_t)((const int8_t*)mat)[i * ld + j];
    return (int64_t)((const int32_t*)mat)[i * ld + j];
}

/* ------------------------------------------------------------------ eq ------------- */

/* closed form: eq(r, i) for an nvars-bit index i, variable 0 = most significant bit */
uint64_t orc_eq_closed(const uint64_t* r, int nvars, uint64_t i)
{
    uint64_t acc = 1;
    for (int t = 0; t < nvars; t++) {
        uint64_t bit = (i >> (nvars - 1 - t)) & 1;
        acc = orc_mul(acc, bit ? r[t] : orc_sub(1, r[t]));
    }
    return acc;
}

/* table E[i] = eq(r, i), i < 2^nvars, by repeated doubling */
void orc_eq_table(const uint64_t* r, int nvars, uint64_t* out)
{
    out[0] = 1;
    for (int t = 0; t < nvars; t++) {
        int64_t len = (int64_t)1 << t;
        for (int64_t i = len - 1; i >= 0; i--) {
            uint64_t hi = orc_mul(out[i], r[t]);
            out[2 * i + 1] = hi;
            out[2 * i] = orc_sub(out[i], hi);
        }
    }
}

/* ------------------------------------------------------------------ MLE ------------ */

/* M~(x, y) = sum_{i,j} eq(x,i) eq(y,j) lift(M[i,j]) straight from the definition; x has
 * ceil_log2(rows) coordinates, y has ceil_log2(cols).  O(rows*cols*(a+c)) -- tiny inputs. */
uint64_t orc_mle_eval_bruteforce(const void* mat, int dtype, int64_t rows, int64_t cols,
                                 int64_t ld, const uint64_t* x, const uint64_t* y)
{
    int a = orc_ceil_log2(rows), c = orc_ceil_log2(cols);
    uint64_t acc = 0;
    for (int64_t i = 0; i < rows; i++)
        for (int64_t j = 0; j < cols; j++) {
            uint64_t w = orc_mul(orc_eq_closed(x, a, (uint64_t)i), orc_eq_closed(y, c, (uint64_t)j));
            acc = orc_add(acc, orc_mul(w, orc_lift(mat_get(mat, dtype, ld, i, j))));
        }
    return acc;
}

/* BIND_ROWS: out[y] = sum_{i<rows} eq[i] lift(M[i,y]), y < cols
 * BIND_COLS: out[i] = sum_{j<cols} lift(M[i,j]) eq[j], i < rows            */
void orc_mle_partial_eval(const void* mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
                          int bind, const uint64_t* eq, uint64_t* out)
{
    if (bind == ORC_BIND_ROWS) {
        for (int64_t y = 0; y < cols; y++) {
            uint64_t acc = 0;
            for (int64_t i = 0; i < rows; i++)
                acc = orc_add(acc, orc_mul(eq[i], orc_lift(mat_get(mat, dtype, ld, i, y))));
            out[y] = acc;
        }
    } else {
        for (int64_t i = 0; i < rows; i++) {
            uint64_t acc = 0;
            for (int64_t j = 0; j < cols; j++)
                acc = orc_add(acc, orc_mul(orc_lift(mat_get(mat, dtype, ld, i, j)), eq[j]));
            out[i] = acc;
        }
    }
}

/* sum_{i,j} eq_row[i] lift(M[i,j]) eq_col[j] */
uint64_t orc_mle_eval_point(const void* mat, int dtype, int64_t rows, int64_t cols, int64_t ld,
                            const uint64_t* eq_row, const uint64_t* eq_col)
{
    uint64_t acc = 0;
    for (int64_t i = 0; i < rows; i++) {
        uint64_t rowsum = 0;
        for (int64_t j = 0; j < cols; j++)
            rowsum = orc_add(rowsum, orc_mul(orc_lift(mat_get(mat, dtype, ld, i, j)), eq_col[j]));
        acc = orc_add(acc, orc_mul(eq_row[i], rowsum));
    }
    return acc;
}

/* ------------------------------------------------------------------ protocol ------- */

/* Prover for the claim C = A*B.  A is m x k int8 (ld lda), B is k x n int8, C is m x n int32.
 * C is used AS GIVEN: the prover never substitutes A*B for it.
 *   1. r_row (a coords), r_col (c coords), r_k (b coords) from the challenge generator.
 *   2. avec[y] = sum_i E_row[i] lift(A[i,y]);  bvec[y] = sum_j lift(B[y,j]) E_col[j];
 *      both zero for k <= y < 2^b.
 *   3. c0 = sum_{i,j} E_row[i] lift(C[i,j]) E_col[j].
 *   4. round j (half = 2^(b-1-j)): g(0) = sum_{y<half} a[y] b[y];
 *      g(1) = sum a[y+half] b[y+half]; g(2) = sum (2a[y+half]-a[y]) (2b[y+half]-b[y]);
 *      then a[y] <- a[y] + r_k[j] (a[y+half]-a[y]), same for b.
 *   5. a_fin = a[0], b_fin = b[0].
 * transcript must hold 3*ceil_log2(k)+3 words.  Returns ORC_OK or ORC_ERR_ARG. */
int orc_sumcheck_matmul_prove(const int8_t* A, const int8_t* B, const int32_t* C,
                              int64_t m, int64_t k, int64_t n,
                              int64_t lda, int64_t ldb, int64_t ldc,
                              uint64_t seed, uint64_t proof_id, uint64_t* transcript)
{
    if (m <= 0 || k <= 0 || n <= 0 || lda < k || ldb < n || ldc < n) return ORC_ERR_ARG;
    int a = orc_ceil_log2(m), b = orc_ceil_log2(k), c = orc_ceil_log2(n);
    int64_t mp = (int64_t)1 << a, kp = (int64_t)1 << b, np = (int64_t)1 << c;

    uint64_t* r_row = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(a + 1));
    uint64_t* r_col = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(c + 1));
    uint64_t* e_row = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)mp);
    uint64_t* e_col = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)np);
    uint64_t* av = (uint64_t*)calloc((size_t)kp, sizeof(uint64_t));
    uint64_t* bv = (uint64_t*)calloc((size_t)kp, sizeof(uint64_t));
    if (!r_row || !r_col || !e_row || !e_col || !av || !bv) {
        free(r_row); free(r_col); free(e_row); free(e_col); free(av); free(bv);
        return ORC_ERR_ARG;
    }
    for (int t = 0; t < a; t++) r_row[t] = orc_challenge(seed, proof_id, 1, (uint32_t)t);
    for (int t = 0; t < c; t++) r_col[t] = orc_challenge(seed, proof_id, 2, (uint32_t)t);
    orc_eq_table(r_row, a, e_row);
    orc_eq_table(r_col, c, e_col);

    orc_mle_partial_eval(A, ORC_I8, m, k, lda, ORC_BIND_ROWS, e_row, av);
    orc_mle_partial_eval(B, ORC_I8, k, n, ldb, ORC_BIND_COLS, e_col, bv);
    uint64_t* w = transcript;
    *w++ = orc_mle_eval_point(C, ORC_I32, m, n, ldc, e_row, e_col);

    for (int j = 0; j < b; j++) {
        int64_t half = (int64_t)1 << (b - 1 - j);
        uint64_t g0 = 0, g1 = 0, g2 = 0;
        for (int64_t y = 0; y < half; y++) {
            uint64_t a0 = av[y], a1 = av[y + half], b0 = bv[y], b1 = bv[y + half];
            uint64_t a2 = orc_sub(orc_add(a1, a1), a0);
            uint64_t b2 = orc_sub(orc_add(b1, b1), b0);
            g0 = orc_add(g0, orc_mul(a0, b0));
            g1 = orc_add(g1, orc_mul(a1, b1));
            g2 = orc_add(g2, orc_mul(a2, b2));
        }
        *w++ = g0; *w++ = g1; *w++ = g2;
        uint64_t r = orc_challenge(seed, proof_id, 3, (uint32_t)j);
        for (int64_t y = 0; y < half; y++) {
            av[y] = orc_add(av[y], orc_mul(r, orc_sub(av[y + half], av[y])));
            bv[y] = orc_add(bv[y], orc_mul(r, orc_sub(bv[y + half], bv[y])));
        }
    }
    *w++ = av[0];
    *w++ = bv[0];
    free(r_row); free(r_col); free(e_row); free(e_col); free(av); free(bv);
    return ORC_OK;
}

/* value at r of the degree-2 polynomial through (0,g0), (1,g1), (2,g2):
 * g(r) = g0 (r-1)(r-2)/2 + g1 r (2-r) + g2 r (r-1)/2                                   */
uint64_t orc_interp_deg2(uint64_t g0, uint64_t g1, uint64_t g2, uint64_t r)
{
    const uint64_t inv2 = 0x7FFFFFFF80000001ULL;   /* (p+1)/2 */
    uint64_t rm1 = orc_sub(r, 1), rm2 = orc_sub(r, 2);
    uint64_t t0 = orc_mul(orc_mul(g0, orc_mul(rm1, rm2)), inv2);
    uint64_t t1 = orc_mul(g1, orc_mul(r, orc_sub(2, r)));
    uint64_t t2 = orc_mul(orc_mul(g2, orc_mul(r, rm1)), inv2);
    return orc_add(orc_add(t0, t1), t2);
}

/* Verifier.  claim <- c0; per round require g(0)+g(1) = claim, claim <- g(r_k[j]); finally
 * require claim = a_fin * b_fin.  Optional expected values for c0 / a_fin / b_fin (the
 * verifier's own evaluations of C~, A~, B~) are compared when non-NULL.
 * *fail_at: -1 accept; j = round j's sum check failed; nrounds = final product check failed;
 * nrounds+1 / +2 / +3 = c0 / a_fin / b_fin differ from the expected value.              */
int orc_sumcheck_verify(const uint64_t* transcript, int nrounds, uint64_t seed,
                        uint64_t proof_id, const uint64_t* expect_c0,
                        const uint64_t* expect_a_fin, const uint64_t* expect_b_fin,
                        int* fail_at)
{
    if (!transcript || nrounds < 0 || !fail_at) return ORC_ERR_ARG;
    for (int t = 0; t < 3 * nrounds + 3; t++)
        if (transcript[t] >= ORC_P) return ORC_ERR_ARG;
    uint64_t claim = transcript[0];
    for (int j = 0; j < nrounds; j++) {
        uint64_t g0 = transcript[1 + 3 * j], g1 = transcript[2 + 3 * j], g2 = transcript[3 + 3 * j];
        if (orc_add(g0, g1) != claim) { *fail_at = j; return ORC_REJECT; }
        claim = orc_interp_deg2(g0, g1, g2, orc_challenge(seed, proof_id, 3, (uint32_t)j));
    }
    uint64_t a_fin = transcript[3 * nrounds + 1], b_fin = transcript[3 * nrounds + 2];
    if (orc_mul(a_fin, b_fin) != claim) { *fail_at = nrounds; return ORC_REJECT; }
    if (expect_c0 && *expect_c0 != transcript[0]) { *fail_at = nrounds + 1; return ORC_REJECT; }
    if (expect_a_fin && *expect_a_fin != a_fin) { *fail_at = nrounds + 2; return ORC_REJECT; }
    if (expect_b_fin && *expect_b_fin != b_fin) { *fail_at = nrounds + 3; return ORC_REJECT; }
    *fail_at = -1;
    return ORC_OK;
}

/* exact integer product C = A*B (int32), the plain triple loop */
void orc_matmul_i8_i32(const int8_t* A, const int8_t* B, int32_t* C,
                       int64_t m, int64_t k, int64_t n)
{
    for (int64_t i = 0; i < m; i++)
        for (int64_t j = 0; j < n; j++) C[i * n + j] = 0;
    for (int64_t i = 0; i < m; i++)
        for (int64_t y = 0; y < k; y++) {
            int32_t aiy = A[i * k + y];
            for (int64_t j = 0; j < n; j++) C[i * n + j] += aiy * (int32_t)B[y * n + j];
        }
}

/* ---------------------------------------------------------------------------------------
 * Batched proof: P product claims C_p = A_p * B_p are proved by ONE sumcheck of their random
 * linear combination over b = max_p ceil(log2 k_p) variables (a member with a smaller k is
 * zero-padded to 2^b like any other: padding k changes neither its product nor its claim) (the standard batching of sumcheck claims
 * over a common hypercube; the paper lists the products to prove -- attention and MLPs,
 * Section 4.1 -- and leaves the proof system and any batching open).
 *
 *   rho_p      = challenge(seed, batch_id, 4, p)             combination coefficients
 *   r_j        = challenge(seed, batch_id, 3, j)             round challenges, shared by all p
 *   r_row, r_col of proof p come from its own proof_id (domains 1 and 2), as in the single proof.
 *
 * Combined claim   c0^B = sum_p rho_p c0_p,  c0_p = C~_p(r_row_p, r_col_p).
 * Round j          g_j^B(X) = sum_p rho_p g_j^(p)(X), g_j^(p) the single-proof round polynomial
 *                  of proof p under the shared challenges r_0..r_{j-1}.
 * After b rounds   a_fin_p = A~_p(r_row_p, r),  b_fin_p = B~_p(r, r_col_p).
 *
 * transcript (1 + 3b + 3P words):
 *   [c0^B, g_0^B(0..2), ..., g_{b-1}^B(0..2), (c0_0, a_fin_0, b_fin_0), ..., (c0_{P-1}, ...)].
 * Every proof keeps its own vectors; there is no sharing of work between proofs beyond the
 * challenges.  Returns ORC_ERR_ARG for a bad shape.                                       */
int orc_sumcheck_matmul_prove_batched(int P, const int8_t* const* A, const int8_t* const* B,
                                      const int32_t* const* C, const int64_t* m, const int64_t* k,
                                      const int64_t* n, const int64_t* lda, const int64_t* ldb,
                                      const int64_t* ldc, uint64_t seed, uint64_t batch_id,
                                      const uint64_t* proof_ids, uint64_t* transcript)
{
    if (P <= 0 || !A || !B || !C || !m || !k || !n || !lda || !ldb || !ldc || !proof_ids || !transcript)
        return ORC_ERR_ARG;
    for (int p = 0; p < P; p++)
        if (m[p] <= 0 || k[p] <= 0 || n[p] <= 0 || lda[p] < k[p] || ldb[p] < n[p] || ldc[p] < n[p])
            return ORC_ERR_ARG;
    int b = 0;
    for (int p = 0; p < P; p++)
        if (orc_ceil_log2(k[p]) > b) b = orc_ceil_log2(k[p]);
    int64_t kp = (int64_t)1 << b;

    uint64_t** av = (uint64_t**)calloc((size_t)P, sizeof(uint64_t*));
    uint64_t** bv = (uint64_t**)calloc((size_t)P, sizeof(uint64_t*));
    uint64_t* rho = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)P);
    if (!av || !bv || !rho) { free(av); free(bv); free(rho); return ORC_ERR_ARG; }
    uint64_t* tail = transcript + 1 + 3 * b;
    uint64_t c0_batch = 0;
    int rc = ORC_OK;
    for (int p = 0; p < P && rc == ORC_OK; p++) {
        int a = orc_ceil_log2(m[p]), c = orc_ceil_log2(n[p]);
        uint64_t* r_row = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(a + 1));
        uint64_t* r_col = (uint64_t*)malloc(sizeof(uint64_t) * (size_t)(c + 1));
        uint64_t* e_row = (uint64_t*)malloc(sizeof(uint64_t) << a);
        uint64_t* e_col = (uint64_t*)malloc(sizeof(uint64_t) << c);
        av[p] = (uint64_t*)calloc((size_t)kp, sizeof(uint64_t));
        bv[p] = (uint64_t*)calloc((size_t)kp, sizeof(uint64_t));
        if (!r_row || !r_col || !e_row || !e_col || !av[p] || !bv[p]) rc = ORC_ERR_ARG;
        else {
            for (int t = 0; t < a; t++) r_row[t] = orc_challenge(seed, proof_ids[p], 1, (uint32_t)t);
            for (int t = 0; t < c; t++) r_col[t] = orc_challenge(seed, proof_ids[p], 2, (uint32_t)t);
            orc_eq_table(r_row, a, e_row);
            orc_eq_table(r_col, c, e_col);
            orc_mle_partial_eval(A[p], ORC_I8, m[p], k[p], lda[p], ORC_BIND_ROWS, e_row, av[p]);
            orc_mle_partial_eval(B[p], ORC_I8, k[p], n[p], ldb[p], ORC_BIND_COLS, e_col, bv[p]);
            rho[p] = orc_challenge(seed, batch_id, 4, (uint32_t)p);
            tail[3 * p] = orc_mle_eval_point(C[p], ORC_I32, m[p], n[p], ldc[p], e_row, e_col);
            c0_batch = orc_add(c0_batch, orc_mul(rho[p], tail[3 * p]));
        }
        free(r_row); free(r_col); free(e_row); free(e_col);
    }
    if (rc == ORC_OK) {
        uint64_t* w = transcript;
        *w++ = c0_batch;
        for (int j = 0; j < b; j++) {
            int64_t half = (int64_t)1 << (b - 1 - j);
            uint64_t r = orc_challenge(seed, batch_id, 3, (uint32_t)j);
            uint64_t g0 = 0, g1 = 0, g2 = 0;
            for (int p = 0; p < P; p++) {
                uint64_t s0 = 0, s1 = 0, s2 = 0;
                for (int64_t y = 0; y < half; y++) {
                    uint64_t a0 = av[p][y], a1 = av[p][y + half], b0 = bv[p][y], b1 = bv[p][y + half];
                    uint64_t a2 = orc_sub(orc_add(a1, a1), a0);
                    uint64_t b2 = orc_sub(orc_add(b1, b1), b0);
                    s0 = orc_add(s0, orc_mul(a0, b0));
                    s1 = orc_add(s1, orc_mul(a1, b1));
                    s2 = orc_add(s2, orc_mul(a2, b2));
                }
                g0 = orc_add(g0, orc_mul(rho[p], s0));
                g1 = orc_add(g1, orc_mul(rho[p], s1));
                g2 = orc_add(g2, orc_mul(rho[p], s2));
                for (int64_t y = 0; y < half; y++) {
                    av[p][y] = orc_add(av[p][y], orc_mul(r, orc_sub(av[p][y + half], av[p][y])));
                    bv[p][y] = orc_add(bv[p][y], orc_mul(r, orc_sub(bv[p][y + half], bv[p][y])));
                }
            }
            *w++ = g0; *w++ = g1; *w++ = g2;
        }
        for (int p = 0; p < P; p++) { tail[3 * p + 1] = av[p][0]; tail[3 * p + 2] = bv[p][0]; }
    }
    for (int p = 0; p < P; p++) { free(av[p]); free(bv[p]); }
    free(av); free(bv); free(rho);
    return rc;
}

/* Verifier of a batched transcript.  claim <- c0^B, which must equal sum_p rho_p c0_p; per round
 * g(0)+g(1) = claim, claim <- g(r_j); finally claim = sum_p rho_p a_fin_p b_fin_p.  expect, when
 * non-NULL, holds the verifier's own 3P values (c0_p, a_fin_p, b_fin_p) and is compared word
 * for word.
 * *fail_at: -1 accept; j = round j; nrounds = the final check; nrounds+1 = c0^B is not the
 * combination of the listed c0_p; nrounds+2+t = word t of the per-proof tail differs from
 * expect.                                                                                 */
int orc_sumcheck_verify_batched(const uint64_t* transcript, int nrounds, int P, uint64_t seed,
                                uint64_t batch_id, const uint64_t* expect, int* fail_at)
{
    if (!transcript || nrounds < 0 || P <= 0 || !fail_at) return ORC_ERR_ARG;
    for (int t = 0; t < 1 + 3 * nrounds + 3 * P; t++)
        if (transcript[t] >= ORC_P) return ORC_ERR_ARG;
    const uint64_t* tail = transcript + 1 + 3 * nrounds;
    uint64_t combo = 0, fin = 0;
    for (int p = 0; p < P; p++) {
        uint64_t rho = orc_challenge(seed, batch_id, 4, (uint32_t)p);
        combo = orc_add(combo, orc_mul(rho, tail[3 * p]));
        fin = orc_add(fin, orc_mul(rho, orc_mul(tail[3 * p + 1], tail[3 * p + 2])));
    }
    uint64_t claim = transcript[0];
    if (claim != combo) { *fail_at = nrounds + 1; return ORC_REJECT; }
    for (int j = 0; j < nrounds; j++) {
        uint64_t g0 = transcript[1 + 3 * j], g1 = transcript[2 + 3 * j], g2 = transcript[3 + 3 * j];
        if (orc_add(g0, g1) != claim) { *fail_at = j; return ORC_REJECT; }
        claim = orc_interp_deg2(g0, g1, g2, orc_challenge(seed, batch_id, 3, (uint32_t)j));
    }
    if (fin != claim) { *fail_at = nrounds; return ORC_REJECT; }
    if (expect)
        for (int t = 0; t < 3 * P; t++)
            if (expect[t] != tail[t]) { *fail_at = nrounds + 2 + t; return ORC_REJECT; }
    *fail_at = -1;
    return ORC_OK;
}
