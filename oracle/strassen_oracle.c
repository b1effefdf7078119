/*
 * CPU oracle for the Strassen-Winograd hot path.  TEST INFRASTRUCTURE ONLY:
 * nothing in the product library includes, links or calls this file; it is
 * compiled by oracle/__init__.py with gcc (-O2 -ffp-contract=off -fopenmp)
 * and used by the tests, the smoke check and the benchmark's CPU baseline.
 *
 * Two independent routines, both plain FP64, row-major:
 *
 *   oracle_classical  -- the definition of the result (the paper's problem
 *       statement, Algorithm 1 "Ensure C = A.B"): C[i][j] = sum_k A[i][k]B[k][j],
 *       k ascending, one multiply and one add per term, never fused.
 *
 *   oracle_sw -- the sequential Strassen-Winograd recursion (Appendix A, with
 *       the three sign/operand typos of the printed table corrected, see
 *       sw_step below), switching to the classical product at or below a
 *       cutoff size (Section 5.4 "CAPS": classical below some size n0), with
 *       dynamic peeling of the last row and column when a size is odd
 *       (Section 3.1 names padding or dynamic peeling; peeling is used here).
 *       Each level combines its seven products either through the U1..U3
 *       chain of Appendix A ('B', as a breadth-first step holds all seven Q at
 *       once) or by folding one Q at a time into the quadrants of C ('D', the
 *       depth-first step of Algorithm 1: "compute contribution of Q_i to C").
 *
 * Pins (tests/test_oracle_*.py): classical against closed forms (identity,
 * permutation, power-of-two diagonal scaling, rank-one products, transposition,
 * Freivalds), a hand-worked golden product and numpy's matmul on integer data;
 * oracle_sw against oracle_classical (exact equality on small-integer inputs
 * for every size/cutoff/schedule in a sweep, odd sizes included), the count of
 * 7^L base products, and the flop closed form F(n) = c_s n^{log2 7} - 5 n^2
 * of Appendix A.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int64_t base_calls;   /* classical products executed at the leaves        */
    int64_t mults;        /* scalar multiplications                           */
    int64_t adds;         /* scalar additions/subtractions (leaf + block adds) */
    int64_t block_adds;   /* matrix additions/subtractions of quadrant size    */
    int64_t peels;        /* levels that split off a last row and column       */
} oracle_counters;

/* C (m x n) = A (m x k) . B (k x n); the definition, k ascending.
 * Rows are split over threads, so the result does not depend on the thread count. */
void oracle_classical(const double *A, int64_t lda, const double *B, int64_t ldb,
                      double *C, int64_t ldc, int64_t m, int64_t n, int64_t k)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < m; ++i) {
        double *c = C + i * ldc;
        if (k == 0) { for (int64_t j = 0; j < n; ++j) c[j] = 0.0; continue; }
        const double a0 = A[i * lda];
        for (int64_t j = 0; j < n; ++j) c[j] = a0 * B[j];
        for (int64_t p = 1; p < k; ++p) {
            const double a = A[i * lda + p];
            const double *b = B + p * ldb;
            for (int64_t j = 0; j < n; ++j) c[j] = c[j] + a * b[j];
        }
    }
}

/* Same definition for a list of sampled output entries: out[t] = row rows[t] of A
 * times column cols[t] of B.  Used where a full product is too slow. */
void oracle_classical_samples(const double *A, int64_t lda, const double *B, int64_t ldb,
                              int64_t k, const int64_t *rows, const int64_t *cols,
                              int64_t count, double *out)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < count; ++t) {
        const double *a = A + rows[t] * lda;
        const double *b = B + cols[t];
        double s = 0.0;
        if (k > 0) s = a[0] * b[0];
        for (int64_t p = 1; p < k; ++p) s = s + a[p] * b[p * ldb];
        out[t] = s;
    }
}

/* ---- quadrant-sized helpers (single-threaded inside; callers parallelise) ---- */

static void blk_add(const double *X, int64_t ldx, const double *Y, int64_t ldy,
                    double *Z, int64_t ldz, int64_t h, oracle_counters *cnt)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < h; ++i)
        for (int64_t j = 0; j < h; ++j)
            Z[i * ldz + j] = X[i * ldx + j] + Y[i * ldy + j];
    cnt->adds += h * h; cnt->block_adds += 1;
}

static void blk_sub(const double *X, int64_t ldx, const double *Y, int64_t ldy,
                    double *Z, int64_t ldz, int64_t h, oracle_counters *cnt)
{
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < h; ++i)
        for (int64_t j = 0; j < h; ++j)
            Z[i * ldz + j] = X[i * ldx + j] - Y[i * ldy + j];
    cnt->adds += h * h; cnt->block_adds += 1;
}

static void blk_copy(const double *X, int64_t ldx, double *Z, int64_t ldz, int64_t h)
{
    for (int64_t i = 0; i < h; ++i)
        memcpy(Z + i * ldz, X + i * ldx, (size_t)h * sizeof(double));
}

static int sw_rec(const double *A, int64_t lda, const double *B, int64_t ldb,
                  double *C, int64_t ldc, int64_t n, int64_t cutoff,
                  const char *sched, oracle_counters *cnt);

/* One Strassen-Winograd step on an even size n = 2h (Appendix A).
 *
 * The table as printed gives T3 = T2 - A12, S2 = B12 + B11, T5 = A12 + T3, which
 * does not reproduce C12, C21 or C22; the reading used here is the standard
 * Winograd form, the only choice of those three entries that satisfies the four
 * block identities with the Q, U and C columns as printed:
 *     T3 = T2 - A11,  S2 = B12 - B11,  T5 = A12 - T3.
 * T_j are the A-side combinations, S_j the B-side ones, Q_j = T_j . S_j.
 */
static int sw_step(const double *A, int64_t lda, const double *B, int64_t ldb,
                   double *C, int64_t ldc, int64_t n, int64_t cutoff,
                   const char *sched, oracle_counters *cnt)
{
    const int64_t h = n / 2;
    const double *A11 = A, *A12 = A + h, *A21 = A + h * lda, *A22 = A + h * lda + h;
    const double *B11 = B, *B12 = B + h, *B21 = B + h * ldb, *B22 = B + h * ldb + h;
    double *C11 = C, *C12 = C + h, *C21 = C + h * ldc, *C22 = C + h * ldc + h;
    const char mode = (sched && *sched) ? *sched : 'B';
    const char *next = (sched && *sched) ? sched + 1 : sched;
    const size_t q = (size_t)h * (size_t)h;

    double *T2 = malloc(q * 8), *T3 = malloc(q * 8), *T4 = malloc(q * 8), *T5 = malloc(q * 8);
    double *S2 = malloc(q * 8), *S3 = malloc(q * 8), *S4 = malloc(q * 8), *S6 = malloc(q * 8);
    int rc = 0;
    if (!T2 || !T3 || !T4 || !T5 || !S2 || !S3 || !S4 || !S6) { rc = -1; goto done_st; }

    blk_add(A21, lda, A22, lda, T2, h, h, cnt);   /* T2 = A21 + A22 */
    blk_sub(T2, h, A11, lda, T3, h, h, cnt);      /* T3 = T2  - A11 */
    blk_sub(A11, lda, A21, lda, T4, h, h, cnt);   /* T4 = A11 - A21 */
    blk_sub(A12, lda, T3, h, T5, h, h, cnt);      /* T5 = A12 - T3  */
    blk_sub(B12, ldb, B11, ldb, S2, h, h, cnt);   /* S2 = B12 - B11 */
    blk_sub(B22, ldb, S2, h, S3, h, h, cnt);      /* S3 = B22 - S2  */
    blk_sub(B22, ldb, B12, ldb, S4, h, h, cnt);   /* S4 = B22 - B12 */
    blk_sub(S3, h, B21, ldb, S6, h, h, cnt);      /* S6 = S3  - B21 */

    /* operands of the seven products; T0,T1,T6 and S0,S1,S5 are plain quadrants */
    const double *TT[7] = { A11, A12, T2, T3, T4, T5, A22 };
    const int64_t ldT[7] = { lda, lda, h, h, h, h, lda };
    const double *SS[7] = { B11, B21, S2, S3, S4, B22, S6 };
    const int64_t ldS[7] = { ldb, ldb, h, h, h, ldb, h };

    if (mode == 'D') {
        /* depth-first step: one Q at a time, folded into C and discarded.
         * Flat contributions (expansion of the U chain):
         *   C11 = Q0+Q1, C12 = Q0+Q3+Q2+Q5, C21 = Q0+Q3+Q4-Q6, C22 = Q0+Q3+Q4+Q2. */
        double *Q = malloc(q * 8);
        if (!Q) { rc = -1; goto done_st; }
        for (int j = 0; j < 7 && rc == 0; ++j) {
            rc = sw_rec(TT[j], ldT[j], SS[j], ldS[j], Q, h, h, cutoff, next, cnt);
            if (rc) break;
            switch (j) {
            case 0: blk_copy(Q, h, C11, ldc, h); blk_copy(Q, h, C12, ldc, h);
                    blk_copy(Q, h, C21, ldc, h); blk_copy(Q, h, C22, ldc, h); break;
            case 1: blk_add(C11, ldc, Q, h, C11, ldc, h, cnt); break;
            case 2: blk_add(C12, ldc, Q, h, C12, ldc, h, cnt);
                    blk_add(C22, ldc, Q, h, C22, ldc, h, cnt); break;
            case 3: blk_add(C12, ldc, Q, h, C12, ldc, h, cnt);
                    blk_add(C21, ldc, Q, h, C21, ldc, h, cnt);
                    blk_add(C22, ldc, Q, h, C22, ldc, h, cnt); break;
            case 4: blk_add(C21, ldc, Q, h, C21, ldc, h, cnt);
                    blk_add(C22, ldc, Q, h, C22, ldc, h, cnt); break;
            case 5: blk_add(C12, ldc, Q, h, C12, ldc, h, cnt); break;
            case 6: blk_sub(C21, ldc, Q, h, C21, ldc, h, cnt); break;
            }
        }
        free(Q);
    } else {
        /* breadth-first step: all seven Q held at once, combined by the U chain */
        double *Q[7] = { 0 };
        for (int j = 0; j < 7; ++j) { Q[j] = malloc(q * 8); if (!Q[j]) rc = -1; }
        for (int j = 0; j < 7 && rc == 0; ++j)
            rc = sw_rec(TT[j], ldT[j], SS[j], ldS[j], Q[j], h, h, cutoff, next, cnt);
        if (rc == 0) {
            double *U1 = T2, *U2 = T3, *U3 = T4;           /* reuse freed operand space */
            blk_add(Q[0], h, Q[3], h, U1, h, h, cnt);      /* U1  = Q0 + Q3 */
            blk_add(U1, h, Q[4], h, U2, h, h, cnt);        /* U2  = U1 + Q4 */
            blk_add(U1, h, Q[2], h, U3, h, h, cnt);        /* U3  = U1 + Q2 */
            blk_add(Q[0], h, Q[1], h, C11, ldc, h, cnt);   /* C11 = Q0 + Q1 */
            blk_add(U3, h, Q[5], h, C12, ldc, h, cnt);     /* C12 = U3 + Q5 */
            blk_sub(U2, h, Q[6], h, C21, ldc, h, cnt);     /* C21 = U2 - Q6 */
            blk_add(U2, h, Q[2], h, C22, ldc, h, cnt);     /* C22 = U2 + Q2 */
        }
        for (int j = 0; j < 7; ++j) free(Q[j]);
    }
done_st:
    free(T2); free(T3); free(T4); free(T5); free(S2); free(S3); free(S4); free(S6);
    return rc;
}

/* Dynamic peeling for odd n = 2h+1 (textbook block algebra):
 *   A = [A1 ac; ar al],  B = [B1 bc; br be],  A1, B1 of size n-1:
 *   C1    = A1.B1 + ac.br      (recursion on n-1, then a rank-one update)
 *   ccol  = A1.bc + ac.be      (last column, first n-1 rows)
 *   crow  = ar.B1 + al.br      (last row, first n-1 columns)
 *   gamma = ar.bc + al.be
 * The last three are written here as full dot products over k = 0..n-1. */
static int sw_peel(const double *A, int64_t lda, const double *B, int64_t ldb,
                   double *C, int64_t ldc, int64_t n, int64_t cutoff,
                   const char *sched, oracle_counters *cnt)
{
    const int64_t e = n - 1;
    int rc = sw_step(A, lda, B, ldb, C, ldc, e, cutoff, sched, cnt);
    if (rc) return rc;
    cnt->peels += 1;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < e; ++i) {
        const double a = A[i * lda + e];
        for (int64_t j = 0; j < e; ++j)
            C[i * ldc + j] = C[i * ldc + j] + a * B[e * ldb + j];
    }
    cnt->mults += e * e; cnt->adds += e * e;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) {           /* last column, all n rows */
        double s = A[i * lda] * B[e];
        for (int64_t p = 1; p < n; ++p) s = s + A[i * lda + p] * B[p * ldb + e];
        C[i * ldc + e] = s;
    }
#pragma omp parallel for schedule(static)
    for (int64_t j = 0; j < e; ++j) {           /* last row, first n-1 columns */
        double s = A[e * lda] * B[j];
        for (int64_t p = 1; p < n; ++p) s = s + A[e * lda + p] * B[p * ldb + j];
        C[e * ldc + j] = s;
    }
    cnt->mults += (2 * n - 1) * n; cnt->adds += (2 * n - 1) * (n - 1);
    return 0;
}

static int sw_rec(const double *A, int64_t lda, const double *B, int64_t ldb,
                  double *C, int64_t ldc, int64_t n, int64_t cutoff,
                  const char *sched, oracle_counters *cnt)
{
    if (n <= cutoff) {
        oracle_classical(A, lda, B, ldb, C, ldc, n, n, n);
        cnt->base_calls += 1;
        cnt->mults += n * n * n;
        cnt->adds += n * n * (n - 1);
        return 0;
    }
    if (n & 1) return sw_peel(A, lda, B, ldb, C, ldc, n, cutoff, sched, cnt);
    return sw_step(A, lda, B, ldb, C, ldc, n, cutoff, sched, cnt);
}

/* C = A.B by Strassen-Winograd; recurse while the current size exceeds cutoff.
 * sched: NULL or "" = every level combines by the U chain; otherwise one char per
 * level, top first, 'B' or 'D' (levels past the end of the string use 'B').
 * Returns 0, -1 on allocation failure, -2 on bad arguments. */
int oracle_sw(const double *A, int64_t lda, const double *B, int64_t ldb,
              double *C, int64_t ldc, int64_t n, int64_t cutoff,
              const char *sched, oracle_counters *cnt)
{
    oracle_counters local;
    if (!cnt) cnt = &local;
    memset(cnt, 0, sizeof *cnt);
    if (n < 1 || cutoff < 1 || !A || !B || !C) return -2;
    return sw_rec(A, lda, B, ldb, C, ldc, n, cutoff, sched, cnt);
}
