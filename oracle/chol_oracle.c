/*
 * Reference Cholesky factorisation, lower triangle, in place.
 *
 * TEST INFRASTRUCTURE ONLY (used by the tests and the smoke check; the GPU library never
 * calls it).  Plain statement of the triple loop that defines the factorisation in the paper
 * (Algorithm 2):
 *
 *     for k:  A[k][k] = sqrt(A[k][k])
 *             for i > k:  A[i][k] = A[i][k] / A[k][k]
 *                         for j in k+1 .. i:  A[i][j] -= A[i][k] * A[j][k]     (update operations)
 *
 * binary64, no reassociation, no fused multiply-add (compile with -ffp-contract=off).  Only
 * entries with j <= i are read or written.  For a fixed k the rows i are independent, so
 * that loop may be spread over host threads without changing any arithmetic.
 *
 * Returns 0, -1 on a bad argument, or k + 1 when the pivot A[k][k] is not positive (the
 * matrix is not positive definite; the factorisation stops there).
 *
 * Parity status: pinned by the CPU tests (hand-worked 3 x 3 example, Pascal matrices whose
 * factor is the binomial triangle, exact integer factors, reconstruction, a library
 * cross-check, detection of an indefinite matrix).
 *
 * oracle_cholesky_lower_leading is the same triple loop with k and j restricted to the first
 * `ncols` columns.  In Algorithm 2 an entry A[i][j] is only ever updated with values of columns
 * k < j, so the first ncols columns of the factor depend on the first ncols columns of A alone and
 * come out exactly as in the full factorisation (same operations, same order): N * ncols^2 / 2
 * multiply-adds instead of N^3 / 6, which lets the tests check the leading columns of the factor of
 * a matrix too large to factor whole on the host.  Pinned by bitwise equality with the leading
 * columns of the full routine, the binomial triangle and the hand-worked example.
 */
#include <math.h>
#include <stdint.h>

int64_t oracle_cholesky_lower(int64_t N, double* A, int64_t lda) {
    if (N < 0 || (N > 0 && (!A || lda < N))) return -1;
    for (int64_t k = 0; k < N; ++k) {
        const double p = A[k * lda + k];
        if (!(p > 0.0)) return k + 1;
        const double d = sqrt(p);
        A[k * lda + k] = d;
        for (int64_t i = k + 1; i < N; ++i) A[i * lda + k] = A[i * lda + k] / d;
#pragma omp parallel for schedule(static) if (N - k > 256)
        for (int64_t i = k + 1; i < N; ++i) {
            const double aik = A[i * lda + k];
            for (int64_t j = k + 1; j <= i; ++j) A[i * lda + j] -= aik * A[j * lda + k];
        }
    }
    return 0;
}

int64_t oracle_cholesky_lower_leading(int64_t N, int64_t ncols, double* A, int64_t lda) {
    if (N < 0 || ncols < 0 || ncols > N || (N > 0 && (!A || lda < ncols))) return -1;
    for (int64_t k = 0; k < ncols; ++k) {
        const double p = A[k * lda + k];
        if (!(p > 0.0)) return k + 1;
        const double d = sqrt(p);
        A[k * lda + k] = d;
        for (int64_t i = k + 1; i < N; ++i) A[i * lda + k] = A[i * lda + k] / d;
#pragma omp parallel for schedule(static) if (N - k > 256)
        for (int64_t i = k + 1; i < N; ++i) {
            const double aik = A[i * lda + k];
            const int64_t jend = i < ncols - 1 ? i : ncols - 1;
            for (int64_t j = k + 1; j <= jend; ++j) A[i * lda + j] -= aik * A[j * lda + k];
        }
    }
    return 0;
}
