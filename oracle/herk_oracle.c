/*
 * Reference definition of the Hermitian rank-k update on the lower triangle.
 *
 * TEST INFRASTRUCTURE ONLY: used by the tests; the product never calls it and it
 * shares no code with the CUDA path.
 *
 * What it follows: the paper treats the symmetric rank-k update (Algorithm 1) and, in
 * its conclusion (Section 6), names other kernels that use the same input several
 * times as the place its ideas extend to.  The Hermitian update is Algorithm 1 over
 * the complex numbers with the second factor conjugated,
 *
 *     C[i][j] <- alpha * sum_k A[i][k] * conj(A[j][k]) + beta * C[i][j]        (i >= j),
 *
 * A complex N x M, C complex Hermitian N x N, alpha and beta real.  With
 * A[i][k] = a + b i and A[j][k] = c + d i one term is (a c + b d) + (b c - a d) i.
 * Complex numbers are stored as (real, imaginary) pairs of binary64; pitches are in
 * complex elements.  For each k the two products of a part are combined first and the
 * result is added to the running sum of that part, sequentially in k, without fused
 * multiply-add (compile with -ffp-contract=off).
 *
 * The diagonal of a Hermitian matrix is real: the imaginary part of C[i][i] is not read
 * and is returned as zero (the terms b a - a b cancel exactly).
 *
 * Besides the value the routine returns, per part, the bound that the parity tolerance
 * is stated in:
 *     Bound[i][j] = ( sum_k |a||c| + |b||d| ,  sum_k |b||c| + |a||d| ).
 *
 * Parity status: pinned by the CPU tests (a hand-worked example; a real A gives the pinned
 * symmetric reference and a zero imaginary part; Gaussian integers against a library
 * product; rows with unit phases giving the identity; multiplication of columns by i
 * changing no bit; row exchange giving the conjugate; the algebra of alpha and beta).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

int oracle_herk_lower(int64_t N, int64_t M, const double* A, int64_t lda,
                      const double* Cin, int64_t ldc, double alpha, double beta,
                      double* Cref, double* Bound, int64_t ldr) {
    if (N < 0 || M < 0) return -1;
    if (N > 0 && (!Cref || !Bound || ldr < N)) return -1;
    if (N > 0 && M > 0 && (!A || lda < M)) return -1;
    if (N > 0 && beta != 0.0 && (!Cin || ldc < N)) return -1;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < N; ++i) {
        for (int64_t j = 0; j <= i; ++j) {
            double sr = 0.0, si = 0.0, br = 0.0, bi = 0.0;
            for (int64_t k = 0; k < M; ++k) {
                const double a = A[2 * (i * lda + k)], b = A[2 * (i * lda + k) + 1];
                const double c = A[2 * (j * lda + k)], d = A[2 * (j * lda + k) + 1];
                sr += a * c + b * d;
                si += b * c - a * d;
                br += fabs(a) * fabs(c) + fabs(b) * fabs(d);
                bi += fabs(b) * fabs(c) + fabs(a) * fabs(d);
            }
            const double pr = (beta == 0.0) ? 0.0 : beta * Cin[2 * (i * ldc + j)];
            const double pi = (beta == 0.0 || i == j) ? 0.0 : beta * Cin[2 * (i * ldc + j) + 1];
            Cref[2 * (i * ldr + j)] = pr + alpha * sr;
            Cref[2 * (i * ldr + j) + 1] = (i == j) ? 0.0 : pi + alpha * si;
            Bound[2 * (i * ldr + j)] = br;
            Bound[2 * (i * ldr + j) + 1] = bi;
        }
    }
    return 0;
}
