/*
 * Reference definition of the symmetric rank-2k update on the lower triangle.
 *
 * TEST INFRASTRUCTURE ONLY: used by the tests; the product never calls it and it
 * shares no code with the CUDA path.
 *
 * What it follows: the paper treats SYRK and Cholesky and, in its conclusion
 * (Section 6), names other kernels that use the same input several times as
 * the place its ideas extend to.  The rank-2k update is the nearest such
 * kernel; its definition is the plain one,
 *
 *     C[i][j] <- alpha * sum_k (A[i][k] * B[j][k] + B[i][k] * A[j][k]) + beta * C[i][j]   (i >= j),
 *
 * with A and B both N x M: the loop nest of Algorithm 1 with the product
 * A[i][k] * A[j][k] replaced by the symmetrised pair.  Everything is binary64;
 * for each k the two products are added to each other first and then to the
 * running sum (so that exchanging A and B changes no bit), sequentially in k,
 * without fused multiply-add (compile with -ffp-contract=off).
 *
 * Besides the value the routine returns the bound
 *     Bd[i][j] = sum_k (|A[i][k]| |B[j][k]| + |B[i][k]| |A[j][k]|)
 * that the parity tolerance is stated in.
 *
 * Parity status: pinned by the CPU tests (B = A gives twice the pinned SYRK
 * reference; exact rationals through an independent loop nest; closed forms;
 * exchange of A and B bit for bit; alpha / beta algebra on integers).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

int oracle_syr2k_lower(int64_t N, int64_t M, const double* A, int64_t lda,
                       const double* B, int64_t ldb, const double* Cin, int64_t ldc,
                       double alpha, double beta, double* Cref, double* Bound, int64_t ldr) {
    if (N < 0 || M < 0) return -1;
    if (N > 0 && (!Cref || !Bound || ldr < N)) return -1;
    if (N > 0 && M > 0 && (!A || !B || lda < M || ldb < M)) return -1;
    if (N > 0 && beta != 0.0 && (!Cin || ldc < N)) return -1;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < N; ++i) {
        for (int64_t j = 0; j <= i; ++j) {
            double s = 0.0, b = 0.0;
            for (int64_t k = 0; k < M; ++k) {
                const double ai = A[i * lda + k], aj = A[j * lda + k];
                const double bi = B[i * ldb + k], bj = B[j * ldb + k];
                s += ai * bj + bi * aj;
                b += fabs(ai) * fabs(bj) + fabs(bi) * fabs(aj);
            }
            const double prior = (beta == 0.0) ? 0.0 : beta * Cin[i * ldc + j];
            Cref[i * ldr + j] = prior + alpha * s;
            Bound[i * ldr + j] = b;
        }
    }
    return 0;
}
