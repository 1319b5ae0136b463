/*
 * Reference definition of the symmetric rank-k update on the lower triangle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * GPU library must compute.  It shares no code with the CUDA path and must be
 * used only by the tests, the smoke check and the CPU-baseline leg of the
 * benchmark; the product never calls it.
 *
 * What it follows: the triple loop that defines SYRK in the paper (Algorithm 1:
 * for i, for j <= i, for k: C[i][j] += A[i][k] * A[j][k]), extended by the
 * scalars alpha and beta of the library's entry point:
 *
 *     C[i][j] <- alpha * sum_k A[i][k] * A[j][k] + beta * C[i][j]     (i >= j)
 *
 * The triangle-block schedule of the paper performs exactly these multiply-adds
 * in another order (Section 5, opening paragraph), so the definition itself is
 * the numeric reference.  Everything is done in binary64: bf16 inputs are
 * widened exactly (their 16 bits are the upper half of a binary32), products of
 * two widened bf16 values are exact in binary64, and only the k-sum rounds.
 * TF32 inputs are binary32 values of which only the TF32 part counts: sign, 8
 * exponent bits and the 10 leading fraction bits, i.e. the 19 high-order bits of
 * the encoding; the 13 low-order bits are dropped (not rounded) before the value
 * is widened.  This is the published TF32 format; the paper itself fixes no
 * input precision.  Products of two such values have at most 22 significant
 * bits and are exact in binary64.
 * FP8 inputs are bytes in the OCP 8-bit floating-point format E4M3: 1 sign bit,
 * 4 exponent bits (bias 7), 3 fraction bits; exponent field 0 holds the
 * subnormals f/8 * 2^-6; there are no infinities and the only NaN is exponent
 * and fraction all ones (0x7F, 0xFF); the largest finite value is 448.  Each
 * byte is decoded exactly; products have at most 8 significant bits.
 * FP16 inputs are IEEE 754 binary16 bit patterns: 1 sign bit, 5 exponent bits
 * (bias 15), 10 fraction bits; exponent field 0 holds zero and the subnormals
 * f * 2^-24, exponent field 31 infinity (f = 0) and NaN.  Each pattern is
 * decoded exactly; products have at most 22 significant bits and exponents of at
 * least -48, so they are exact in binary64 (and in binary32).
 * The k-sum is sequential, with no reassociation and no fused multiply-add
 * (compile with -ffp-contract=off).
 *
 * Rows are independent, so the outer loop may be spread over host threads
 * (OpenMP); that changes no arithmetic within an entry.
 *
 * Besides the reference value the routines return the bound matrix
 *     B[i][j] = sum_k |A[i][k]| * |A[j][k]|
 * that the parity tolerance is stated in.
 *
 * Parity status: pinned (closed forms, an independent outer-product loop nest
 * on small inputs, symmetry, exact-integer cases, alpha/beta algebra) by the
 * CPU tests.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_DTYPE_F64 = 0, ORACLE_DTYPE_BF16_F32 = 1, ORACLE_DTYPE_TF32_F32 = 2, ORACLE_DTYPE_E4M3_F32 = 3,
       ORACLE_DTYPE_F16_F32 = 4 };

static inline double widen_bf16(uint16_t bits) {
    union { uint32_t u; float f; } x;
    x.u = ((uint32_t)bits) << 16;
    return (double)x.f;
}

static inline double widen_tf32(uint32_t bits) {
    union { uint32_t u; float f; } x;
    x.u = bits & 0xFFFFE000u;              /* keep sign, exponent, 10 fraction bits */
    return (double)x.f;
}

static inline double widen_e4m3(uint8_t bits) {
    const int sign = bits >> 7, e = (bits >> 3) & 15, f = bits & 7;
    double v;
    if (e == 15 && f == 7) return NAN;
    if (e == 0) v = ldexp((double)f, -9);                 /* f/8 * 2^-6 */
    else v = ldexp((double)(8 + f), e - 10);              /* (1 + f/8) * 2^(e-7) */
    return sign ? -v : v;
}

static inline double widen_f16(uint16_t bits) {
    const int sign = bits >> 15, e = (bits >> 10) & 31, f = bits & 1023;
    double v;
    if (e == 31) v = f ? NAN : INFINITY;
    else if (e == 0) v = ldexp((double)f, -24);           /* f/1024 * 2^-14 */
    else v = ldexp((double)(1024 + f), e - 25);           /* (1 + f/1024) * 2^(e-15) */
    return sign ? -v : v;
}

/* Element A[r][k] as a double, for any input type. */
static inline double a_at(const void* A, int64_t lda, int dtype, int64_t r, int64_t k) {
    if (dtype == ORACLE_DTYPE_F64) return ((const double*)A)[r * lda + k];
    if (dtype == ORACLE_DTYPE_TF32_F32) return widen_tf32(((const uint32_t*)A)[r * lda + k]);
    if (dtype == ORACLE_DTYPE_E4M3_F32) return widen_e4m3(((const uint8_t*)A)[r * lda + k]);
    if (dtype == ORACLE_DTYPE_F16_F32) return widen_f16(((const uint16_t*)A)[r * lda + k]);
    return widen_bf16(((const uint16_t*)A)[r * lda + k]);
}

/* Element C_in[i][j] as a double (binary64 C, or binary32 C for bf16, TF32, FP8 and FP16 inputs). */
static inline double c_at(const void* C, int64_t ldc, int dtype, int64_t i, int64_t j) {
    if (dtype == ORACLE_DTYPE_F64) return ((const double*)C)[i * ldc + j];
    return (double)((const float*)C)[i * ldc + j];
}

/* One entry: the k loop of Algorithm 1, then alpha and beta. */
static void one_entry(int64_t M, const void* A, int64_t lda, int dtype,
                      const void* Cin, int64_t ldc, double alpha, double beta,
                      int64_t i, int64_t j, double* ref, double* bound) {
    double s = 0.0, b = 0.0;
    for (int64_t k = 0; k < M; ++k) {
        double x = a_at(A, lda, dtype, i, k);
        double y = a_at(A, lda, dtype, j, k);
        s += x * y;
        b += fabs(x) * fabs(y);
    }
    double prior = (beta == 0.0) ? 0.0 : beta * c_at(Cin, ldc, dtype, i, j);
    *ref = prior + alpha * s;
    *bound = b;
}

/*
 * Whole lower triangle.  Cref and Bound are N x ldr binary64, row-major; only
 * entries with i >= j are written.  Cin may be NULL when beta == 0 (it is not
 * read then).  Returns 0, or -1 on a bad argument.
 */
int oracle_syrk_lower(int64_t N, int64_t M, const void* A, int64_t lda,
                      const void* Cin, int64_t ldc, double alpha, double beta,
                      int dtype, double* Cref, double* Bound, int64_t ldr) {
    if (N < 0 || M < 0 || dtype < ORACLE_DTYPE_F64 || dtype > ORACLE_DTYPE_F16_F32) return -1;
    if (N > 0 && (!Cref || !Bound || ldr < N)) return -1;
    if (N > 0 && M > 0 && (!A || lda < M)) return -1;
    if (N > 0 && beta != 0.0 && (!Cin || ldc < N)) return -1;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < N; ++i) {
        for (int64_t j = 0; j <= i; ++j) {
            one_entry(M, A, lda, dtype, Cin, ldc, alpha, beta, i, j,
                      &Cref[i * ldr + j], &Bound[i * ldr + j]);
        }
    }
    return 0;
}

/*
 * A list of entries (I[p], J[p]), p < P, each computed exactly as above; used
 * to check sampled outputs at sizes where the whole triangle is too slow.
 * Pairs with I[p] < J[p] are rejected.
 */
int oracle_syrk_entries(int64_t P, const int64_t* I, const int64_t* J,
                        int64_t N, int64_t M, const void* A, int64_t lda,
                        const void* Cin, int64_t ldc, double alpha, double beta,
                        int dtype, double* ref, double* bound) {
    if (P < 0 || N < 0 || M < 0) return -1;
    if (dtype < ORACLE_DTYPE_F64 || dtype > ORACLE_DTYPE_F16_F32) return -1;
    for (int64_t p = 0; p < P; ++p)
        if (I[p] < J[p] || J[p] < 0 || I[p] >= N) return -1;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t p = 0; p < P; ++p)
        one_entry(M, A, lda, dtype, Cin, ldc, alpha, beta, I[p], J[p], &ref[p], &bound[p]);
    return 0;
}

/* The N x M operand (row pitch lda) widened element by element to binary64, exactly, by the functions above:
 * dst is N x M, dense.  For references of other updates on the same input types (the rank-2k update), so
 * that every reference reads a storage format through the one pinned decoder.  Returns 0, or -1 on a bad
 * argument. */
int oracle_widen(int64_t N, int64_t M, const void* A, int64_t lda, int dtype, double* dst) {
    if (N < 0 || M < 0 || lda < (M > 1 ? M : 1) || dtype < 0 || dtype > 4 || ((N > 0 && M > 0) && (!A || !dst))) return -1;
    for (int64_t r = 0; r < N; ++r)
        for (int64_t k = 0; k < M; ++k) dst[r * M + k] = a_at(A, lda, dtype, r, k);
    return 0;
}

/* Host threads the loops above run on. */
int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
