// Plain-load SYRK and the scale-only kernel.
//
// syrk_plain: one thread per entry (i, j), j <= i, of the result of Algorithm 1 of the
// paper with alpha/beta; no TMA, no alignment requirement.  It is the slow path for
// inputs whose base address or row pitch is not a multiple of 16 bytes, for either storage
// order of A (N x M, or M x N for the Gram form).
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "kernels.h"

namespace tbsyrk {
namespace {

template <typename TA, typename TC> struct Widen;
template <> struct Widen<double, double> { static __device__ double get(const double* p) { return *p; } };
template <> struct Widen<__nv_bfloat16, float> {
    static __device__ float get(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};

template <> struct Widen<__half, float> {
    static __device__ float get(const __half* p) { return __half2float(*p); }
};

// binary32 read as TF32: the 13 low-order bits of the encoding are dropped.
template <> struct Widen<float, float> {
    static __device__ float get(const float* p) { return __uint_as_float(__float_as_uint(*p) & 0xFFFFE000u); }
};

// FP8 E4M3 byte: (-1)^s * 2^(e-7) * (1 + f/8); e = 0: 2^-6 * f/8; e = 15, f = 7: NaN.
template <> struct Widen<uint8_t, float> {
    static __device__ float get(const uint8_t* p) {
        const int b = *p, e = (b >> 3) & 15, f = b & 7;
        float v = (e == 0) ? ldexpf(float(f), -9) : ldexpf(float(8 + f), e - 10);
        if (e == 15 && f == 7) v = __int_as_float(0x7FC00000);
        return (b & 0x80) ? -v : v;
    }
};

template <typename TA, typename TC>
__global__ void syrk_plain_kernel(int64_t N, int64_t M, const TA* __restrict__ A, int64_t row_stride,
                                  int64_t col_stride, TC* __restrict__ C, int64_t ldc, TC alpha, TC beta, int upper) {
    const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t i = int64_t(blockIdx.y) * blockDim.y + threadIdx.y;
    if (i >= N || j >= N || (upper ? j < i : j > i)) return;
    const TA* ai = A + i * row_stride;       // row i of the N x M operand, whichever way it is stored
    const TA* aj = A + j * row_stride;
    TC s = TC(0);
    for (int64_t k = 0; k < M; ++k)
        s = fma(Widen<TA, TC>::get(ai + k * col_stride), Widen<TA, TC>::get(aj + k * col_stride), s);
    TC* c = C + i * ldc + j;
    *c = (beta == TC(0)) ? alpha * s : alpha * s + beta * *c;
}

__global__ void syr2k_plain_kernel(int64_t N, int64_t M, const double* __restrict__ A, int64_t lda,
                                   const double* __restrict__ B, int64_t ldb, double* __restrict__ C, int64_t ldc,
                                   double alpha, double beta) {
    const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t i = int64_t(blockIdx.y) * blockDim.y + threadIdx.y;
    if (i >= N || j > i) return;
    double s = 0.0;
    for (int64_t k = 0; k < M; ++k)
        s = fma(A[i * lda + k], B[j * ldb + k], fma(B[i * ldb + k], A[j * lda + k], s));
    double* c = C + i * ldc + j;
    *c = (beta == 0.0) ? alpha * s : alpha * s + beta * *c;
}

// Hermitian rank-k update, one thread per entry (i, j), j <= i; complex numbers as (re, im) pairs.
__global__ void herk_plain_kernel(int64_t N, int64_t M, const double* __restrict__ A, int64_t lda,
                                  double* __restrict__ C, int64_t ldc, double alpha, double beta) {
    const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t i = int64_t(blockIdx.y) * blockDim.y + threadIdx.y;
    if (i >= N || j > i) return;
    const double* ai = A + 2 * i * lda;
    const double* aj = A + 2 * j * lda;
    double sr = 0.0, si = 0.0;
    for (int64_t k = 0; k < M; ++k) {
        const double a = ai[2 * k], b = ai[2 * k + 1], c = aj[2 * k], d = aj[2 * k + 1];
        sr = fma(a, c, fma(b, d, sr));
        si = fma(b, c, fma(-a, d, si));
    }
    double* c = C + 2 * (i * ldc + j);
    double vr = alpha * sr, vi = alpha * si;
    if (beta != 0.0) { vr += beta * c[0]; if (i != j) vi += beta * c[1]; }
    c[0] = vr;
    c[1] = (i == j) ? 0.0 : vi;
}

// The same for the storage types that accumulate in binary32 (each product is exact in binary32).
template <typename TA>
__global__ void syr2k_plain_f32_kernel(int64_t N, int64_t M, const TA* __restrict__ A, int64_t lda, const TA* __restrict__ B,
                                       int64_t ldb, float* __restrict__ C, int64_t ldc, float alpha, float beta) {
    const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t i = int64_t(blockIdx.y) * blockDim.y + threadIdx.y;
    if (i >= N || j > i) return;
    float s = 0.f;
    for (int64_t k = 0; k < M; ++k)
        s = fmaf(Widen<TA, float>::get(A + i * lda + k), Widen<TA, float>::get(B + j * ldb + k),
                 fmaf(Widen<TA, float>::get(B + i * ldb + k), Widen<TA, float>::get(A + j * lda + k), s));
    float* c = C + i * ldc + j;
    *c = (beta == 0.f) ? alpha * s : alpha * s + beta * *c;
}

template <typename TC>
__global__ void scale_lower_kernel(int64_t N, TC* __restrict__ C, int64_t ldc, TC beta, int upper) {
    const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t i = int64_t(blockIdx.y) * blockDim.y + threadIdx.y;
    if (i >= N || j >= N || (upper ? j < i : j > i)) return;
    TC* c = C + i * ldc + j;
    *c = (beta == TC(0)) ? TC(0) : beta * *c;
}

inline dim3 grid2d(int64_t N, dim3 block) {
    return dim3(unsigned((N + block.x - 1) / block.x), unsigned((N + block.y - 1) / block.y));
}

}  // namespace

cudaError_t launch_syrk_plain(int dtype, int64_t N, int64_t M, const void* A, int64_t lda, void* C,
                              int64_t ldc, double alpha, double beta, int a_is_m_by_n, cudaStream_t stream, int upper) {
    if (N == 0) return cudaSuccess;
    const dim3 block(32, 8);
    const int64_t rs = a_is_m_by_n ? 1 : lda, cs = a_is_m_by_n ? lda : 1;
    if (dtype == 0)
        syrk_plain_kernel<double, double><<<grid2d(N, block), block, 0, stream>>>(
            N, M, static_cast<const double*>(A), rs, cs, static_cast<double*>(C), ldc, alpha, beta, upper);
    else if (dtype == 3)
        syrk_plain_kernel<uint8_t, float><<<grid2d(N, block), block, 0, stream>>>(
            N, M, static_cast<const uint8_t*>(A), rs, cs, static_cast<float*>(C), ldc, float(alpha), float(beta), upper);
    else if (dtype == 4)
        syrk_plain_kernel<__half, float><<<grid2d(N, block), block, 0, stream>>>(
            N, M, static_cast<const __half*>(A), rs, cs, static_cast<float*>(C), ldc, float(alpha), float(beta), upper);
    else if (dtype == 2)
        syrk_plain_kernel<float, float><<<grid2d(N, block), block, 0, stream>>>(
            N, M, static_cast<const float*>(A), rs, cs, static_cast<float*>(C), ldc, float(alpha), float(beta), upper);
    else
        syrk_plain_kernel<__nv_bfloat16, float><<<grid2d(N, block), block, 0, stream>>>(
            N, M, static_cast<const __nv_bfloat16*>(A), rs, cs, static_cast<float*>(C), ldc,
            float(alpha), float(beta), upper);
    return cudaGetLastError();
}

cudaError_t launch_syr2k_plain(int64_t N, int64_t M, const double* A, int64_t lda, const double* B, int64_t ldb,
                               double* C, int64_t ldc, double alpha, double beta, cudaStream_t stream) {
    if (N == 0) return cudaSuccess;
    const dim3 block(32, 8);
    syr2k_plain_kernel<<<grid2d(N, block), block, 0, stream>>>(N, M, A, lda, B, ldb, C, ldc, alpha, beta);
    return cudaGetLastError();
}

cudaError_t launch_herk_plain(int64_t N, int64_t M, const double* A, int64_t lda, double* C, int64_t ldc,
                              double alpha, double beta, cudaStream_t stream) {
    if (N == 0) return cudaSuccess;
    const dim3 block(32, 8);
    herk_plain_kernel<<<grid2d(N, block), block, 0, stream>>>(N, alpha == 0.0 ? 0 : M, A, lda, C, ldc, alpha, beta);
    return cudaGetLastError();
}

cudaError_t launch_syr2k_plain_f32(int dtype, int64_t N, int64_t M, const void* A, int64_t lda, const void* B, int64_t ldb,
                                   float* C, int64_t ldc, float alpha, float beta, cudaStream_t stream) {
    if (N == 0) return cudaSuccess;
    const dim3 block(32, 8);
    const dim3 grid = grid2d(N, block);
    if (dtype == 3)
        syr2k_plain_f32_kernel<uint8_t><<<grid, block, 0, stream>>>(N, M, static_cast<const uint8_t*>(A), lda,
                                                                    static_cast<const uint8_t*>(B), ldb, C, ldc, alpha, beta);
    else if (dtype == 4)
        syr2k_plain_f32_kernel<__half><<<grid, block, 0, stream>>>(N, M, static_cast<const __half*>(A), lda,
                                                                   static_cast<const __half*>(B), ldb, C, ldc, alpha, beta);
    else if (dtype == 2)
        syr2k_plain_f32_kernel<float><<<grid, block, 0, stream>>>(N, M, static_cast<const float*>(A), lda,
                                                                  static_cast<const float*>(B), ldb, C, ldc, alpha, beta);
    else
        syr2k_plain_f32_kernel<__nv_bfloat16><<<grid, block, 0, stream>>>(N, M, static_cast<const __nv_bfloat16*>(A), lda,
                                                                          static_cast<const __nv_bfloat16*>(B), ldb, C, ldc, alpha, beta);
    return cudaGetLastError();
}

cudaError_t launch_scale_lower(int dtype, int64_t N, void* C, int64_t ldc, double beta,
                               cudaStream_t stream, int upper) {
    if (N == 0) return cudaSuccess;
    const dim3 block(32, 8);
    if (dtype == 0)
        scale_lower_kernel<double><<<grid2d(N, block), block, 0, stream>>>(N, static_cast<double*>(C), ldc, beta, upper);
    else
        scale_lower_kernel<float><<<grid2d(N, block), block, 0, stream>>>(N, static_cast<float*>(C), ldc, float(beta), upper);
    return cudaGetLastError();
}

}  // namespace tbsyrk
