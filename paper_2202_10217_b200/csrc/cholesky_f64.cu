// Large Block Cholesky (Algorithm 5 of the paper, LBC) in FP64, lower triangle, in place.
//
// Right-looking blocked factorisation with block size b (default 512).  For the panel of
// columns I0 = [o, o + b):
//   1. A[I0, I0] <- its Cholesky factor                      (the paper's OOC_CHOL step)
//   2. A[I1, I0] <- A[I1, I0] * L00^-T, I1 = [o + b, N)      (the paper's OOC_TRSM step)
//   3. A[I1, I1] <- A[I1, I1] - A[I1, I0] * A[I1, I0]^T      (TBS: syrk_lower with alpha = -1,
//                                                             beta = 1, K = b, trailing view)
// Steps 1 and 2 are only cited by the paper; here they run in 128-column sub-steps.  A leaf
// kernel (one thread block) factors a 128 x 128 diagonal block in shared memory and inverts
// the factor; the rows below are solved as a product with that inverse (FP64 tensor-core
// kernel in two-operand mode) and the rest of the panel is updated by a small SYRK (inside the
// panel) and a product (below it).  Step 3 is the library's triangle-block SYRK.
#include <algorithm>
#include <mutex>

#include "../../include/tbsyrk.h"
#include "kernels.h"
#include "runtime.h"

namespace tbsyrk {
namespace {

constexpr int kLeaf = 128;
constexpr int kLeafThreads = 512;
constexpr int kPacked = kLeaf * (kLeaf + 1) / 2;                 // lower triangle, row-packed
constexpr int kLeafSmem = 2 * kPacked * int(sizeof(double));     // factor + inverse

__device__ __forceinline__ int pk(int i, int k) { return i * (i + 1) / 2 + k; }

// Factor the m x m block at A (lower triangle, row pitch lda) in place and write the inverse
// of the factor, as a full 128 x 128 row-major matrix with zeros above the diagonal and
// beyond m, to W.  On a non-positive pivot k, *info <- pivot_base + k + 1 if it is still 0.
__global__ void __launch_bounds__(kLeafThreads)
chol_leaf_kernel(double* __restrict__ A, int64_t lda, int m, double* __restrict__ W,
                 long long* __restrict__ info, long long pivot_base) {
    extern __shared__ double leaf_smem[];
    double* Ls = leaf_smem;
    double* Ws = leaf_smem + kPacked;
    __shared__ int s_bad;
    __shared__ double part[kLeafThreads];
    const int tid = threadIdx.x;
    const int col = tid & (kLeaf - 1), sub = tid >> 7;            // 4 threads share a column index

    if (tid == 0) s_bad = 0;
    for (int r = sub; r < m; r += 4)
        if (col <= r) Ls[pk(r, col)] = A[r * lda + col];
    __syncthreads();

    // ---- Cholesky, right-looking, one column per step (Algorithm 2 on the block) ----
    for (int k = 0; k < m; ++k) {
        const double p = Ls[pk(k, k)];
        if (!(p > 0.0)) {                                         // uniform: every thread reads the same p
            if (tid == 0) { atomicCAS(reinterpret_cast<unsigned long long*>(info), 0ull,
                                      static_cast<unsigned long long>(pivot_base + k + 1)); s_bad = 1; }
            break;
        }
        const double d = sqrt(p);
        __syncthreads();
        if (tid == 0) Ls[pk(k, k)] = d;
        if (sub == 0 && col > k && col < m) Ls[pk(col, k)] = Ls[pk(col, k)] / d;     // column k below the pivot
        __syncthreads();
        for (int i = k + 1 + sub; i < m; i += 4)                  // trailing update, 4 rows at a time
            if (col > k && col <= i) Ls[pk(i, col)] -= Ls[pk(i, k)] * Ls[pk(col, k)];
        __syncthreads();
    }
    __syncthreads();
    const bool bad = s_bad != 0;

    // ---- inverse of the factor: W[i][j] = (delta_ij - sum_{k=j}^{i-1} L[i][k] W[k][j]) / L[i][i] ----
    // Row by row; column j is shared by the 4 threads (sub = 0..3) that split the k-sum.
    if (!bad) {
        for (int i = 0; i < m; ++i) {
            double s = 0.0;
            if (col < i)
                for (int k = col + sub; k < i; k += 4) s -= Ls[pk(i, k)] * Ws[pk(k, col)];
            // combine the 4 partial sums of a column (they sit in 4 different warps)
            part[tid] = s;
            __syncthreads();
            if (sub == 0 && col <= i) {
                double acc = (col == i) ? 1.0 : 0.0;
                acc += part[col] + part[col + kLeaf] + part[col + 2 * kLeaf] + part[col + 3 * kLeaf];
                Ws[pk(i, col)] = acc / Ls[pk(i, i)];
            }
            __syncthreads();
        }
    }

    // ---- write back ----
    for (int r = sub; r < kLeaf; r += 4) {
        double w = 0.0;
        if (!bad && r < m && col <= r) w = Ws[pk(r, col)];
        W[r * kLeaf + col] = w;
        if (!bad && r < m && col <= r) A[r * lda + col] = Ls[pk(r, col)];
    }
}

struct CholWorkspace {
    double* w = nullptr;          // (block / 128) inverses, 128 x 128 each
    size_t w_bytes = 0;
    double* t = nullptr;          // N x 128 staging of a solved column block
    size_t t_bytes = 0;
    long long* info = nullptr;
};
std::mutex g_chol_mu;
CholWorkspace g_ws[64];

int gemm_nt(DeviceState* ds, int64_t nrows, int64_t ncols, int64_t K, const double* P, int64_t ldp,
            const double* Q, int64_t ldq, double* D, int64_t ldd, double alpha, double beta, cudaStream_t st) {
    if (nrows <= 0 || ncols <= 0 || K <= 0) return SYRK_OK;
    CUtensorMap tp, tq, td;
    int rc = encode_tensor_map_2d(&tp, SYRK_DTYPE_F64, P, nrows, K, ldp, f64_tile(), f64_bk());
    if (rc != SYRK_OK) return rc;
    rc = encode_tensor_map_2d(&tq, SYRK_DTYPE_F64, Q, ncols, K, ldq, f64_tile(), f64_bk());
    if (rc != SYRK_OK) return rc;
    const bool d_tma = beta != 0.0 && (reinterpret_cast<uintptr_t>(D) & 15) == 0 && (ldd & 1) == 0 &&
                       encode_tensor_map_f64_plain(&td, D, nrows, ncols, ldd, f64_tile(), f64_tile()) == SYRK_OK;
    return launch_gemm_nt_f64(tp, tq, d_tma ? &td : nullptr, nrows, ncols, K, D, ldd, alpha, beta, ds->d_status,
                              st) == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}

}  // namespace
}  // namespace tbsyrk

using namespace tbsyrk;

extern "C" int cholesky_lower(int64_t N, double* A, int64_t lda, int64_t block, void* stream) {
    if (N < 0 || N >= (int64_t(1) << 31) - 256) return SYRK_ERR_SIZE;
    if (N == 0) return SYRK_OK;
    if (!A) return SYRK_ERR_NULL;
    if (lda < N) return SYRK_ERR_LD;
    if ((reinterpret_cast<uintptr_t>(A) & 15) != 0 || (lda & 1) != 0) return SYRK_ERR_LD;   // TMA rules for the panels
    if (block == 0) block = 512;
    if (block < kLeaf || block > 4096 || block % kLeaf != 0) return SYRK_ERR_SIZE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    std::lock_guard<std::mutex> lock(runtime().mu);
    DeviceState* ds = nullptr;
    int rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    if (ds->device < 0 || ds->device >= 64) return SYRK_ERR_NO_DEVICE;
    CholWorkspace& ws = g_ws[ds->device];
    {
        std::lock_guard<std::mutex> l2(g_chol_mu);
        void* p = ws.w;
        if ((rc = ensure_device_bytes(&p, &ws.w_bytes, size_t(block / kLeaf) * kLeaf * kLeaf * sizeof(double))) != SYRK_OK) return rc;
        ws.w = static_cast<double*>(p);
        p = ws.t;
        if ((rc = ensure_device_bytes(&p, &ws.t_bytes, size_t(N) * kLeaf * sizeof(double))) != SYRK_OK) return rc;
        ws.t = static_cast<double*>(p);
        if (!ws.info && cudaMalloc(&ws.info, sizeof(long long)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_ALLOC; }
        static bool leaf_configured = false;
        if (!leaf_configured) {
            if (cudaFuncSetAttribute(chol_leaf_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLeafSmem) != cudaSuccess) {
                cudaGetLastError(); return SYRK_ERR_CUDA;
            }
            leaf_configured = true;
        }
    }
    if (cudaMemsetAsync(ws.info, 0, sizeof(long long), st) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }

    for (int64_t o = 0; o < N; o += block) {
        const int64_t bb = std::min<int64_t>(block, N - o);
        for (int64_t cj = o; cj < o + bb; cj += kLeaf) {
            const int m = int(std::min<int64_t>(kLeaf, o + bb - cj));
            double* Wj = ws.w + size_t((cj - o) / kLeaf) * kLeaf * kLeaf;
            chol_leaf_kernel<<<1, kLeafThreads, kLeafSmem, st>>>(A + cj * lda + cj, lda, m, Wj, ws.info, cj);
            if (cudaGetLastError() != cudaSuccess) return SYRK_ERR_CUDA;
            const int64_t below = N - (cj + m);
            if (below <= 0) continue;
            double* panel = A + (cj + m) * lda + cj;              // rows below the leaf, its m columns
            // solve: panel <- panel * L_jj^-T  (through the staging buffer: the product is not in place)
            if ((rc = gemm_nt(ds, below, m, m, panel, lda, Wj, kLeaf, ws.t, kLeaf, 1.0, 0.0, st)) != SYRK_OK) return rc;
            if (cudaMemcpy2DAsync(panel, size_t(lda) * 8, ws.t, size_t(kLeaf) * 8, size_t(m) * 8, size_t(below),
                                  cudaMemcpyDeviceToDevice, st) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
            const int64_t rem = o + bb - (cj + m);                // panel columns still to be updated
            if (rem <= 0) continue;
            // inside the panel: square block [cj+m, o+bb)^2, lower triangle
            if ((rc = syrk_run_device(rem, m, panel, lda, A + (cj + m) * lda + (cj + m), lda, -1.0, 1.0,
                                      SYRK_DTYPE_F64, st)) != SYRK_OK) return rc;
            // below the panel: rows [o+bb, N) x columns [cj+m, o+bb)
            const int64_t nb = N - (o + bb);
            if ((rc = gemm_nt(ds, nb, rem, m, A + (o + bb) * lda + cj, lda, panel, lda, A + (o + bb) * lda + (cj + m), lda,
                              -1.0, 1.0, st)) != SYRK_OK) return rc;
        }
        const int64_t nb = N - (o + bb);
        if (nb > 0) {                                             // the TBS step of Algorithm 5
            if ((rc = syrk_run_device(nb, bb, A + (o + bb) * lda + o, lda, A + (o + bb) * lda + (o + bb), lda, -1.0, 1.0,
                                      SYRK_DTYPE_F64, st)) != SYRK_OK) return rc;
        }
    }
    return SYRK_OK;
}

extern "C" int64_t cholesky_last_info(void* /*stream*/) {
    std::lock_guard<std::mutex> lock(runtime().mu);
    DeviceState* ds = nullptr;
    int rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    if (ds->device < 0 || ds->device >= 64 || !g_ws[ds->device].info) return 0;
    long long v = 0;
    if (cudaMemcpy(&v, g_ws[ds->device].info, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
    return int64_t(v);
}

namespace tbsyrk {
void release_cholesky_workspaces() {
    std::lock_guard<std::mutex> l2(g_chol_mu);
    for (CholWorkspace& ws : g_ws) {
        if (ws.w) cudaFree(ws.w);
        if (ws.t) cudaFree(ws.t);
        if (ws.info) cudaFree(ws.info);
        ws = CholWorkspace{};
    }
    cudaGetLastError();
}
}  // namespace tbsyrk
