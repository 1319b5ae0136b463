// Large Block Cholesky (Algorithm 5 of the paper, LBC) in FP64, lower triangle, in place.
//
// Right-looking blocked factorisation with block size b (default 512, 1024 from N = 16384 on).  For the panel of
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
constexpr int kNb = 32;                                         // inner block of the leaf
constexpr int kLs = kLeaf + 1;                                  // padded row pitch of the factor in shared memory
constexpr int kWs = kNb + 1;                                    // padded row pitch of a 32 x 32 block
constexpr int kLeafSmem = (kLeaf * kLs + 4 * kNb * kWs + kNb * kWs) * int(sizeof(double));

// Factor the m x m block at A (lower triangle, row pitch lda) in place and write the inverse
// of the factor, as a full 128 x 128 row-major matrix with zeros above the diagonal and
// beyond m, to W.  On a non-positive pivot k, *info <- pivot_base + k + 1 if it is still 0.
//
// Blocked right-looking Cholesky on 32 x 32 blocks, all in shared memory (rows beyond m are
// padded with the identity): one warp factors a diagonal block column by column (Algorithm 2)
// and inverts it; all 16 warps then solve the block rows below with that inverse and update
// the trailing blocks.  The inverse of the whole factor is assembled block by block,
// W[I][J] = -W[I][I] * sum_{K=J}^{I-1} L[I][K] * W[K][J], over the storage of L's off-diagonal
// blocks once L has been written back.
__global__ void __launch_bounds__(kLeafThreads)
chol_leaf_kernel(double* __restrict__ A, int64_t lda, int m, double* __restrict__ W,
                 long long* __restrict__ info, long long pivot_base) {
    extern __shared__ double leaf_smem[];
    double* Lf = leaf_smem;                                       // 128 x 129
    double* Wd = leaf_smem + kLeaf * kLs;                         // 4 diagonal inverses, 32 x 33 each
    double* Tb = Wd + 4 * kNb * kWs;                              // one 32 x 33 scratch block
    __shared__ int s_bad;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) s_bad = 0;
    for (int r = warp; r < kLeaf; r += kLeafThreads / 32)
        for (int c = lane; c < kLeaf; c += 32)
            Lf[r * kLs + c] = (r < m && c <= r) ? A[r * lda + c] : ((r == c) ? 1.0 : 0.0);
    __syncthreads();

    for (int J = 0; J < kLeaf / kNb; ++J) {
        const int j0 = J * kNb;
        double* Wj = Wd + J * kNb * kWs;
        if (warp == 0) {
            // ---- diagonal block in registers: lane r holds row r; values travel by shuffle ----
            double* D = Lf + j0 * kLs + j0;
            double row[kNb];
#pragma unroll
            for (int c = 0; c < kNb; ++c) row[c] = D[lane * kLs + c];
            bool bad = false;
#pragma unroll
            for (int k = 0; k < kNb; ++k) {                        // Algorithm 2 on the block
                const double p = __shfl_sync(0xffffffffu, row[k], k);
                if (!(p > 0.0)) {                                  // same value in every lane
                    if (!bad && lane == 0) {
                        atomicCAS(reinterpret_cast<unsigned long long*>(info), 0ull,
                                  static_cast<unsigned long long>(pivot_base + j0 + k + 1));
                        s_bad = 1;
                    }
                    bad = true;
                }
                const double d = sqrt(bad ? 1.0 : p);
                if (lane == k) row[k] = d;
                if (lane > k) row[k] = row[k] / d;
                const double l = row[k];                           // L[lane][k] for lane >= k
#pragma unroll
                for (int c = k + 1; c < kNb; ++c) {
                    const double lc = __shfl_sync(0xffffffffu, l, c);       // L[c][k]
                    if (lane >= c) row[c] -= l * lc;
                }
            }
#pragma unroll
            for (int c = 0; c < kNb; ++c)
                if (c <= lane) D[lane * kLs + c] = row[c];
            __syncwarp();
            // ---- its inverse: lane j holds column j, W[i][j] = (delta_ij - sum_k L[i][k] W[k][j]) / L[i][i];
            //      L[i][k] is read from shared memory (same address in every lane) ----
            if (!bad) {
                double w[kNb];
#pragma unroll
                for (int i = 0; i < kNb; ++i) {
                    double sacc = (i == lane) ? 1.0 : 0.0;
#pragma unroll
                    for (int k = 0; k < i; ++k)
                        if (k >= lane) sacc -= D[i * kLs + k] * w[k];
                    w[i] = (i >= lane) ? sacc / D[i * kLs + i] : 0.0;
                    Wj[i * kWs + lane] = w[i];
                }
            }
        }
        __syncthreads();
        if (s_bad) break;
        // ---- block rows below: X = P * W_JJ^T (each row belongs to one warp: read, then write) ----
        for (int r = j0 + kNb + warp; r < kLeaf; r += kLeafThreads / 32) {
            double acc = 0.0;
            for (int k = 0; k <= lane; ++k) acc += Lf[r * kLs + j0 + k] * Wj[lane * kWs + k];
            __syncwarp();
            Lf[r * kLs + j0 + lane] = acc;
        }
        __syncthreads();
        // ---- trailing update: L[r][c] -= sum_k X[r][k] X[c][k], c <= r ----
        for (int r = j0 + kNb + warp; r < kLeaf; r += kLeafThreads / 32) {
            for (int c = j0 + kNb + lane; c <= r; c += 32) {
                double acc = 0.0;
#pragma unroll 8
                for (int k = 0; k < kNb; ++k) acc += Lf[r * kLs + j0 + k] * Lf[c * kLs + j0 + k];
                Lf[r * kLs + c] -= acc;
            }
        }
        __syncthreads();
    }
    const bool bad = s_bad != 0;

    // ---- the factor goes back to A ----
    if (!bad)
        for (int r = warp; r < m; r += kLeafThreads / 32)
            for (int c = lane; c <= r; c += 32) A[r * lda + c] = Lf[r * kLs + c];

    // ---- off-diagonal blocks of the inverse, in the place of L's ----
    if (!bad) {
        for (int I = 1; I < kLeaf / kNb; ++I) {
            for (int J = 0; J < I; ++J) {
                // T = sum_{K=J}^{I-1} L[I][K] * W[K][J]; two elements per thread (rows tid/32 and +16)
                double t0 = 0.0, t1 = 0.0;
                const int r0 = warp, r1 = warp + 16;
                for (int K = J; K < I; ++K) {
                    const double* Lik = Lf + (I * kNb) * kLs + K * kNb;
                    const double* Wkj = (K == J) ? (Wd + J * kNb * kWs) : (Lf + (K * kNb) * kLs + J * kNb);
                    const int wp = (K == J) ? kWs : kLs;
#pragma unroll 8
                    for (int k = 0; k < kNb; ++k) {
                        const double w = Wkj[k * wp + lane];
                        t0 += Lik[r0 * kLs + k] * w;
                        t1 += Lik[r1 * kLs + k] * w;
                    }
                }
                Tb[r0 * kWs + lane] = t0;
                Tb[r1 * kWs + lane] = t1;
                __syncthreads();
                // W[I][J] = -W[I][I] * T
                const double* Wi = Wd + I * kNb * kWs;
                double o0 = 0.0, o1 = 0.0;
                for (int k = 0; k <= r1; ++k) {
                    const double tv = Tb[k * kWs + lane];
                    if (k <= r0) o0 -= Wi[r0 * kWs + k] * tv;
                    o1 -= Wi[r1 * kWs + k] * tv;
                }
                Lf[(I * kNb + r0) * kLs + J * kNb + lane] = o0;
                Lf[(I * kNb + r1) * kLs + J * kNb + lane] = o1;
                __syncthreads();
            }
        }
    }

    // ---- the inverse goes to W (zeros above the diagonal and beyond m) ----
    for (int r = warp; r < kLeaf; r += kLeafThreads / 32)
        for (int c = lane; c < kLeaf; c += 32) {
            double w = 0.0;
            if (!bad && r < m && c <= r)
                w = ((r / kNb) == (c / kNb)) ? Wd[(r / kNb) * kNb * kWs + (r % kNb) * kWs + (c % kNb)] : Lf[r * kLs + c];
            W[r * kLeaf + c] = w;
        }
}

struct CholWorkspace {
    double* w = nullptr;          // (block / 128) inverses, 128 x 128 each
    size_t w_bytes = 0;
    double* t = nullptr;          // N x 128 staging of a solved column block
    size_t t_bytes = 0;
    long long* info = nullptr;
    cudaStream_t panel_stream = nullptr;   // panel factorisations run here, ahead of the trailing update
    cudaEvent_t ev_panel = nullptr, ev_rest = nullptr;
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
    return launch_gemm_nt_f64(tp, tq, d_tma ? &td : nullptr, nrows, ncols, K, D, ldd, alpha, beta,
                              status_for_stream(ds, st), st) == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
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
    if (block == 0) block = (N >= 16384) ? 1024 : 512;
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
        if (!ws.panel_stream) {
            int lo = 0, hi = 0;
            cudaDeviceGetStreamPriorityRange(&lo, &hi);
            if (cudaStreamCreateWithPriority(&ws.panel_stream, cudaStreamNonBlocking, hi) != cudaSuccess ||
                cudaEventCreateWithFlags(&ws.ev_panel, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventCreateWithFlags(&ws.ev_rest, cudaEventDisableTiming) != cudaSuccess) {
                cudaGetLastError(); return SYRK_ERR_CUDA;
            }
        }
        static bool leaf_configured[64] = {};
        if (!leaf_configured[ds->device]) {
            if (cudaFuncSetAttribute(chol_leaf_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLeafSmem) != cudaSuccess) {
                cudaGetLastError(); return SYRK_ERR_CUDA;
            }
            leaf_configured[ds->device] = true;
        }
    }
    if (cudaMemsetAsync(ws.info, 0, sizeof(long long), st) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }

    // One panel of look-ahead: the trailing update of panel p is split into the columns of panel
    // p + 1 (done first, on the panel stream) and the rest (on the caller's stream); panel p + 1
    // is then factored on the panel stream while the rest of update p is still running.
    cudaStream_t sp = ws.panel_stream;
    cudaEvent_t ev_panel = ws.ev_panel, ev_rest = ws.ev_rest;
    auto chk = [](cudaError_t e) { if (e != cudaSuccess) { cudaGetLastError(); return false; } return true; };
    if (!chk(cudaEventRecord(ev_rest, st)) || !chk(cudaStreamWaitEvent(sp, ev_rest, 0))) return SYRK_ERR_CUDA;   // sp starts after the caller's prior work

    for (int64_t o = 0; o < N; o += block) {
        const int64_t bb = std::min<int64_t>(block, N - o);
        // ---- panel [o, o + bb) on the panel stream: factor, solve the rows below ----
        for (int64_t cj = o; cj < o + bb; cj += kLeaf) {
            const int m = int(std::min<int64_t>(kLeaf, o + bb - cj));
            double* Wj = ws.w + size_t((cj - o) / kLeaf) * kLeaf * kLeaf;
            chol_leaf_kernel<<<1, kLeafThreads, kLeafSmem, sp>>>(A + cj * lda + cj, lda, m, Wj, ws.info, cj);
            if (cudaGetLastError() != cudaSuccess) return SYRK_ERR_CUDA;
            const int64_t below = N - (cj + m);
            if (below <= 0) continue;
            double* panel = A + (cj + m) * lda + cj;              // rows below the leaf, its m columns
            // solve: panel <- panel * L_jj^-T  (through the staging buffer: the product is not in place)
            if ((rc = gemm_nt(ds, below, m, m, panel, lda, Wj, kLeaf, ws.t, kLeaf, 1.0, 0.0, sp)) != SYRK_OK) return rc;
            if (!chk(cudaMemcpy2DAsync(panel, size_t(lda) * 8, ws.t, size_t(kLeaf) * 8, size_t(m) * 8, size_t(below),
                                       cudaMemcpyDeviceToDevice, sp))) return SYRK_ERR_CUDA;
            const int64_t rem = o + bb - (cj + m);                // panel columns still to be updated
            if (rem <= 0) continue;
            // inside the panel: square block [cj+m, o+bb)^2, lower triangle
            if ((rc = syrk_run_device(rem, m, panel, lda, A + (cj + m) * lda + (cj + m), lda, -1.0, 1.0,
                                      SYRK_DTYPE_F64, sp)) != SYRK_OK) return rc;
            // below the panel: rows [o+bb, N) x columns [cj+m, o+bb)
            const int64_t nb = N - (o + bb);
            if ((rc = gemm_nt(ds, nb, rem, m, A + (o + bb) * lda + cj, lda, panel, lda, A + (o + bb) * lda + (cj + m), lda,
                              -1.0, 1.0, sp)) != SYRK_OK) return rc;
        }
        const int64_t o1 = o + bb, nb = N - o1;
        if (nb <= 0) break;
        // ---- trailing update A[I1,I1] -= A[I1,I0] A[I1,I0]^T (the TBS step of Algorithm 5), in two parts ----
        const double* P = A + o1 * lda + o;                       // A[I1, I0]: nb x bb
        const int64_t b1 = std::min<int64_t>(block, nb);          // width of the next panel
        // (a) columns of the next panel, on the panel stream: its diagonal block and the rows below it.
        //     They lie inside the region part (b) of the previous update wrote: wait for it.
        if (!chk(cudaStreamWaitEvent(sp, ev_rest, 0))) return SYRK_ERR_CUDA;
        if ((rc = syrk_run_device(b1, bb, P, lda, A + o1 * lda + o1, lda, -1.0, 1.0, SYRK_DTYPE_F64, sp)) != SYRK_OK) return rc;
        if ((rc = gemm_nt(ds, nb - b1, b1, bb, P + b1 * lda, lda, P, lda, A + (o1 + b1) * lda + o1, lda, -1.0, 1.0, sp)) != SYRK_OK) return rc;
        if (!chk(cudaEventRecord(ev_panel, sp))) return SYRK_ERR_CUDA;
        // (b) the rest, on the caller's stream, concurrently with the next panel's factorisation
        if (nb - b1 > 0) {
            if (!chk(cudaStreamWaitEvent(st, ev_panel, 0))) return SYRK_ERR_CUDA;
            // One block per item: the panel stream's blocks, of higher priority, then get the SMs
            // that this update's blocks free one by one; persistent blocks would hold every SM
            // until the update ends and the look-ahead would wait behind it.
            if ((rc = syrk_run_device(nb - b1, bb, P + b1 * lda, lda, A + (o1 + b1) * lda + (o1 + b1), lda, -1.0, 1.0,
                                      SYRK_DTYPE_F64, st, SYRK_F64_LAUNCH_PER_ITEM)) != SYRK_OK) return rc;
            if (!chk(cudaEventRecord(ev_rest, st))) return SYRK_ERR_CUDA;
        }
        // The next panel's factorisation (next iteration, panel stream) touches only the columns that
        // part (a) wrote, so it runs concurrently with part (b).
    }
    // the caller's stream continues after everything on the panel stream
    if (!chk(cudaEventRecord(ev_panel, sp)) || !chk(cudaStreamWaitEvent(st, ev_panel, 0))) return SYRK_ERR_CUDA;
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
        if (ws.panel_stream) cudaStreamDestroy(ws.panel_stream);
        if (ws.ev_panel) cudaEventDestroy(ws.ev_panel);
        if (ws.ev_rest) cudaEventDestroy(ws.ev_rest);
        ws = CholWorkspace{};
    }
    cudaGetLastError();
}
}  // namespace tbsyrk
