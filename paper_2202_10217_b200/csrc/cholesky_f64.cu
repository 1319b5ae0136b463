// Large Block Cholesky (Algorithm 5 of the paper, LBC) in FP64, lower triangle, in place.
//
// Right-looking blocked factorisation with block size b (default 512, 1024 from N = 16384 on).  For the panel of
// columns I0 = [o, o + b):
//   1. A[I0, I0] <- its Cholesky factor                      (the paper's OOC_CHOL step)
//   2. A[I1, I0] <- A[I1, I0] * L00^-T, I1 = [o + b, N)      (the paper's OOC_TRSM step)
//   3. A[I1, I1] <- A[I1, I1] - A[I1, I0] * A[I1, I0]^T      (TBS: syrk_lower with alpha = -1,
//                                                             beta = 1, K = b, trailing view)
// Steps 1 and 2 are only cited by the paper; here they run in 128-column sub-steps.  A leaf
// kernel (one thread block) factors a 128 x 128 diagonal block in shared memory; the rows below
// are solved against it by blocked forward substitution (64 rows per thread block, in place) and
// the rest of the panel is updated by a small SYRK (inside the panel) and a product (below it,
// FP64 tensor-core kernel in two-operand mode).  No triangular factor is inverted anywhere.
// Step 3 is the library's triangle-block SYRK.
#include <algorithm>
#include <mutex>

#include "../../include/tbsyrk.h"
#include "kernels.h"
#include "runtime.h"

namespace tbsyrk {
namespace {

constexpr int kLeaf = 128;
constexpr int kLeafThreads = 512;
constexpr int kNb = 32;                                         // inner block of the leaf and of the row solve
constexpr int kLs = kLeaf + 1;                                  // padded row pitch of a 128-column block in shared memory
constexpr int kLeafSmem = kLeaf * kLs * int(sizeof(double));

// Algorithm 2 of the paper on one 32 x 32 diagonal block D (row pitch kLs, shared memory) by one warp: lane r
// holds row r in registers and values travel by shuffle.  A non-positive pivot k sets *info (if still 0) to
// pivot_base + k + 1 and *bad_flag.  Kept out of line so that the row stays in registers (inlined into the
// leaf kernel the compiler left it in local memory, which made the leaf three times slower).
__device__ __noinline__ void factor_diag_block(double* D, int lane, long long* info, long long pivot_base, int* bad_flag) {
    double row[kNb];
#pragma unroll
    for (int c = 0; c < kNb; ++c) row[c] = D[lane * kLs + c];
    bool bad = false;
#pragma unroll
    for (int k = 0; k < kNb; ++k) {
        const double p = __shfl_sync(0xffffffffu, row[k], k);
        if (!(p > 0.0)) {                                  // same value in every lane
            if (!bad && lane == 0) {
                atomicCAS(reinterpret_cast<unsigned long long*>(info), 0ull,
                          static_cast<unsigned long long>(pivot_base + k + 1));
                *bad_flag = 1;
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
}

// Factor the m x m block at A (lower triangle, row pitch lda) in place.  On a non-positive pivot k,
// *info <- pivot_base + k + 1 if it is still 0, and A is left as it was.
//
// Blocked right-looking Cholesky on 32 x 32 blocks, all in shared memory (rows beyond m are padded with
// the identity): one warp factors a diagonal block column by column (Algorithm 2 of the paper on the
// block, a row per lane, values travelling by shuffle); all 16 warps then solve the block rows below by
// forward substitution against that block (x L_JJ^T = p, one row per warp and pass: lane c divides, the
// lanes after it subtract) and update the trailing blocks.  Nothing is inverted.
__global__ void __launch_bounds__(kLeafThreads)
chol_leaf_kernel(double* __restrict__ A, int64_t lda, int m, long long* __restrict__ info, long long pivot_base) {
    extern __shared__ double leaf_smem[];
    double* Lf = leaf_smem;                                       // 128 x 129
    __shared__ int s_bad;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) s_bad = 0;
    for (int r = warp; r < kLeaf; r += kLeafThreads / 32)
        for (int c = lane; c < kLeaf; c += 32)
            Lf[r * kLs + c] = (r < m && c <= r) ? A[r * lda + c] : ((r == c) ? 1.0 : 0.0);
    __syncthreads();

    for (int J = 0; J < kLeaf / kNb; ++J) {
        const int j0 = J * kNb;
        if (warp == 0) factor_diag_block(Lf + j0 * kLs + j0, lane, info, pivot_base + j0, &s_bad);
        __syncthreads();
        if (s_bad) break;
        // ---- block rows below: x L_JJ^T = p by forward substitution; lane c holds entry c of the row and
        //      the reciprocal of L_JJ[c][c] (one division per pivot instead of one per row and pivot) ----
        const double rdiag = 1.0 / Lf[(j0 + lane) * kLs + j0 + lane];
        for (int r = j0 + kNb + warp; r < kLeaf; r += kLeafThreads / 32) {
            double p = Lf[r * kLs + j0 + lane];
#pragma unroll 4
            for (int c = 0; c < kNb; ++c) {
                if (lane == c) p = p * rdiag;
                const double x = __shfl_sync(0xffffffffu, p, c);
                if (lane > c) p -= x * Lf[(j0 + lane) * kLs + j0 + c];          // L_JJ[lane][c]
            }
            Lf[r * kLs + j0 + lane] = p;
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
    // ---- the factor goes back to A ----
    if (!s_bad)
        for (int r = warp; r < m; r += kLeafThreads / 32)
            for (int c = lane; c <= r; c += 32) A[r * lda + c] = Lf[r * kLs + c];
}

// Rows below a factored leaf: P <- P L^-T for the n_rows x m block P (row pitch ldp), L the m x m lower
// triangular factor at `L` (row pitch ldl), m <= 128 - the paper's OOC_TRSM step for one 128-column
// sub-step, by blocked forward substitution (nothing is inverted, so the backward error does not depend on
// the condition of L's diagonal blocks).  A thread block holds L and 64 rows of P in shared memory; per
// 32-column block J: (a) x_J L_JJ^T = p_J row by row, a thread per row with the row in registers (L_JJ
// is read by every lane at the same address; its diagonal enters as reciprocals), then (b) the blocks to its right lose x_J L_KJ^T, every warp
// taking a share of the columns (two rows per lane, the L values again broadcast).
constexpr int kTrsmRows = 64;
constexpr int kTrsmThreads = 256;
constexpr int kTrsmSmem = (kLeaf * kLs + kTrsmRows * kLs) * int(sizeof(double));

template <int kCols>    // columns of the update a warp takes: 12, 8 or 4 (96, 64 or 32 columns over 8 warps)
__device__ __forceinline__ void trsm_update(const double* __restrict__ Ls, double* __restrict__ Xs, int j0, int warp, int lane) {
    const int c0 = j0 + kNb + warp * kCols;                       // this warp's first column
    double acc[2][kCols];
#pragma unroll
    for (int e = 0; e < kCols; ++e) acc[0][e] = acc[1][e] = 0.0;
#pragma unroll 4
    for (int k = 0; k < kNb; ++k) {
        const double x0 = Xs[lane * kLs + j0 + k], x1 = Xs[(lane + 32) * kLs + j0 + k];
#pragma unroll
        for (int e = 0; e < kCols; ++e) {
            const double l = Ls[(c0 + e) * kLs + j0 + k];          // same address in every lane
            acc[0][e] += x0 * l;
            acc[1][e] += x1 * l;
        }
    }
#pragma unroll
    for (int e = 0; e < kCols; ++e) {
        Xs[lane * kLs + c0 + e] -= acc[0][e];
        Xs[(lane + 32) * kLs + c0 + e] -= acc[1][e];
    }
}

__global__ void __launch_bounds__(kTrsmThreads)
trsm_rows_kernel(const double* __restrict__ L, int64_t ldl, int m, double* __restrict__ P, int64_t ldp, int64_t n_rows) {
    extern __shared__ double trsm_smem[];
    double* Ls = trsm_smem;                                        // 128 x 129: lower triangle of L, identity beyond m
    double* Xs = trsm_smem + kLeaf * kLs;                          // 64 x 129: this block's rows of P
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int64_t row0 = int64_t(blockIdx.x) * kTrsmRows;
    for (int r = warp; r < kLeaf; r += kTrsmThreads / 32)
        for (int c = lane; c < kLeaf; c += 32)
            Ls[r * kLs + c] = (r < m && c <= r) ? L[r * ldl + c] : ((r == c) ? 1.0 : 0.0);
    for (int r = warp; r < kTrsmRows; r += kTrsmThreads / 32)
        for (int c = lane; c < kLeaf; c += 32)
            Xs[r * kLs + c] = (row0 + r < n_rows && c < m) ? P[(row0 + r) * ldp + c] : 0.0;
    __syncthreads();
    // The diagonal of L is replaced by its reciprocals (one division per pivot for the whole block); the
    // padding column of each row of Ls is free for that.
    if (tid < kLeaf) Ls[tid * kLs + kLeaf] = 1.0 / Ls[tid * kLs + tid];
    __syncthreads();
    for (int J = 0; J < kLeaf / kNb; ++J) {
        const int j0 = J * kNb;
        if (tid < kTrsmRows) {                                     // (a) a row per thread
            double p[kNb];
#pragma unroll
            for (int c = 0; c < kNb; ++c) p[c] = Xs[tid * kLs + j0 + c];
#pragma unroll
            for (int c = 0; c < kNb; ++c) {
                p[c] = p[c] * Ls[(j0 + c) * kLs + kLeaf];
#pragma unroll
                for (int d = c + 1; d < kNb; ++d) p[d] -= p[c] * Ls[(j0 + d) * kLs + j0 + c];
            }
#pragma unroll
            for (int c = 0; c < kNb; ++c) Xs[tid * kLs + j0 + c] = p[c];
        }
        __syncthreads();
        if (J == 0) trsm_update<12>(Ls, Xs, j0, warp, lane);       // (b)
        else if (J == 1) trsm_update<8>(Ls, Xs, j0, warp, lane);
        else if (J == 2) trsm_update<4>(Ls, Xs, j0, warp, lane);
        __syncthreads();
    }
    for (int r = warp; r < kTrsmRows; r += kTrsmThreads / 32)
        for (int c = lane; c < m; c += 32)
            if (row0 + r < n_rows) P[(row0 + r) * ldp + c] = Xs[r * kLs + c];
}

struct CholWorkspace {
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
            if (cudaFuncSetAttribute(chol_leaf_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kLeafSmem) != cudaSuccess ||
                cudaFuncSetAttribute(trsm_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTrsmSmem) != cudaSuccess) {
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
            chol_leaf_kernel<<<1, kLeafThreads, kLeafSmem, sp>>>(A + cj * lda + cj, lda, m, ws.info, cj);
            if (cudaGetLastError() != cudaSuccess) return SYRK_ERR_CUDA;
            const int64_t below = N - (cj + m);
            if (below <= 0) continue;
            double* panel = A + (cj + m) * lda + cj;              // rows below the leaf, its m columns
            // solve in place: panel <- panel * L_jj^-T by forward substitution
            trsm_rows_kernel<<<unsigned((below + kTrsmRows - 1) / kTrsmRows), kTrsmThreads, kTrsmSmem, sp>>>(
                A + cj * lda + cj, lda, m, panel, lda, below);
            if (cudaGetLastError() != cudaSuccess) return SYRK_ERR_CUDA;
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
        if (ws.info) cudaFree(ws.info);
        if (ws.panel_stream) cudaStreamDestroy(ws.panel_stream);
        if (ws.ev_panel) cudaEventDestroy(ws.ev_panel);
        if (ws.ev_rest) cudaEventDestroy(ws.ev_rest);
        ws = CholWorkspace{};
    }
    cudaGetLastError();
}
}  // namespace tbsyrk
