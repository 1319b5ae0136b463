// FP64 triangle-block SYRK kernel for sm_100a.
//
// One thread block per work item of the tiled TBS schedule (Algorithm 4 and
// Section 5.1.4 of the paper).  An item names up to 8 row segments of A (32 rows
// each) and up to 16 output tiles C[seg x, seg y]; for a triangle block the tiles
// are all pairs among k = 6 segments, so the block streams 6 segments per K-step
// where a square block of the same accumulator count streams 8.
//
//   producer warp : plain TMA tile loads (no multicast) of the item's segments,
//                   16 columns of A per stage, into a 6-stage shared-memory ring
//                   (128-byte swizzle), signalled through mbarriers;
//   16 MMA warps  : warp w owns tile w: a 32 x 32 accumulator held in registers as
//                   4 x 4 blocks of mma.sync m8n8k4 (FP64 tensor core, DMMA).  Each of the
//                   SM's four schedulers has its own DMMA pipe, so an item lasts as long as
//                   its busiest scheduler.  A triangle block has 15 tiles: its 15 warps then
//                   leave out their last 8 x 8 block and the 16th warp owns those 15 blocks -
//                   itself a triangle block over the last 8 rows of the six segments - so
//                   that every warp issues 15 DMMAs per k-slice instead of 16, 16, 16, 12;
//   epilogue      : alpha * acc (+ beta * C) written for entries with col <= row
//                   only, two doubles per store where alignment allows.  With beta != 0
//                   the producer also TMA-loads the item's old C tiles (those below the
//                   diagonal) into the ring's stages as the last K-steps release them, so
//                   the epilogue reads them from shared memory instead of waiting on HBM.
//
// Accumulators (the C block) stay on chip for the whole M loop and each entry of
// C is read (beta != 0) and written exactly once, as in the paper's generic
// out-of-core scheme (Algorithm 3).
#include "device_utils.cuh"
#include "kernels.h"
#include "tbs_plan.h"

namespace tbsyrk {
namespace f64 {

constexpr int kTile = 32;                       // b
constexpr int kBK = 16;                         // columns of A per stage (128 bytes)
constexpr int kStages = 6;
constexpr int kSegBytes = kTile * kBK * 8;      // 4096
constexpr int kStageBytes = kMaxSeg * kSegBytes;
constexpr int kMmaWarps = 16;
constexpr int kThreads = (kMmaWarps + 1) * 32;  // + producer warp
constexpr int kCTileBytes = kTile * kTile * 8;   // one old C tile in a ring stage (4 per stage)
constexpr int kSmemBytes = kStages * kStageBytes + 2 * kStages * 8 + 1024;

__device__ __forceinline__ void dmma884(double (&c)[2], double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c[0]), "+d"(c[1])
                 : "d"(a), "d"(b));
}

// The M loop of one warp's tile.  kSkipLast leaves out block (3, 3), which the 16th warp of
// a triangle block computes.  Returns false when a bounded wait ran out.
template <bool kSkipLast>
__device__ __forceinline__ bool tile_mainloop(double (&acc)[4][4][2], const uint8_t* smem, uint32_t xbase,
                                              uint32_t ybase, const uint32_t (&off)[4], int n_ksteps,
                                              uint64_t* full_bar, uint64_t* empty_bar, volatile int* abort_flag,
                                              int lane) {
    for (int ks = 0; ks < n_ksteps; ++ks) {
        const int st = ks % kStages;
        if (!mbar_wait_bounded(&full_bar[st], (ks / kStages) & 1, abort_flag)) return false;
        const uint8_t* px = smem + st * kStageBytes + xbase;
        const uint8_t* py = smem + st * kStageBytes + ybase;
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
            double a[4], b[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                a[j] = *reinterpret_cast<const double*>(px + off[sl] + j * 1024);
                b[j] = *reinterpret_cast<const double*>(py + off[sl] + j * 1024);
            }
#pragma unroll
            for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                for (int ni = 0; ni < 4; ++ni)
                    if (!(kSkipLast && mi == 3 && ni == 3)) dmma884(acc[mi][ni], a[mi], b[ni]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[st]);
    }
    return true;
}

__global__ void __launch_bounds__(kThreads, 1)
syrk_f64_tbs_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, const WorkItem* __restrict__ items, int64_t N,
                    int64_t ncols, int32_t gemm_col_tiles, int32_t n_ksteps, double* __restrict__ C,
                    int64_t ldc, double alpha, double beta, int vec_ok, int c_tma, int* __restrict__ status) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
    uint64_t* empty_bar = full_bar + kStages;
    __shared__ WorkItem s_item;
    __shared__ volatile int s_abort;
    __shared__ int s_scavenge;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    // Two-operand mode (gemm_col_tiles > 0): D = alpha * P * Q^T + beta * D without a triangle
    // mask; block b owns the 4 x 4 tile rectangle (b / column groups, b % column groups), its
    // column segments come from Q (tmB, the first `pad` segments), its row segments from P (tmA).
    const bool gemm = gemm_col_tiles > 0;
    if (gemm) {
        if (tid == 0) {
            const int n_cg = (gemm_col_tiles + 3) / 4;
            const int64_t row_tiles = (N + kTile - 1) / kTile;
            const int64_t rg = blockIdx.x / n_cg, cg = blockIdx.x % n_cg;
            const int nc = int(min(int64_t(4), int64_t(gemm_col_tiles) - cg * 4));
            const int nr = int(min(int64_t(4), row_tiles - rg * 4));
            for (int y = 0; y < nc; ++y) s_item.seg[y] = int32_t(cg * 4 + y);
            for (int x = 0; x < nr; ++x) s_item.seg[nc + x] = int32_t(rg * 4 + x);
            int tt = 0;
            for (int x = 0; x < nr; ++x)
                for (int y = 0; y < nc; ++y) { s_item.tile_x[tt] = uint8_t(nc + x); s_item.tile_y[tt] = uint8_t(y); ++tt; }
            s_item.n_seg = nc + nr; s_item.n_tile = tt; s_item.kind = kRect; s_item.pad = nc;
        }
    } else if (tid < int(sizeof(WorkItem) / 4)) {
        reinterpret_cast<int32_t*>(&s_item)[tid] = reinterpret_cast<const int32_t*>(&items[blockIdx.x])[tid];
    }
    if (tid == 0) s_abort = 0;
    __syncthreads();

    const int n_seg = s_item.n_seg, n_tile = s_item.n_tile;
    if (tid == 0) {
        bool ok = n_seg >= 1 && n_seg <= kMaxSeg && n_tile >= 1 && n_tile <= kMmaWarps;
        for (int s = 0; ok && s < n_seg; ++s)
            ok = s_item.seg[s] >= 0 && int64_t(s_item.seg[s]) * kTile < ((gemm && s < s_item.pad) ? ncols : N);
        for (int t = 0; ok && t < n_tile; ++t)
            ok = s_item.tile_x[t] < n_seg && s_item.tile_y[t] < n_seg;
        // A triangle block in the generator's tile order (x = 1..5, y < x): the 16th warp helps.
        bool tri = ok && s_item.kind == kTri && n_seg == 6 && n_tile == 15;
        for (int x = 1, t = 0; tri && x < 6; ++x)
            for (int y = 0; y < x; ++y, ++t) tri = tri && s_item.tile_x[t] == x && s_item.tile_y[t] == y;
        s_scavenge = tri ? 1 : 0;
        if (!ok) { s_abort = 1; atomicOr(status, kStatusBadItem); }
        else {
            for (int s = 0; s < kStages; ++s) {
                mbar_init(&full_bar[s], 1);
                mbar_init(&empty_bar[s], tri ? kMmaWarps : n_tile);
            }
            mbar_fence_init();
        }
    }
    __syncthreads();
    if (s_abort) return;

    if (warp == kMmaWarps) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            prefetch_tensormap(&tmA);
            int issued = 0;
            for (int ks = 0; ks < n_ksteps; ++ks) {
                const int st = ks % kStages;
                if (ks >= kStages &&
                    !mbar_wait_bounded(&empty_bar[st], ((ks / kStages) - 1) & 1, &s_abort)) {
                    s_abort = 1; atomicOr(status, kStatusWaitEmpty); break;
                }
                mbar_arrive_expect_tx(&full_bar[st], uint32_t(n_seg) * kSegBytes);
                uint8_t* dst = smem + st * kStageBytes;
                for (int s = 0; s < n_seg; ++s)
                    tma_load_2d(dst + s * kSegBytes, (gemm && s < s_item.pad) ? &tmB : &tmA, ks * kBK,
                                s_item.seg[s] * kTile, &full_bar[st]);
                issued = ks + 1;
            }
            if (c_tma && !s_abort) {
                // Old C: ring step n_ksteps + j carries tiles 4j .. 4j+3 (8 KB each, row pitch 256 B).
                prefetch_tensormap(&tmC);
                for (int j = 0; 4 * j < n_tile; ++j) {
                    const int q = n_ksteps + j, st = q % kStages;
                    if (q >= kStages && !mbar_wait_bounded(&empty_bar[st], ((q / kStages) - 1) & 1, &s_abort)) {
                        s_abort = 1; atomicOr(status, kStatusWaitEmpty); break;
                    }
                    int below = 0;
                    for (int tt = 4 * j; tt < n_tile && tt < 4 * j + 4; ++tt)
                        below += (gemm || s_item.seg[s_item.tile_x[tt]] != s_item.seg[s_item.tile_y[tt]]) ? 1 : 0;
                    if (below == 0) { mbar_arrive(&full_bar[st]); continue; }
                    mbar_arrive_expect_tx(&full_bar[st], uint32_t(below) * kCTileBytes);
                    uint8_t* dst = smem + st * kStageBytes;
                    for (int tt = 4 * j; tt < n_tile && tt < 4 * j + 4; ++tt) {
                        const int rx = s_item.seg[s_item.tile_x[tt]], cy = s_item.seg[s_item.tile_y[tt]];
                        if (gemm || rx != cy) tma_load_2d(dst + (tt & 3) * kCTileBytes, &tmC, cy * kTile, rx * kTile, &full_bar[st]);
                    }
                    issued = q + 1;
                }
            }
            if (s_abort) {
                // Winding down: let the copies still in flight land before the block exits.
                for (int ks = (issued > kStages ? issued - kStages : 0); ks < issued; ++ks) {
                    volatile int dummy = 0;
                    mbar_wait_bounded(&full_bar[ks % kStages], (ks / kStages) & 1, &dummy);
                }
            }
        }
        return;
    }
    const bool scavenge = s_scavenge != 0;
    if (warp >= n_tile && !scavenge) return;

    // ------------------------------ MMA warps ------------------------------
    // Fragment addressing.  Lane (g, t) of an m8n8k4 fragment holds (row g, k = t).  The four
    // k-slices of a stage take k = 8*(t>>1) + 2*sl + (t&1): any assignment of the stage's 16
    // columns to (slice, t) is valid as long as both operands use the same one, and this one
    // makes every half-warp's 16 loads hit 16 different 8-byte bank pairs under the 128-byte
    // swizzle (16-byte chunk index ^ row % 8).
    const int g = lane >> 2, t = lane & 3;
    uint32_t off[4];
#pragma unroll
    for (int sl = 0; sl < 4; ++sl)
        off[sl] = uint32_t(g * 128 + ((((t >> 1) << 2 | sl) ^ g) << 4) + ((t & 1) << 3));
    const bool use_beta = (beta != 0.0);

    if (scavenge && warp == kMmaWarps - 1) {
        // ------------- 16th warp of a triangle block: the 15 left-out 8 x 8 blocks -------------
        double sacc[15][2];
#pragma unroll
        for (int q = 0; q < 15; ++q) sacc[q][0] = sacc[q][1] = 0.0;
        for (int ks = 0; ks < n_ksteps; ++ks) {
            const int st = ks % kStages;
            if (!mbar_wait_bounded(&full_bar[st], (ks / kStages) & 1, &s_abort)) {
                s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitFull); return;
            }
            const uint8_t* base = smem + st * kStageBytes + 3 * 1024;      // rows 24..31 of every segment
#pragma unroll
            for (int sl = 0; sl < 4; ++sl) {
                double f[6];
#pragma unroll
                for (int s = 0; s < 6; ++s) f[s] = *reinterpret_cast<const double*>(base + s * kSegBytes + off[sl]);
                int q = 0;
#pragma unroll
                for (int x = 1; x < 6; ++x)
#pragma unroll
                    for (int y = 0; y < x; ++y, ++q) dmma884(sacc[q], f[x], f[y]);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty_bar[st]);
        }
        if (c_tma) {                                                    // all four old-C ring steps
            for (int j = 0; j < 4; ++j) {
                const int qs = n_ksteps + j;
                if (!mbar_wait_bounded(&full_bar[qs % kStages], (qs / kStages) & 1, &s_abort)) {
                    s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitFull); return;
                }
            }
        }
        int q = 0;
#pragma unroll
        for (int x = 1; x < 6; ++x)
#pragma unroll
            for (int y = 0; y < x; ++y, ++q) {
                const int64_t r = int64_t(s_item.seg[x]) * kTile + 24 + g;
                const int64_t c = int64_t(s_item.seg[y]) * kTile + 24 + 2 * t;
                if (r >= N) continue;                                   // tile below the diagonal: c + 1 < r
                double* p = C + r * ldc + c;
                double v0 = alpha * sacc[q][0], v1 = alpha * sacc[q][1];
                if (c_tma) {
                    const double2 o = *reinterpret_cast<const double2*>(
                        smem + ((n_ksteps + (q >> 2)) % kStages) * kStageBytes + (q & 3) * kCTileBytes +
                        (24 + g) * (kTile * 8) + (24 + 2 * t) * 8);
                    v0 += beta * o.x; v1 += beta * o.y;
                } else if (use_beta) { v0 += beta * p[0]; v1 += beta * p[1]; }
                if (vec_ok) *reinterpret_cast<double2*>(p) = make_double2(v0, v1);
                else { p[0] = v0; p[1] = v1; }
            }
        return;
    }

    const int sx = s_item.tile_x[warp], sy = s_item.tile_y[warp];
    const uint32_t xbase = uint32_t(sx) * kSegBytes, ybase = uint32_t(sy) * kSegBytes;

    double acc[4][4][2];
#pragma unroll
    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) acc[mi][ni][0] = acc[mi][ni][1] = 0.0;

    const bool alive = scavenge
        ? tile_mainloop<true>(acc, smem, xbase, ybase, off, n_ksteps, full_bar, empty_bar, &s_abort, lane)
        : tile_mainloop<false>(acc, smem, xbase, ybase, off, n_ksteps, full_bar, empty_bar, &s_abort, lane);
    if (!alive) { s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitFull); return; }

    // ------------------------------ epilogue ------------------------------
    const int64_t row0 = int64_t(s_item.seg[sx]) * kTile, col0 = int64_t(s_item.seg[sy]) * kTile;
    const uint8_t* old_tile = nullptr;                  // this warp's old C tile in shared memory
    if (c_tma && (gemm || row0 != col0)) {
        const int qs = n_ksteps + (warp >> 2);
        if (!mbar_wait_bounded(&full_bar[qs % kStages], (qs / kStages) & 1, &s_abort)) {
            s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitFull); return;
        }
        old_tile = smem + (qs % kStages) * kStageBytes + (warp & 3) * kCTileBytes;
    }
#pragma unroll
    for (int mi = 0; mi < 4; ++mi) {
        const int64_t r = row0 + mi * 8 + g;
        if (r >= N) continue;
        const int64_t cmax = gemm ? ncols - 1 : r;      // last column this row may touch
        double* crow = C + r * ldc;
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
            if (scavenge && mi == 3 && ni == 3) continue;             // written by the 16th warp
            const int64_t c = col0 + ni * 8 + 2 * t;
            if (c > cmax) continue;
            const bool both = (c + 1 <= cmax);
            double v0 = alpha * acc[mi][ni][0], v1 = alpha * acc[mi][ni][1];
            if (use_beta) {
                double2 o = make_double2(0.0, 0.0);
                if (old_tile) o = *reinterpret_cast<const double2*>(old_tile + (mi * 8 + g) * (kTile * 8) + (ni * 8 + 2 * t) * 8);
                else if (both && vec_ok) o = *reinterpret_cast<const double2*>(crow + c);
                else { o.x = crow[c]; if (both) o.y = crow[c + 1]; }
                v0 += beta * o.x; v1 += beta * o.y;
            }
            if (both) {
                if (vec_ok) *reinterpret_cast<double2*>(crow + c) = make_double2(v0, v1);
                else { crow[c] = v0; crow[c + 1] = v1; }
            } else {
                crow[c] = v0;
            }
        }
    }
}

}  // namespace f64

namespace {
cudaError_t configure_f64_kernel() {
    // The shared-memory attribute belongs to a device's context: set it once per device.
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(f64::syrk_f64_tbs_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, f64::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    return cudaSuccess;
}
}  // namespace

cudaError_t launch_syrk_f64(const CUtensorMap& tmA, const CUtensorMap* tmC, const WorkItem* d_items,
                            int64_t n_items, int64_t N, int64_t M, double* C, int64_t ldc, double alpha,
                            double beta, int* d_status, cudaStream_t stream) {
    cudaError_t e = configure_f64_kernel();
    if (e != cudaSuccess) return e;
    if (n_items == 0) return cudaSuccess;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 1) == 0) ? 1 : 0;
    const int32_t n_ksteps = int32_t((M + f64::kBK - 1) / f64::kBK);
    const int c_tma = (tmC != nullptr && beta != 0.0 && vec_ok) ? 1 : 0;
    CUtensorMap none{};
    f64::syrk_f64_tbs_kernel<<<dim3(unsigned(n_items)), dim3(f64::kThreads), f64::kSmemBytes, stream>>>(
        tmA, tmA, c_tma ? *tmC : none, d_items, N, N, 0, n_ksteps, C, ldc, alpha, beta, vec_ok, c_tma, d_status);
    return cudaGetLastError();
}

cudaError_t launch_gemm_nt_f64(const CUtensorMap& tmP, const CUtensorMap& tmQ, const CUtensorMap* tmD,
                               int64_t nrows, int64_t ncols, int64_t K, double* D, int64_t ldd, double alpha,
                               double beta, int* d_status, cudaStream_t stream) {
    cudaError_t e = configure_f64_kernel();
    if (e != cudaSuccess) return e;
    if (nrows == 0 || ncols == 0) return cudaSuccess;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(D) & 15) == 0 && (ldd & 1) == 0) ? 1 : 0;
    const int32_t n_ksteps = int32_t((K + f64::kBK - 1) / f64::kBK);
    const int c_tma = (tmD != nullptr && beta != 0.0 && vec_ok) ? 1 : 0;
    const int64_t row_tiles = (nrows + f64::kTile - 1) / f64::kTile, col_tiles = (ncols + f64::kTile - 1) / f64::kTile;
    const int64_t blocks = ((row_tiles + 3) / 4) * ((col_tiles + 3) / 4);
    CUtensorMap none{};
    f64::syrk_f64_tbs_kernel<<<dim3(unsigned(blocks)), dim3(f64::kThreads), f64::kSmemBytes, stream>>>(
        tmP, tmQ, c_tma ? *tmD : none, nullptr, nrows, ncols, int32_t(col_tiles), n_ksteps, D, ldd, alpha, beta,
        vec_ok, c_tma, d_status);
    return cudaGetLastError();
}

int f64_tile() { return f64::kTile; }
int f64_bk() { return f64::kBK; }
int f64_stages() { return f64::kStages; }

}  // namespace tbsyrk
