// FP64 triangle-block SYRK kernels for sm_100a.
//
// Work items of the tiled TBS schedule (Algorithm 4 and Section 5.1.4 of the paper) are run
// by thread blocks of 16 MMA warps and one producer warp.  An item names up to 8 row
// segments of A (32 rows each) and up to 16 output tiles C[seg x, seg y]; for a triangle
// block the tiles are all pairs among k = 6 segments, so the block streams 6 segments per
// K-step where a square block of the same accumulator count streams 8.
//
//   producer warp : plain TMA tile loads (no multicast) of the item's segments,
//                   16 columns of A per stage, into a shared-memory ring of stages
//                   (128-byte swizzle; six stages, three in the persistent form), signalled through mbarriers;
//   16 MMA warps  : warp w owns tile w: a 32 x 32 accumulator held in registers as
//                   4 x 4 blocks of mma.sync m8n8k4 (FP64 tensor core, DMMA).  Each of the
//                   SM's four schedulers has its own DMMA pipe, so an item lasts as long as
//                   its busiest scheduler.  A triangle block has 15 tiles: its 15 warps then
//                   leave out their last 8 x 8 block and the 16th warp owns those 15 blocks -
//                   itself a triangle block over the last 8 rows of the six segments - so
//                   that every warp issues 15 DMMAs per k-slice instead of 16, 16, 16, 12;
//   epilogue      : (one block per item) alpha * acc (+ beta * C) written for entries with col <= row
//                   only, two doubles per store where alignment allows.  With beta != 0
//                   the producer also TMA-loads the item's old C tiles (those below the
//                   diagonal) into the ring's stages as the last K-steps release them, so
//                   the epilogue reads them from shared memory instead of waiting on HBM.
//
// Two launch forms share this code.  One block per item (the hardware block scheduler hands
// out the items; used for short lists and for the two-operand mode), and a persistent form,
// one block per SM, whose producer draws the next item from a global counter and publishes
// it to the MMA warps through a small ring in shared memory: the ring of stages then runs on
// across items.  In the persistent form the MMA warps do not write C themselves: they leave their
// accumulators in a shared-memory image and three more warps write it out while the next item's M loop
// runs.  The same two forms serve the rank-2k and the Hermitian updates (two warps per tile) and strided batches.
//
// Accumulators (the C block) stay on chip for the whole M loop and each entry of
// C is read (beta != 0) and written exactly once, as in the paper's generic
// out-of-core scheme (Algorithm 3).
#include <mutex>

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
constexpr int kCTileBytes = kTile * kTile * 8;  // one old C tile in a ring stage (4 per stage)
constexpr int kSmemBytes = kStages * kStageBytes + 2 * kStages * 8 + 1024;
constexpr int kItemRing = 16;                   // published items in flight (persistent form)
constexpr int kSyr2kSlots = kMaxSeg / 2;        // rank-2k update: segments of A in slots 0..3, of B in slots 4..7

__device__ __forceinline__ void dmma884(double (&c)[2], double a, double b) {
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c[0]), "+d"(c[1])
                 : "d"(a), "d"(b));
}

// The write-out arithmetic, alpha * acc + beta * old, in one fixed rounding sequence - the product alpha * acc
// rounded, then one fused multiply-add - so that every role and both launch forms give the same bits whatever
// the compiler would contract.  (With beta == 1 the second step is the correctly rounded sum.)
__device__ __forceinline__ double scaled(double alpha, double acc) { return __dmul_rn(alpha, acc); }
__device__ __forceinline__ double plus_old(double v, double beta, double old) { return __fma_rn(beta, old, v); }

// What every role of a block needs to know about the call.
struct Call {
    uint8_t* smem;                 // the ring of stages
    uint32_t smem32, bars32;       // shared-space addresses of the ring and of full_bar[0] (MMA warps use these)
    uint32_t empties32;            // ... and of empty_bar[0]
    uint64_t* full_bar;
    uint64_t* empty_bar;           // 16 arrivals (one per MMA warp) free a stage
    volatile int* abort_flag;
    int* status;
    const CUtensorMap* tmA;        // row segments
    const CUtensorMap* tmB;        // column segments of the two-operand mode (else == tmA)
    const CUtensorMap* tmC;        // old C tiles (c_tma)
    int64_t N, ncols;
    int32_t n_ksteps;
    double* C;
    int64_t ldc;
    double alpha, beta;
    int vec_ok, c_tma;
    int32_t batch;                 // matrix of a strided batch the block works on (tensor maps are 3-D), or -1
    int32_t k0;                    // first K-step of the block's slice of the inner dimension (K-split calls)
    bool syr2k;                    // rank-2k update: slots 0..3 hold segments of A, slots 4..7 the same rows of B (tmB)
    bool herk;                     // Hermitian update: A is the real view (re, im interleaved) of a complex operand, C complex
    bool gemm;
};
// Tail K-split units: bit 1 of Call::vec_ok is set and Call::C points at the unit's partial tiles (16 slots
// of 32 x 32, slot q at q * 1024) instead of at the result matrix.
constexpr int kVecOkPartial = 2;
constexpr int kPartTileElems = kTile * kTile;            // 1024 doubles per partial tile
constexpr int kPartUnitElems = kMmaWarps * kPartTileElems; // one unit: a slot per MMA warp

// Ring steps of one item: its K-steps, then (c_tma) one step per group of four tiles of old C.
__device__ __forceinline__ int c_steps_of(const Call& k, int n_tile) { return k.c_tma ? (n_tile + 3) / 4 : 0; }

// ---------------------------------------------------------------------------------------------
// Producer (one thread): fetch one item's ring steps, starting at global step g.
// ---------------------------------------------------------------------------------------------
template <bool kTN, int kSt = kStages>
__device__ __forceinline__ bool produce_item(const Call& k, const WorkItem& it, uint32_t& g) {
    const int n_seg = it.n_seg, n_tile = it.n_tile;
    for (int ks = 0; ks < k.n_ksteps; ++ks, ++g) {
        const uint32_t st = g % kSt;
        if (g >= kSt && !mbar_wait_bounded(&k.empty_bar[st], ((g / kSt) - 1) & 1, k.abort_flag)) {
            *k.abort_flag = 1; atomicOr(k.status, kStatusWaitEmpty); return false;
        }
        mbar_arrive_expect_tx(&k.full_bar[st], uint32_t(k.syr2k ? 2 * n_seg : n_seg) * kSegBytes);
        uint8_t* dst = k.smem + st * kStageBytes;
        if (k.syr2k) {
            for (int s = 0; s < n_seg; ++s) {
                tma_load_2d(dst + s * kSegBytes, k.tmA, (k.k0 + ks) * kBK, it.seg[s] * kTile, &k.full_bar[st]);
                tma_load_2d(dst + (kSyr2kSlots + s) * kSegBytes, k.tmB, (k.k0 + ks) * kBK, it.seg[s] * kTile, &k.full_bar[st]);
            }
        } else if (kTN) {
            // A stored M x N: a segment's 32 columns x 16 rows of A arrive as two boxes of 16 x 16
            // (128-byte rows of 16 columns, one row per k), 2 KB each.
            for (int s = 0; s < n_seg; ++s)
                for (int h = 0; h < 2; ++h)
                    tma_load_box(dst + s * kSegBytes + h * (kSegBytes / 2), k.tmA, it.seg[s] * kTile + h * 16,
                                 (k.k0 + ks) * kBK, k.batch, &k.full_bar[st]);
        } else {
            for (int s = 0; s < n_seg; ++s)
                tma_load_box(dst + s * kSegBytes, (k.gemm && s < it.pad) ? k.tmB : k.tmA, (k.k0 + ks) * kBK,
                             it.seg[s] * kTile, k.batch, &k.full_bar[st]);
        }
    }
    // Old C: ring step j carries tiles 4j .. 4j+3 (8 KB each, row pitch 256 B), those below the diagonal.
    const int n_c = c_steps_of(k, n_tile);
    for (int j = 0; j < n_c; ++j, ++g) {
        const uint32_t st = g % kSt;
        if (g >= kSt && !mbar_wait_bounded(&k.empty_bar[st], ((g / kSt) - 1) & 1, k.abort_flag)) {
            *k.abort_flag = 1; atomicOr(k.status, kStatusWaitEmpty); return false;
        }
        int below = 0;
        for (int tt = 4 * j; tt < n_tile && tt < 4 * j + 4; ++tt)
            below += (k.gemm || it.seg[it.tile_x[tt]] != it.seg[it.tile_y[tt]]) ? 1 : 0;
        if (below == 0) { mbar_arrive(&k.full_bar[st]); continue; }
        mbar_arrive_expect_tx(&k.full_bar[st], uint32_t(below) * kCTileBytes);
        uint8_t* dst = k.smem + st * kStageBytes;
        for (int tt = 4 * j; tt < n_tile && tt < 4 * j + 4; ++tt) {
            const int rx = it.seg[it.tile_x[tt]], cy = it.seg[it.tile_y[tt]];
            if (k.gemm || rx != cy)
                tma_load_box(dst + (tt & 3) * kCTileBytes, k.tmC, cy * kTile, rx * kTile, k.batch, &k.full_bar[st]);
        }
    }
    return true;
}

// After a give-up: let the copies still in flight land before the block exits.
template <int kSt = kStages>
__device__ void drain_producer(const Call& k, uint32_t g) {
    for (uint32_t i = (g > kSt ? g - kSt : 0); i < g; ++i) {
        volatile int dummy = 0;
        mbar_wait_bounded(&k.full_bar[i % kSt], (i / kSt) & 1, &dummy);
    }
}

// Checks an item before any role uses it and, outside the two-operand mode, records in `pad`
// whether it is a triangle block in the generator's tile order (x = 1..5, y < x): for those
// the 16th MMA warp takes the last 8 x 8 block of every tile.  (One thread decides this once per
// item; the MMA warps only read the flag.)
__device__ bool prepare_item(const Call& k, WorkItem& it, bool upper = false) {
    bool ok = it.n_seg >= 1 && it.n_seg <= kMaxSeg && it.n_tile >= 1 && it.n_tile <= kMmaWarps;
    if (k.syr2k) ok = ok && it.n_seg <= kSyr2kSlots && it.n_tile <= kMmaWarps / 2;
    if (k.herk) ok = ok && it.n_tile <= kMmaWarps / 2;
    for (int s = 0; ok && s < it.n_seg; ++s)
        ok = it.seg[s] >= 0 && int64_t(it.seg[s]) * kTile < ((k.gemm && s < it.pad) ? k.ncols : k.N);
    for (int t = 0; ok && t < it.n_tile; ++t) ok = it.tile_x[t] < it.n_seg && it.tile_y[t] < it.n_seg;
    if (ok && !k.gemm) {
        bool tri = !k.syr2k && !k.herk && it.kind == kTri && it.n_seg == 6 && it.n_tile == 15;
        for (int x = 1, q = 0; tri && x < 6; ++x)
            for (int y = 0; y < x; ++y, ++q)      // the upper-triangle form holds the same tiles transposed
                tri = tri && it.tile_x[q] == (upper ? y : x) && it.tile_y[q] == (upper ? x : y);
        it.pad = tri ? 1 : 0;
    }
    return ok;
}

// ---------------------------------------------------------------------------------------------
// MMA warps
// ---------------------------------------------------------------------------------------------
// The MMA warps address shared memory by 32-bit shared-space addresses: fewer registers held
// across the M loop than with generic pointers.
__device__ __forceinline__ double lds_f64(uint32_t addr) {
    double v;
    asm volatile("ld.shared.f64 %0, [%1];" : "=d"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ bool try_wait32(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool wait_full_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status, int lane) {
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!try_wait32(bar, parity)) {
        if ((++spins & 0x3FFu) == 0 && (*abort_flag != 0 || global_timer_ns() - t0 > kWaitLimitNs)) {
            *abort_flag = 1;
            if (lane == 0) atomicOr(status, kStatusWaitFull);
            return false;
        }
    }
    return true;
}
__device__ __forceinline__ bool wait_full_at(const Call& k, uint32_t st, uint32_t parity, int lane) {
    const uint32_t bar = k.bars32 + st * 8;
    if (try_wait32(bar, parity)) return true;
    return wait_full_slow(bar, parity, k.abort_flag, k.status, lane);
}
__device__ __forceinline__ void release_at(const Call& k, uint32_t st, int lane) {
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(k.empties32 + st * 8) : "memory");
}
__device__ __forceinline__ bool wait_full(const Call& k, uint32_t g, int lane) {
    return wait_full_at(k, g % kStages, (g / kStages) & 1, lane);
}
__device__ __forceinline__ void release(const Call& k, uint32_t g, int lane) { release_at(k, g % kStages, lane); }

// The M loop of one warp's tile.  kSkipLast leaves out block (3, 3), which the 16th warp of
// a triangle block computes.  Returns false when a bounded wait ran out.
// Shared-memory address of a fragment element.  A stored N x M (kTN false): 8-row group j of a
// segment is 1024 bytes further, k-slice sl flips the 16-byte chunk.  A stored M x N (kTN true):
// see fragment_offset_tn.
template <bool kTN>
__device__ __forceinline__ uint32_t frag_addr(uint32_t p, int j, int sl) {
    if (kTN) return (p ^ uint32_t(((sl & 1) << 5) ^ ((j & 1) << 6))) + uint32_t((sl & 1) * 256 + (sl >> 1) * 1024 + (j >> 1) * 2048);
    return (p ^ uint32_t(sl << 4)) + uint32_t(j * 1024);
}

template <bool kSkipLast, bool kTN, int kSt = kStages>
__device__ __forceinline__ bool tile_mainloop(double (&acc)[4][4][2], const Call& k, uint32_t xbase, uint32_t ybase,
                                              uint32_t off0, uint32_t g0, int lane) {
    uint32_t st = g0 % kSt, parity = (g0 / kSt) & 1;              // stage and phase, advanced step by step
    for (int ks = 0; ks < k.n_ksteps; ++ks) {
        if (!wait_full_at(k, st, parity, lane)) return false;
        const uint32_t stage = k.smem32 + st * kStageBytes;
        const uint32_t px = (stage + xbase) | off0, py = (stage + ybase) | off0;   // 1024-aligned | offset < 1024
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
            double a[4], b[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                a[j] = lds_f64(frag_addr<kTN>(px, j, sl));
                b[j] = lds_f64(frag_addr<kTN>(py, j, sl));
            }
#pragma unroll
            for (int mi = 0; mi < 4; ++mi)
#pragma unroll
                for (int ni = 0; ni < 4; ++ni)
                    if (!(kSkipLast && mi == 3 && ni == 3)) dmma884(acc[mi][ni], a[mi], b[ni]);
        }
        release_at(k, st, lane);
        if (++st == kSt) { st = 0; parity ^= 1; }
    }
    return true;
}


__device__ __forceinline__ uint32_t fragment_offset(int lane) {
    // Lane (g, t) of an m8n8k4 fragment holds (row g, k = t).  The four k-slices of a stage take
    // k = 8*(t>>1) + 2*sl + (t&1): any assignment of the stage's 16 columns to (slice, t) is valid as
    // long as both operands use the same one, and this one makes every half-warp's 16 loads hit 16
    // different 8-byte bank pairs under the 128-byte swizzle (16-byte chunk index ^ row % 8).
    // Byte offset of slice sl within a 1024-byte group of 8 rows:
    //   g*128 + ((((t>>1)<<2 | sl) ^ g) << 4) + ((t&1) << 3)  ==  (slice 0's offset) ^ (sl << 4).
    const int g = lane >> 2, t = lane & 3;
    return uint32_t(g * 128 + ((((t >> 1) << 2) ^ g) << 4) + ((t & 1) << 3));
}

__device__ __forceinline__ uint32_t fragment_offset_tn(int lane) {
    // A stored M x N: a stage holds, per segment, two boxes of 16 k-rows x 16 columns (128-byte rows,
    // 16-byte chunk index ^ k % 8).  Column n = 8j + g of the segment is in box j>>1, chunk
    // 4(j&1) + (g>>1), half g&1.  Slice sl and lane t take k = (t&1) + 4(t>>1) + 2(sl&1) + 8(sl>>1): the
    // four k rows of a slice then fall on both halves of the banks (rows k and k^4 differ in chunk
    // bit 2), so a warp's 256 bytes take the minimum of two wavefronts.  With disjoint bits, the
    // address of (j, sl) is  (lane part ^ ((sl&1)<<5 ^ (j&1)<<6)) + (sl&1)*256 + (sl>>1)*1024 + (j>>1)*2048.
    const int g = lane >> 2, t = lane & 3;
    const int k_lane = (t & 1) + 4 * (t >> 1);
    return uint32_t(k_lane * 128 + ((((g >> 1) ^ k_lane)) << 4) + ((g & 1) << 3));
}

// The M loop of the 16th warp of a triangle block: block q = (x, y), y < x, of the 15 left-out 8 x 8 blocks
// is the product of rows 24..31 of segments x and y (kSwap: of y and x, the block as the tile stored above
// the diagonal holds it).
template <bool kTN, int kSt = kStages, bool kSwap = false>
__device__ __forceinline__ bool scavenger_mainloop(double (&sacc)[15][2], const Call& k, uint32_t off0, uint32_t g0, int lane) {
#pragma unroll
    for (int q = 0; q < 15; ++q) sacc[q][0] = sacc[q][1] = 0.0;
    uint32_t st = g0 % kSt, parity = (g0 / kSt) & 1;
    for (int ks = 0; ks < k.n_ksteps; ++ks) {
        if (!wait_full_at(k, st, parity, lane)) return false;
        const uint32_t base = (k.smem32 + st * kStageBytes) | off0;
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
            double f[6];
#pragma unroll
            for (int j = 0; j < 6; ++j) f[j] = lds_f64(frag_addr<kTN>(base, 3, sl) + j * kSegBytes);   // rows 24..31 of every segment
            int q = 0;
#pragma unroll
            for (int x = 1; x < 6; ++x)
#pragma unroll
                for (int y = 0; y < x; ++y, ++q) dmma884(sacc[q], kSwap ? f[y] : f[x], kSwap ? f[x] : f[y]);
        }
        release_at(k, st, lane);
        if (++st == kSt) { st = 0; parity ^= 1; }
    }
    return true;
}

// 16th warp of a triangle block: the 15 left-out 8 x 8 blocks.  g0 = the item's first ring step,
// n_c = its old-C steps.
template <bool kTN, bool kUpper>
__device__ __forceinline__ bool scavenger_role(const Call& k, const WorkItem& it, uint32_t g0, int n_c, int lane) {
    const int gq = lane >> 2, t = lane & 3;
    const uint32_t gc = g0 + uint32_t(k.n_ksteps);
    const bool use_beta = (k.beta != 0.0);
    const uint32_t off0 = kTN ? fragment_offset_tn(lane) : fragment_offset(lane);
    int32_t seg[6];
#pragma unroll
    for (int s = 0; s < 6; ++s) seg[s] = it.seg[s];
    double sacc[15][2];
    if (!scavenger_mainloop<kTN>(sacc, k, off0, g0, lane)) return false;
    for (int j = 0; j < n_c; ++j)
        if (!wait_full(k, gc + j, lane)) return false;
    int q = 0;
#pragma unroll
    for (int x = 1; x < 6; ++x)
#pragma unroll
        for (int y = 0; y < x; ++y, ++q) {
            if (kUpper) {
                // The block belongs to the tile stored above the diagonal: rows of segment y, columns of
                // segment x, i.e. the accumulator transposed: this lane's two values go to rows 2t, 2t+1,
                // column gq of the 8 x 8 block.
                const int64_t c = int64_t(seg[x]) * kTile + 24 + gq;
                if (c >= k.N) continue;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int64_t r = int64_t(seg[y]) * kTile + 24 + 2 * t + e;
                    if (r >= k.N) continue;
                    double* p = k.C + r * k.ldc + c;
                    double v = scaled(k.alpha, sacc[q][e]);
                    if (n_c > 0)
                        v = plus_old(v, k.beta, *reinterpret_cast<const double*>(
                                 k.smem + ((gc + (q >> 2)) % kStages) * kStageBytes + (q & 3) * kCTileBytes +
                                 (24 + 2 * t + e) * (kTile * 8) + (24 + gq) * 8));
                    else if (use_beta) v = plus_old(v, k.beta, *p);
                    *p = v;
                }
                continue;
            }
            if (k.vec_ok & kVecOkPartial) {                         // partial tile q of a K-slice: raw sums, no mask
                *reinterpret_cast<double2*>(k.C + q * kPartTileElems + (24 + gq) * kTile + 24 + 2 * t) =
                    make_double2(sacc[q][0], sacc[q][1]);
                continue;
            }
            const int64_t r = int64_t(seg[x]) * kTile + 24 + gq;
            const int64_t c = int64_t(seg[y]) * kTile + 24 + 2 * t;
            if (r >= k.N) continue;                                 // tile below the diagonal: c + 1 < r
            double* p = k.C + r * k.ldc + c;
            double v0 = scaled(k.alpha, sacc[q][0]), v1 = scaled(k.alpha, sacc[q][1]);
            if (n_c > 0) {
                const double2 o = *reinterpret_cast<const double2*>(
                    k.smem + ((gc + (q >> 2)) % kStages) * kStageBytes + (q & 3) * kCTileBytes +
                    (24 + gq) * (kTile * 8) + (24 + 2 * t) * 8);
                v0 = plus_old(v0, k.beta, o.x); v1 = plus_old(v1, k.beta, o.y);
            } else if (use_beta) { v0 = plus_old(v0, k.beta, p[0]); v1 = plus_old(v1, k.beta, p[1]); }
            if (k.vec_ok) *reinterpret_cast<double2*>(p) = make_double2(v0, v1);
            else { p[0] = v0; p[1] = v1; }
        }
    for (int j = 0; j < n_c; ++j) release(k, gc + j, lane);
    return true;
}

// A warp with a tile (tile number `warp` of the item).  `scavenge`: block (3, 3) is left to the 16th warp.
template <bool kTN, bool kUpper>
__device__ __forceinline__ bool tile_role(const Call& k, const WorkItem& it, uint32_t g0, int n_c, bool scavenge,
                                          int warp, int lane) {
    const int gq = lane >> 2, t = lane & 3;
    const uint32_t gc = g0 + uint32_t(k.n_ksteps);
    const bool use_beta = (k.beta != 0.0);
    const uint32_t off0 = kTN ? fragment_offset_tn(lane) : fragment_offset(lane);
    const int sx = it.tile_x[warp], sy = it.tile_y[warp];
    const int64_t row0 = int64_t(it.seg[sx]) * kTile, col0 = int64_t(it.seg[sy]) * kTile;
    const uint32_t xbase = uint32_t(sx) * kSegBytes, ybase = uint32_t(sy) * kSegBytes;

    double acc[4][4][2];
#pragma unroll
    for (int mi = 0; mi < 4; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) acc[mi][ni][0] = acc[mi][ni][1] = 0.0;

    const bool alive = scavenge ? tile_mainloop<true, kTN>(acc, k, xbase, ybase, off0, g0, lane)
                                : tile_mainloop<false, kTN>(acc, k, xbase, ybase, off0, g0, lane);
    if (!alive) return false;

    for (int j = 0; j < n_c; ++j)
        if (!wait_full(k, gc + j, lane)) return false;
    const uint8_t* old_tile = nullptr;                  // this warp's old C tile in shared memory
    if (n_c > 0 && (k.gemm || row0 != col0))
        old_tile = k.smem + ((gc + (warp >> 2)) % kStages) * kStageBytes + (warp & 3) * kCTileBytes;
    if (kUpper) {
        // Upper-triangle form: row r keeps columns r .. N-1; either value of a pair may be the one kept.
#pragma unroll
        for (int mi = 0; mi < 4; ++mi) {
            const int64_t r = row0 + mi * 8 + gq;
            if (r >= k.N) continue;
            double* crow = k.C + r * k.ldc;
#pragma unroll
            for (int ni = 0; ni < 4; ++ni) {
                if (scavenge && mi == 3 && ni == 3) continue;             // written by the 16th warp
                const int64_t c = col0 + ni * 8 + 2 * t;
                const bool ok0 = c >= r && c < k.N, ok1 = c + 1 >= r && c + 1 < k.N;
                if (!ok0 && !ok1) continue;
                double v0 = scaled(k.alpha, acc[mi][ni][0]), v1 = scaled(k.alpha, acc[mi][ni][1]);
                if (use_beta) {
                    double2 o = make_double2(0.0, 0.0);
                    if (old_tile) o = *reinterpret_cast<const double2*>(old_tile + (mi * 8 + gq) * (kTile * 8) + (ni * 8 + 2 * t) * 8);
                    else { if (ok0) o.x = crow[c]; if (ok1) o.y = crow[c + 1]; }
                    v0 = plus_old(v0, k.beta, o.x); v1 = plus_old(v1, k.beta, o.y);
                }
                if (ok0 && ok1 && k.vec_ok) *reinterpret_cast<double2*>(crow + c) = make_double2(v0, v1);
                else { if (ok0) crow[c] = v0; if (ok1) crow[c + 1] = v1; }
            }
        }
        for (int j = 0; j < n_c; ++j) release(k, gc + j, lane);
        return true;
    }
    if (!kUpper && (k.vec_ok & kVecOkPartial)) {
        // A K-slice of a tail item: the raw sums of this warp's tile go to slot `warp` of the unit's partial
        // tiles, all 32 x 32 entries (the reduction applies alpha, beta and the triangle mask).
        double* out = k.C + warp * kPartTileElems;
#pragma unroll
        for (int mi = 0; mi < 4; ++mi)
#pragma unroll
            for (int ni = 0; ni < 4; ++ni) {
                if (scavenge && mi == 3 && ni == 3) continue;             // written by the 16th warp
                *reinterpret_cast<double2*>(out + (mi * 8 + gq) * kTile + ni * 8 + 2 * t) =
                    make_double2(acc[mi][ni][0], acc[mi][ni][1]);
            }
        return true;
    }
#pragma unroll
    for (int mi = 0; mi < 4; ++mi) {
        const int64_t r = row0 + mi * 8 + gq;
        if (r >= k.N) continue;
        const int64_t cmax = k.gemm ? k.ncols - 1 : r;  // last column this row may touch
        double* crow = k.C + r * k.ldc;
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
            if (scavenge && mi == 3 && ni == 3) continue;             // written by the 16th warp
            const int64_t c = col0 + ni * 8 + 2 * t;
            if (c > cmax) continue;
            const bool both = (c + 1 <= cmax);
            double v0 = scaled(k.alpha, acc[mi][ni][0]), v1 = scaled(k.alpha, acc[mi][ni][1]);
            if (use_beta) {
                double2 o = make_double2(0.0, 0.0);
                if (old_tile) o = *reinterpret_cast<const double2*>(old_tile + (mi * 8 + gq) * (kTile * 8) + (ni * 8 + 2 * t) * 8);
                else if (both && k.vec_ok) o = *reinterpret_cast<const double2*>(crow + c);
                else { o.x = crow[c]; if (both) o.y = crow[c + 1]; }
                v0 = plus_old(v0, k.beta, o.x); v1 = plus_old(v1, k.beta, o.y);
            }
            if (both) {
                if (k.vec_ok) *reinterpret_cast<double2*>(crow + c) = make_double2(v0, v1);
                else { crow[c] = v0; crow[c + 1] = v1; }
            } else {
                crow[c] = v0;
            }
        }
    }
    for (int j = 0; j < n_c; ++j) release(k, gc + j, lane);
    return true;
}

// Rank-2k update: warp w owns rows 16 (w & 1) .. + 15 of tile w >> 1 and adds both products,
// A_x B_y^T and B_x A_y^T, into the same 16 x 32 accumulator (2 x 4 blocks of m8n8k4): 16 DMMAs per
// k-slice and warp, as for a whole tile of the rank-k update.  N x M operands, lower triangle.
template <int kSt = kStages>
__device__ __forceinline__ bool syr2k_mainloop(double (&acc)[2][4][2], const Call& k, int sx, int sy, int half,
                                               uint32_t off0, uint32_t g0, int lane) {
    const uint32_t xa = uint32_t(sx) * kSegBytes, ya = uint32_t(sy) * kSegBytes;
    const uint32_t xb = uint32_t(kSyr2kSlots + sx) * kSegBytes, yb = uint32_t(kSyr2kSlots + sy) * kSegBytes;
#pragma unroll
    for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) acc[mi][ni][0] = acc[mi][ni][1] = 0.0;
    uint32_t st = g0 % kSt, parity = (g0 / kSt) & 1;
    for (int ks = 0; ks < k.n_ksteps; ++ks) {
        if (!wait_full_at(k, st, parity, lane)) return false;
        const uint32_t stage = k.smem32 + st * kStageBytes;
        const uint32_t pxa = (stage + xa) | off0, pya = (stage + ya) | off0;
        const uint32_t pxb = (stage + xb) | off0, pyb = (stage + yb) | off0;
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
            double a1[2], a2[2], b1[4], b2[4];
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) {
                a1[mi] = lds_f64(frag_addr<false>(pxa, 2 * half + mi, sl));
                a2[mi] = lds_f64(frag_addr<false>(pxb, 2 * half + mi, sl));
            }
#pragma unroll
            for (int ni = 0; ni < 4; ++ni) {
                b1[ni] = lds_f64(frag_addr<false>(pyb, ni, sl));
                b2[ni] = lds_f64(frag_addr<false>(pya, ni, sl));
            }
#pragma unroll
            for (int mi = 0; mi < 2; ++mi)
#pragma unroll
                for (int ni = 0; ni < 4; ++ni) {
                    dmma884(acc[mi][ni], a1[mi], b1[ni]);
                    dmma884(acc[mi][ni], a2[mi], b2[ni]);
                }
        }
        release_at(k, st, lane);
        if (++st == kSt) { st = 0; parity ^= 1; }
    }
    return true;
}

__device__ __forceinline__ bool syr2k_tile_role(const Call& k, const WorkItem& it, uint32_t g0, int n_c, int warp, int lane) {
    const int gq = lane >> 2, t = lane & 3;
    const int tile = warp >> 1, half = warp & 1;
    const uint32_t gc = g0 + uint32_t(k.n_ksteps);
    const bool use_beta = (k.beta != 0.0);
    const int sx = it.tile_x[tile], sy = it.tile_y[tile];
    const int64_t row0 = int64_t(it.seg[sx]) * kTile, col0 = int64_t(it.seg[sy]) * kTile;

    double acc[2][4][2];
    if (!syr2k_mainloop(acc, k, sx, sy, half, fragment_offset(lane), g0, lane)) return false;

    for (int j = 0; j < n_c; ++j)
        if (!wait_full(k, gc + j, lane)) return false;
    const uint8_t* old_tile = nullptr;
    if (n_c > 0 && row0 != col0)
        old_tile = k.smem + ((gc + (tile >> 2)) % kStages) * kStageBytes + (tile & 3) * kCTileBytes;
#pragma unroll
    for (int mi = 0; mi < 2; ++mi) {
        const int rr = (2 * half + mi) * 8 + gq;            // row inside the tile
        const int64_t r = row0 + rr;
        if (r >= k.N) continue;
        double* crow = k.C + r * k.ldc;
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
            const int64_t c = col0 + ni * 8 + 2 * t;
            if (c > r) continue;
            const bool both = (c + 1 <= r);
            double v0 = scaled(k.alpha, acc[mi][ni][0]), v1 = scaled(k.alpha, acc[mi][ni][1]);
            if (use_beta) {
                double2 o = make_double2(0.0, 0.0);
                if (old_tile) o = *reinterpret_cast<const double2*>(old_tile + rr * (kTile * 8) + (ni * 8 + 2 * t) * 8);
                else { o.x = crow[c]; if (both) o.y = crow[c + 1]; }
                v0 = plus_old(v0, k.beta, o.x); v1 = plus_old(v1, k.beta, o.y);
            }
            if (both && k.vec_ok) *reinterpret_cast<double2*>(crow + c) = make_double2(v0, v1);
            else { crow[c] = v0; if (both) crow[c + 1] = v1; }
        }
    }
    for (int j = 0; j < n_c; ++j) release(k, gc + j, lane);
    return true;
}

// Hermitian rank-k update, C <- alpha * A * A^H + beta * C with A complex N x M (pairs re, im) and C complex:
// the stages hold the real view of A (row i = 2M reals).  With A[i][k] = a + b i and A[j][k] = c + d i,
//     Re C[i][j] = sum a c + b d = (row i of the view) . (row j of the view),
//     Im C[i][j] = sum b c - a d = (row i of the view) . (row j of the view of i * A),   i * (c + d i) = -d + c i.
// Lanes t and t ^ 1 of a fragment hold the two parts of one complex number (k = ... + (t & 1)), so the
// fragment of i * A is the partner's shared-memory word (address ^ 8) with the sign changed in the even lanes.
// Warp w owns rows 16 (w & 1) .. + 15 of tile w >> 1 with one 16 x 32 accumulator per part: 16 DMMAs per
// k-slice and warp, as for a whole tile of the rank-k update.  Lower triangle; the diagonal's imaginary part is
// written as zero and not read.  k.C and k.ldc address complex elements (two doubles each).
__device__ __forceinline__ double flip_sign(double v, uint32_t mask) {
    return __hiloint2double(__double2hiint(v) ^ int(mask), __double2loint(v));
}
template <int kSt = kStages>
__device__ __forceinline__ bool herk_mainloop(double (&re)[2][4][2], double (&im)[2][4][2], const Call& k, int sx, int sy,
                                              int half, uint32_t g0, int lane) {
    const uint32_t off0 = fragment_offset(lane);
    const uint32_t flip = (lane & 1) ? 0u : 0x80000000u;
    const uint32_t xa = uint32_t(sx) * kSegBytes, ya = uint32_t(sy) * kSegBytes;
#pragma unroll
    for (int mi = 0; mi < 2; ++mi)
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) re[mi][ni][0] = re[mi][ni][1] = im[mi][ni][0] = im[mi][ni][1] = 0.0;
    uint32_t st = g0 % kSt, parity = (g0 / kSt) & 1;
    for (int ks = 0; ks < k.n_ksteps; ++ks) {
        if (!wait_full_at(k, st, parity, lane)) return false;
        const uint32_t stage = k.smem32 + st * kStageBytes;
        const uint32_t px = (stage + xa) | off0, py = (stage + ya) | off0;
#pragma unroll
        for (int sl = 0; sl < 4; ++sl) {
            double a[2], b[4], r[4];
#pragma unroll
            for (int mi = 0; mi < 2; ++mi) a[mi] = lds_f64(frag_addr<false>(px, 2 * half + mi, sl));
#pragma unroll
            for (int ni = 0; ni < 4; ++ni) {
                const uint32_t addr = frag_addr<false>(py, ni, sl);
                b[ni] = lds_f64(addr);
                r[ni] = flip_sign(lds_f64(addr ^ 8u), flip);
            }
#pragma unroll
            for (int mi = 0; mi < 2; ++mi)
#pragma unroll
                for (int ni = 0; ni < 4; ++ni) {
                    dmma884(re[mi][ni], a[mi], b[ni]);
                    dmma884(im[mi][ni], a[mi], r[ni]);
                }
        }
        release_at(k, st, lane);
        if (++st == kSt) { st = 0; parity ^= 1; }
    }
    return true;
}

__device__ __forceinline__ bool herk_tile_role(const Call& k, const WorkItem& it, uint32_t g0, int warp, int lane) {
    const int gq = lane >> 2, t = lane & 3;
    const int tile = warp >> 1, half = warp & 1;
    const bool use_beta = (k.beta != 0.0);
    const int sx = it.tile_x[tile], sy = it.tile_y[tile];
    const int64_t row0 = int64_t(it.seg[sx]) * kTile, col0 = int64_t(it.seg[sy]) * kTile;

    double re[2][4][2], im[2][4][2];
    if (!herk_mainloop(re, im, k, sx, sy, half, g0, lane)) return false;

#pragma unroll
    for (int mi = 0; mi < 2; ++mi) {
        const int64_t r = row0 + (2 * half + mi) * 8 + gq;
        if (r >= k.N) continue;
        double* crow = k.C + 2 * r * k.ldc;
#pragma unroll
        for (int ni = 0; ni < 4; ++ni) {
            const int64_t c = col0 + ni * 8 + 2 * t;
            if (c > r) continue;
            const bool both = (c + 1 <= r);
            double2 v0 = make_double2(scaled(k.alpha, re[mi][ni][0]), scaled(k.alpha, im[mi][ni][0]));
            double2 v1 = make_double2(scaled(k.alpha, re[mi][ni][1]), scaled(k.alpha, im[mi][ni][1]));
            if (use_beta) {
                const double2 o0 = *reinterpret_cast<const double2*>(crow + 2 * c);
                v0.x = plus_old(v0.x, k.beta, o0.x); v0.y = plus_old(v0.y, k.beta, o0.y);
                if (both) {
                    const double2 o1 = *reinterpret_cast<const double2*>(crow + 2 * c + 2);
                    v1.x = plus_old(v1.x, k.beta, o1.x); v1.y = plus_old(v1.y, k.beta, o1.y);
                }
            }
            if (c == r) v0.y = 0.0;
            if (c + 1 == r) v1.y = 0.0;
            *reinterpret_cast<double2*>(crow + 2 * c) = v0;
            if (both) *reinterpret_cast<double2*>(crow + 2 * c + 2) = v1;
        }
    }
    return true;
}

// One MMA warp's share of one item: its ring steps from global step g on, then its write-out.
// Every warp waits for and releases every ring step of the item, with or without work in it.
template <bool kTN, bool kUpper, bool kSyr2k = false, bool kHerk = false>
__device__ __forceinline__ bool mma_warp_item(const Call& k, const WorkItem& it, uint32_t& g, int warp, int lane) {
    const int n_tile = it.n_tile;
    const int n_c = c_steps_of(k, n_tile);
    const uint32_t g0 = g;
    g += uint32_t(k.n_ksteps + n_c);
    if (kSyr2k || kHerk) {
        if (warp < 2 * n_tile) return kHerk ? herk_tile_role(k, it, g0, warp, lane) : syr2k_tile_role(k, it, g0, n_c, warp, lane);
        for (uint32_t s = g0; s < g; ++s) {             // no work in this item: keep the ring moving
            if (!wait_full(k, s, lane)) return false;
            release(k, s, lane);
        }
        return true;
    }
    const bool scavenge = !k.gemm && it.pad != 0;      // set by prepare_item
    if (scavenge && warp == kMmaWarps - 1) return scavenger_role<kTN, kUpper>(k, it, g0, n_c, lane);
    if (warp < n_tile) return tile_role<kTN, kUpper>(k, it, g0, n_c, scavenge, warp, lane);
    for (uint32_t s = g0; s < g; ++s) {                 // no tile in this item: keep the ring moving
        if (!wait_full(k, s, lane)) return false;
        release(k, s, lane);
    }
    return true;
}

// ---------------------------------------------------------------------------------------------
// One block per item.  Two-operand mode (gemm_col_tiles > 0): D = alpha * P * Q^T + beta * D
// without a triangle mask; block b owns the 4 x 4 tile rectangle (b / column groups, b % column
// groups), its column segments come from Q (tmB, the first `pad` segments), its row segments
// from P (tmA).
// ---------------------------------------------------------------------------------------------
template <bool kTN, bool kUpper, bool kSyr2k = false, bool kHerk = false>
__global__ void __launch_bounds__(kThreads, 1)
syrk_f64_tbs_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const __grid_constant__ CUtensorMap tmC, const WorkItem* __restrict__ items, int64_t N,
                    int64_t ncols, int32_t gemm_col_tiles, int32_t n_ksteps, double* __restrict__ C,
                    int64_t ldc, double alpha, double beta, int vec_ok, int c_tma, int* __restrict__ status,
                    int64_t items_per_batch, int64_t c_batch_stride, int32_t slice_ksteps,
                    int32_t tail_first, int32_t tail_slices, double* __restrict__ tail_partial) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ WorkItem s_item;
    __shared__ volatile int s_abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    Call k;
    k.smem = smem;
    k.full_bar = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes);
    k.empty_bar = k.full_bar + kStages;
    k.smem32 = smem_u32(smem); k.bars32 = smem_u32(k.full_bar); k.empties32 = k.bars32 + kStages * 8;
    k.abort_flag = &s_abort; k.status = status;
    k.tmA = &tmA; k.tmB = &tmB; k.tmC = &tmC;
    k.N = N; k.ncols = ncols; k.n_ksteps = n_ksteps; k.C = C; k.ldc = ldc; k.alpha = alpha; k.beta = beta;
    k.vec_ok = vec_ok; k.c_tma = c_tma; k.gemm = gemm_col_tiles > 0; k.syr2k = kSyr2k; k.herk = kHerk;
    // Strided batch: the grid holds the work list once per matrix; the tensor maps are 3-D.
    // K-split (slice_ksteps > 0): the grid holds the list once per slice of the inner dimension;
    // slice s takes K-steps [s * slice_ksteps, ...) of the 2-D maps and writes partial matrix s.
    // Tail K-split (tail_slices > 1): blocks [0, tail_first) run items 0 .. tail_first - 1 whole; the blocks
    // after them run the remaining items in tail_slices slices of the inner dimension each (item-major),
    // writing raw partial tiles that a second kernel sums in slice order.
    k.batch = -1; k.k0 = 0;
    int64_t item_index = blockIdx.x;
    if (tail_slices > 1 && int64_t(blockIdx.x) >= int64_t(tail_first)) {
        const int64_t u = int64_t(blockIdx.x) - tail_first;
        const int32_t sl = int32_t(u % tail_slices);
        item_index = tail_first + u / tail_slices;
        k.k0 = int32_t(int64_t(n_ksteps) * sl / tail_slices);
        k.n_ksteps = int32_t(int64_t(n_ksteps) * (sl + 1) / tail_slices) - k.k0;
        k.C = tail_partial + u * kPartUnitElems;
        k.vec_ok = 1 | kVecOkPartial;
        k.c_tma = 0;
    }
    if (items_per_batch > 0) {
        const int32_t group = int32_t(int64_t(blockIdx.x) / items_per_batch);
        item_index = int64_t(blockIdx.x) % items_per_batch;
        k.C = C + int64_t(group) * c_batch_stride;
        if (slice_ksteps > 0) {
            k.k0 = group * slice_ksteps;
            k.n_ksteps = min(slice_ksteps, n_ksteps - k.k0);
        } else {
            k.batch = group;
        }
    }

    if (k.gemm) {
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
        reinterpret_cast<int32_t*>(&s_item)[tid] = reinterpret_cast<const int32_t*>(&items[item_index])[tid];
    }
    if (tid == 0) s_abort = 0;
    __syncthreads();
    if (tid == 0) {
        if (!prepare_item(k, s_item, kUpper)) { s_abort = 1; atomicOr(status, kStatusBadItem); }
        else {
            for (int s = 0; s < kStages; ++s) { mbar_init(&k.full_bar[s], 1); mbar_init(&k.empty_bar[s], kMmaWarps); }
            mbar_fence_init();
        }
    }
    __syncthreads();
    if (s_abort) return;

    uint32_t g = 0;
    if (warp == kMmaWarps) {
        if (lane == 0) {
            prefetch_tensormap(&tmA);
            if (kSyr2k) prefetch_tensormap(&tmB);
            if (c_tma) prefetch_tensormap(&tmC);
            produce_item<kTN>(k, s_item, g);
            if (s_abort) drain_producer(k, g);
        }
        return;
    }
    mma_warp_item<kTN, kUpper, kSyr2k, kHerk>(k, s_item, g, warp, lane);
}

// ---------------------------------------------------------------------------------------------
// Persistent form: one block per SM; the producer draws items from counter[0] (zero at launch;
// counter[1] counts the producers that are done) and publishes them through a ring of kItemRing
// slots.  The producer is never more than kPStages ring steps - hence fewer than kItemRing items -
// ahead of the slowest MMA warp, so a slot is rewritten only after every warp has read it.
//
// Write-out off the MMA warps: at the end of an item an MMA warp only copies its accumulators into a
// 128 KB image in shared memory (one 32 x 32 slot per tile) and goes on with the next item's stages, which
// are already in the ring; three write-out warps then form alpha * acc + beta * C from the image and store
// it while the DMMA pipes work on the next item.  (With the write-out in the MMA warps all sixteen do it at
// once and the pipes idle for the 128 KB that one SM has to move per item.)  The image takes the room of
// three of the six stages: this form runs a 3-stage ring, and old C is read from memory by the write-out
// warps, which have an item's duration to hide that latency.
// ---------------------------------------------------------------------------------------------
constexpr int kPStages = 3;
constexpr int kOutWarps = 3;
constexpr int kOutBatch = 4;                     // row pairs of a tile a write-out warp has in flight
constexpr int kPThreads = (kMmaWarps + 1 + kOutWarps) * 32;
constexpr int kImageBytes = kMmaWarps * kCTileBytes;
constexpr int kPSmemBytes = kPStages * kStageBytes + kImageBytes + (2 * kPStages + 2) * 8 + 1024;

// Entry (row r, 16-byte chunk c) of a tile's image: chunk index flipped in bit 2 on odd rows, so that both the
// fragment-shaped stores of the MMA warps (rows g, g + 1 x chunks 4 ni + t per quarter warp) and the row-shaped
// loads of the write-out warps are free of bank conflicts.
__device__ __forceinline__ uint32_t image_offset(int r, int c) { return uint32_t(r * 256 + ((c ^ ((r & 1) << 2)) << 4)); }
__device__ __forceinline__ void sts_f64x2(uint32_t addr, double v0, double v1) {
    asm volatile("st.shared.v2.f64 [%0], {%1, %2};" ::"r"(addr), "d"(v0), "d"(v1) : "memory");
}
__device__ __forceinline__ double2 lds_f64x2(uint32_t addr) {
    double2 v;
    asm volatile("ld.shared.v2.f64 {%0, %1}, [%2];" : "=d"(v.x), "=d"(v.y) : "r"(addr) : "memory");
    return v;
}

// What the persistent form adds to Call: the image and its two barriers (full: 16 arrivals, one per MMA warp
// and item; empty: one arrival per write-out warp and item).
struct Image {
    uint32_t base32, full32, empty32;
};

// Every MMA warp, with or without a tile in the item, passes this wait before its arrival on the image's full
// barrier: a warp's arrival for item i + 1 then cannot fall into the barrier phase of item i (the image of item
// i is only released after that phase has completed and the write-out warps have read it).  The ring of stages
// alone does not guarantee that for items of three K-steps or fewer.
__device__ __forceinline__ bool wait_image_empty(const Call& k, const Image& im, uint32_t item_no, int lane) {
    if (item_no == 0) return true;
    const uint32_t parity = (item_no - 1) & 1;
    if (try_wait32(im.empty32, parity)) return true;
    return wait_full_slow(im.empty32, parity, k.abort_flag, k.status, lane);
}

// The update a persistent launch runs: rank-k, rank-2k (two warps per tile, the rows of B in the stages' upper
// slots) or Hermitian (two warps per tile, a real and an imaginary accumulator; the image holds complex entries,
// 16 KB per tile, 16-byte entries with the index flipped in bit 0 on odd rows).
constexpr int kModeSyrk = 0, kModeSyr2k = 1, kModeHerk = 2;

// Keeps the ring moving for a warp without work in an item.
__device__ __forceinline__ bool idle_mainloop_p(const Call& k, uint32_t g0, int lane) {
    uint32_t st = g0 % kPStages, parity = (g0 / kPStages) & 1;
    for (int ks = 0; ks < k.n_ksteps; ++ks) {
        if (!wait_full_at(k, st, parity, lane)) return false;
        release_at(k, st, lane);
        if (++st == kPStages) { st = 0; parity ^= 1; }
    }
    return true;
}

// One MMA warp's share of item number item_no of its block: the M loop, then its accumulators into the image.
template <bool kTN, bool kUpper, int kMode>
__device__ __forceinline__ bool mma_warp_item_p(const Call& k, const Image& im, const WorkItem& it, uint32_t& g,
                                                uint32_t item_no, int warp, int lane) {
    const int gq = lane >> 2, t = lane & 3;
    const int n_tile = it.n_tile;
    const uint32_t g0 = g;
    g += uint32_t(k.n_ksteps);
    if (kMode != kModeSyrk) {
        if (warp < 2 * n_tile) {
            const int tile = warp >> 1, half = warp & 1;
            const int sx = it.tile_x[tile], sy = it.tile_y[tile];
            if (kMode == kModeSyr2k) {
                double acc[2][4][2];
                if (!syr2k_mainloop<kPStages>(acc, k, sx, sy, half, fragment_offset(lane), g0, lane)) return false;
                if (!wait_image_empty(k, im, item_no, lane)) return false;
                const uint32_t tile32 = im.base32 + tile * kCTileBytes;
#pragma unroll
                for (int mi = 0; mi < 2; ++mi)
#pragma unroll
                    for (int ni = 0; ni < 4; ++ni)
                        sts_f64x2(tile32 + image_offset((2 * half + mi) * 8 + gq, ni * 4 + t), scaled(k.alpha, acc[mi][ni][0]),
                                  scaled(k.alpha, acc[mi][ni][1]));
            } else {
                double re[2][4][2], imag[2][4][2];
                if (!herk_mainloop<kPStages>(re, imag, k, sx, sy, half, g0, lane)) return false;
                if (!wait_image_empty(k, im, item_no, lane)) return false;
                const uint32_t tile32 = im.base32 + tile * 2 * kCTileBytes;
                const int diag = int(it.seg[sx] == it.seg[sy]);          // a tile on the diagonal: Im C[i][i] = 0
#pragma unroll
                for (int mi = 0; mi < 2; ++mi)
#pragma unroll
                    for (int ni = 0; ni < 4; ++ni)
#pragma unroll
                        for (int e = 0; e < 2; ++e) {
                            const int r = (2 * half + mi) * 8 + gq, c = ni * 8 + 2 * t + e;
                            sts_f64x2(tile32 + uint32_t(r * 512 + ((c ^ (r & 1)) << 4)), scaled(k.alpha, re[mi][ni][e]),
                                      (diag && r == c) ? 0.0 : scaled(k.alpha, imag[mi][ni][e]));
                        }
            }
        } else if (!idle_mainloop_p(k, g0, lane) || !wait_image_empty(k, im, item_no, lane)) {
            return false;
        }
        __syncwarp();
        if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(im.full32) : "memory");
        return true;
    }
    const bool scavenge = it.pad != 0;                  // set by prepare_item
    const uint32_t off0 = kTN ? fragment_offset_tn(lane) : fragment_offset(lane);
    if (scavenge && warp == kMmaWarps - 1) {
        double sacc[15][2];
        if (!scavenger_mainloop<kTN, kPStages, kUpper>(sacc, k, off0, g0, lane)) return false;
        if (!wait_image_empty(k, im, item_no, lane)) return false;
#pragma unroll
        for (int q = 0; q < 15; ++q)                    // block (3, 3) of tile q
            sts_f64x2(im.base32 + q * kCTileBytes + image_offset(24 + gq, 12 + t), scaled(k.alpha, sacc[q][0]), scaled(k.alpha, sacc[q][1]));
    } else if (warp < n_tile) {
        const uint32_t xbase = uint32_t(it.tile_x[warp]) * kSegBytes, ybase = uint32_t(it.tile_y[warp]) * kSegBytes;
        double acc[4][4][2];
#pragma unroll
        for (int mi = 0; mi < 4; ++mi)
#pragma unroll
            for (int ni = 0; ni < 4; ++ni) acc[mi][ni][0] = acc[mi][ni][1] = 0.0;
        const bool alive = scavenge ? tile_mainloop<true, kTN, kPStages>(acc, k, xbase, ybase, off0, g0, lane)
                                    : tile_mainloop<false, kTN, kPStages>(acc, k, xbase, ybase, off0, g0, lane);
        if (!alive) return false;
        if (!wait_image_empty(k, im, item_no, lane)) return false;
        const uint32_t tile32 = im.base32 + warp * kCTileBytes;
#pragma unroll
        for (int mi = 0; mi < 4; ++mi)
#pragma unroll
            for (int ni = 0; ni < 4; ++ni) {
                if (scavenge && mi == 3 && ni == 3) continue;         // written by the 16th warp
                sts_f64x2(tile32 + image_offset(mi * 8 + gq, ni * 4 + t), scaled(k.alpha, acc[mi][ni][0]), scaled(k.alpha, acc[mi][ni][1]));
            }
    } else if (!idle_mainloop_p(k, g0, lane) || !wait_image_empty(k, im, item_no, lane)) {   // no tile in this item
        return false;
    }
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(im.full32) : "memory");
    return true;
}

// A write-out warp's share of one item: tiles out_warp, out_warp + 3, ... of the image, which holds alpha * acc.
// A warp instruction covers two rows of a tile (16 lanes x 16 bytes each): 256 contiguous bytes of C per row.
// The DMMA pipes are the FP64 pipes, and the MMA warps keep them full: an FP64 instruction issued from here
// waits behind them for most of an item.  So beta == 0 is a copy, and beta == 1 an addition done by the
// memory system (red.global.add.f64, one per entry and call: the result does not depend on any order, and it is
// the correctly rounded sum that the multiply-add of the other launch form gives for beta == 1); any other
// beta does its multiply-add here and is slow - the automatic choice of the launch form avoids it.
__device__ __forceinline__ void red_add_f64(double* p, double v) {
    asm volatile("red.global.add.f64 [%0], %1;" ::"l"(p), "d"(v) : "memory");
}
template <bool kUpper>
__device__ __forceinline__ void write_out_item(const Call& k, const Image& im, const WorkItem& it, double* C, int out_warp, int lane) {
    const int mode = (k.beta == 0.0) ? 0 : (k.beta == 1.0 ? 1 : 2);
    const int half = lane >> 4, c16 = lane & 15;
    for (int q = out_warp; q < it.n_tile; q += kOutWarps) {
        const int64_t row0 = int64_t(it.seg[it.tile_x[q]]) * kTile, col0 = int64_t(it.seg[it.tile_y[q]]) * kTile;
        const uint32_t tile32 = im.base32 + q * kCTileBytes;
        for (int i0 = 0; i0 < 16; i0 += kOutBatch) {
            double2 v[kOutBatch];
#pragma unroll
            for (int i = 0; i < kOutBatch; ++i) v[i] = lds_f64x2(tile32 + uint32_t((2 * (i0 + i) + half) * 256 + (c16 << 4)));
#pragma unroll
            for (int i = 0; i < kOutBatch; ++i) {
                const int r = 2 * (i0 + i) + half;
                const int64_t R = row0 + r, c = col0 + 2 * (c16 ^ ((r & 1) << 2));
                if (R >= k.N) continue;                                // beyond the last row
                // the entries of the pair (c, c + 1) that lie in the stored triangle
                const bool ok0 = kUpper ? (c >= R && c < k.N) : (c <= R);
                const bool ok1 = kUpper ? (c + 1 >= R && c + 1 < k.N) : (c + 1 <= R);
                if (!ok0 && !ok1) continue;
                double* p = C + R * k.ldc + c;
                if (mode == 0) {
                    if (ok0 && ok1 && (k.vec_ok & 1)) *reinterpret_cast<double2*>(p) = v[i];
                    else { if (ok0) p[0] = v[i].x; if (ok1) p[1] = v[i].y; }
                } else if (mode == 1) {
                    if (ok0) red_add_f64(p, v[i].x);
                    if (ok1) red_add_f64(p + 1, v[i].y);
                } else {
                    if (ok0) p[0] = plus_old(v[i].x, k.beta, p[0]);
                    if (ok1) p[1] = plus_old(v[i].y, k.beta, p[1]);
                }
            }
        }
    }
}

// A K-slice of a tail item (tail K-split, persistent form): the raw sums of every tile go to the unit's partial
// tiles (slot q at q * 1024 doubles, row-major 32 x 32), all entries; the reduction kernel applies alpha, beta and
// the triangle mask.
__device__ __forceinline__ void write_out_partial(const Image& im, const WorkItem& it, double* unit, int out_warp, int lane) {
    const int half = lane >> 4, c16 = lane & 15;
    for (int q = out_warp; q < it.n_tile; q += kOutWarps) {
        const uint32_t tile32 = im.base32 + q * kCTileBytes;
        double* dst = unit + q * kPartTileElems;
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
            const int r = 2 * i + half;
            const double2 v = lds_f64x2(tile32 + uint32_t(r * 256 + (c16 << 4)));
            *reinterpret_cast<double2*>(dst + r * kTile + 2 * (c16 ^ ((r & 1) << 2))) = v;
        }
    }
}

// The same for the Hermitian update: complex entries (re, im) of 16 bytes, a warp instruction covers one row of a
// tile (512 contiguous bytes of C); lower triangle; the diagonal's imaginary part is stored as zero, never read.
__device__ __forceinline__ void write_out_item_herk(const Call& k, const Image& im, const WorkItem& it, int out_warp, int lane) {
    const int mode = (k.beta == 0.0) ? 0 : (k.beta == 1.0 ? 1 : 2);
    for (int q = out_warp; q < it.n_tile; q += kOutWarps) {
        const int64_t row0 = int64_t(it.seg[it.tile_x[q]]) * kTile, col0 = int64_t(it.seg[it.tile_y[q]]) * kTile;
        const uint32_t tile32 = im.base32 + q * 2 * kCTileBytes;
        for (int r0 = 0; r0 < kTile; r0 += kOutBatch) {
            double2 v[kOutBatch];
#pragma unroll
            for (int i = 0; i < kOutBatch; ++i) v[i] = lds_f64x2(tile32 + uint32_t((r0 + i) * 512 + (lane << 4)));
#pragma unroll
            for (int i = 0; i < kOutBatch; ++i) {
                const int r = r0 + i;
                const int64_t R = row0 + r, c = col0 + (lane ^ (r & 1));
                if (R >= k.N || c > R) continue;
                double* p = k.C + 2 * (R * k.ldc + c);
                if (mode == 0) {
                    *reinterpret_cast<double2*>(p) = v[i];
                } else if (mode == 1) {
                    red_add_f64(p, v[i].x);
                    if (c == R) p[1] = 0.0; else red_add_f64(p + 1, v[i].y);
                } else {
                    p[0] = plus_old(v[i].x, k.beta, p[0]);
                    p[1] = (c == R) ? 0.0 : plus_old(v[i].y, k.beta, p[1]);
                }
            }
        }
    }
}

// kTail (rank-k update, lower triangle): tickets [0, tail_first) are the list's first items, whole; the tickets after
// them are the remaining items in tail_slices slices of the inner dimension each (item-major), whose raw sums go to
// `tail_partial` for tail_reduce_f64_kernel - smaller units for the last round, as in the one-block-per-item form.
template <bool kTN, bool kUpper, int kMode = kModeSyrk, bool kBatched = false, bool kTail = false>
__global__ void __launch_bounds__(kPThreads, 1)
syrk_f64_tbs_persistent_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                               const WorkItem* __restrict__ items,
                               int64_t n_items, int* __restrict__ counter, int64_t N, int32_t n_ksteps,
                               double* __restrict__ C, int64_t ldc, double alpha, double beta, int vec_ok,
                               int* __restrict__ status, int64_t items_per_batch, int64_t c_batch_stride,
                               int32_t tail_first, int32_t tail_slices, double* __restrict__ tail_partial) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    __shared__ WorkItem s_ring[kItemRing];
    __shared__ int32_t s_batch[kItemRing];        // strided batch (kBatched): the matrix an item belongs to
    __shared__ int32_t s_unit[kItemRing];         // kTail: the slice unit an entry of the ring is (-1: a whole item) ...
    __shared__ int32_t s_nk[kItemRing];           // ... and its number of K-steps
    __shared__ uint64_t s_item_bar[kItemRing];
    __shared__ volatile int s_abort;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    Call k;
    k.smem = smem;
    k.full_bar = reinterpret_cast<uint64_t*>(smem + kPStages * kStageBytes + kImageBytes);
    k.empty_bar = k.full_bar + kPStages;
    uint64_t* image_bar = k.empty_bar + kPStages;            // [0] full, [1] empty
    k.smem32 = smem_u32(smem); k.bars32 = smem_u32(k.full_bar); k.empties32 = k.bars32 + kPStages * 8;
    k.abort_flag = &s_abort; k.status = status;
    k.tmA = &tmA; k.tmB = &tmB; k.tmC = &tmA;
    k.N = N; k.ncols = N; k.n_ksteps = n_ksteps; k.C = C; k.ldc = ldc; k.alpha = alpha; k.beta = beta;
    k.vec_ok = vec_ok; k.c_tma = 0; k.gemm = false; k.batch = -1; k.k0 = 0;
    k.syr2k = kMode == kModeSyr2k; k.herk = kMode == kModeHerk;
    Image im;
    im.base32 = k.smem32 + kPStages * kStageBytes;
    im.full32 = smem_u32(&image_bar[0]);
    im.empty32 = smem_u32(&image_bar[1]);

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < kPStages; ++s) { mbar_init(&k.full_bar[s], 1); mbar_init(&k.empty_bar[s], kMmaWarps); }
        mbar_init(&image_bar[0], kMmaWarps);
        mbar_init(&image_bar[1], kOutWarps);
        for (int s = 0; s < kItemRing; ++s) mbar_init(&s_item_bar[s], 1);
        mbar_fence_init();
    }
    __syncthreads();

    // Warps 0..2 write out, warp 3 produces, warps 4..19 are MMA warps 0..15 (four per scheduler).
    uint32_t g = 0;
    if (warp == kOutWarps) {
        if (lane == 0) {
            prefetch_tensormap(&tmA);
            if (kMode == kModeSyr2k) prefetch_tensormap(&tmB);
            for (uint32_t slot = 0;; ++slot) {
                WorkItem& dst = s_ring[slot % kItemRing];
                const int64_t idx = s_abort ? n_items : int64_t(atomicAdd(counter, 1));
                bool last = idx >= n_items;
                if (!last) {
                    // strided batch: tickets run over (matrix, item) pairs, matrix-major; the 3-D tensor map takes the
                    // matrix as its last coordinate.  (A template parameter: with k.batch a constant the producer's loads
                    // are the 2-D ones without a branch: a few instructions more per load in this thread cost 0.5 % of a
                    // call.  Issuing the loads from several lanes, fetching the next item ahead of time, or moving this
                    // warp to another scheduler gained nothing - all measured.)
                    int64_t item_idx = idx;
                    if (kBatched) {
                        const int32_t matrix = int32_t(uint32_t(idx) / uint32_t(items_per_batch));
                        item_idx = idx - int64_t(matrix) * items_per_batch;
                        k.batch = matrix;
                        s_batch[slot % kItemRing] = matrix;
                    }
                    if (kTail) {
                        int32_t unit = -1, k0 = 0, nk = n_ksteps;
                        if (idx >= tail_first) {
                            unit = int32_t(idx) - tail_first;
                            const int32_t sl = unit % tail_slices;
                            item_idx = tail_first + unit / tail_slices;
                            k0 = int32_t(int64_t(n_ksteps) * sl / tail_slices);
                            nk = int32_t(int64_t(n_ksteps) * (sl + 1) / tail_slices) - k0;
                        }
                        k.k0 = k0; k.n_ksteps = nk;
                        s_unit[slot % kItemRing] = unit;
                        s_nk[slot % kItemRing] = nk;
                    }
                    for (int w = 0; w < int(sizeof(WorkItem) / 4); ++w)
                        reinterpret_cast<int32_t*>(&dst)[w] = reinterpret_cast<const int32_t*>(&items[item_idx])[w];
                    if (!prepare_item(k, dst, kUpper)) { s_abort = 1; atomicOr(status, kStatusBadItem); last = true; }
                }
                if (last) dst.n_tile = -1;                        // end marker
                mbar_arrive(&s_item_bar[slot % kItemRing]);       // publishes the slot (release)
                if (last) break;
                if (!produce_item<kTN, kPStages>(k, dst, g)) {     // gave up: tell the other warps to stop as well
                    WorkItem& end = s_ring[(slot + 1) % kItemRing];
                    end.n_tile = -1;
                    mbar_arrive(&s_item_bar[(slot + 1) % kItemRing]);
                    break;
                }
            }
            if (s_abort) drain_producer<kPStages>(k, g);
            // The last producer to get here puts both tickets back to zero for the next launch
            // on this stream: by then no block draws any more.
            if (atomicAdd(counter + 1, 1) == int(gridDim.x) - 1) { atomicExch(counter, 0); atomicExch(counter + 1, 0); }
        }
        return;
    }
    if (warp < kOutWarps) {
        // Write-out warps: item after item, one item behind the MMA warps at most (they wait for the image to be
        // empty before they fill it again), so the slot of the item ring is still the item's.
        const int out_warp = warp;
        for (uint32_t slot = 0;; ++slot) {
            if (!mbar_wait_bounded(&s_item_bar[slot % kItemRing], (slot / kItemRing) & 1, &s_abort)) {
                s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitFull); return;
            }
            const WorkItem& it = s_ring[slot % kItemRing];
            if (it.n_tile < 0) return;
            if (!mbar_wait_bounded(&image_bar[0], slot & 1, &s_abort)) {
                if (s_abort == 0) { s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitFull); }
                return;
            }
            if (kMode == kModeHerk) write_out_item_herk(k, im, it, out_warp, lane);
            else if (kTail && s_unit[slot % kItemRing] >= 0)
                write_out_partial(im, it, tail_partial + int64_t(s_unit[slot % kItemRing]) * kPartUnitElems, out_warp, lane);
            else write_out_item<kUpper>(k, im, it, kBatched ? k.C + int64_t(s_batch[slot % kItemRing]) * c_batch_stride : k.C,
                                        out_warp, lane);
            __syncwarp();
            if (lane == 0) mbar_arrive(&image_bar[1]);
        }
    }
    for (uint32_t slot = 0;; ++slot) {
        if (!mbar_wait_bounded(&s_item_bar[slot % kItemRing], (slot / kItemRing) & 1, &s_abort)) {
            s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitFull); return;
        }
        const WorkItem& it = s_ring[slot % kItemRing];
        if (it.n_tile < 0) return;
        if (kTail) {                                       // a slice's raw sums are left unscaled
            k.n_ksteps = s_nk[slot % kItemRing];
            k.alpha = s_unit[slot % kItemRing] >= 0 ? 1.0 : alpha;
        }
        if (!mma_warp_item_p<kTN, kUpper, kMode>(k, im, it, g, slot, warp - kOutWarps - 1, lane)) return;
    }
}

// K-split calls: stored triangle of C <- alpha * (sum of the slices' partial matrices, in slice
// order) + beta * C.  Partial matrix s is N x N with row pitch N at partial + s * N * N.
__global__ void __launch_bounds__(256)
splitk_reduce_f64_kernel(int64_t N, int32_t slices, const double* __restrict__ partial, double* __restrict__ C,
                         int64_t ldc, double alpha, double beta, int upper) {
    const int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x;
    const int64_t i = int64_t(blockIdx.y) * blockDim.y + threadIdx.y;
    if (i >= N || j >= N || (upper ? j < i : j > i)) return;
    double s = 0.0;
    for (int32_t sl = 0; sl < slices; ++sl) s += partial[(int64_t(sl) * N + i) * N + j];
    double* c = C + i * ldc + j;
    *c = (beta == 0.0) ? scaled(alpha, s) : plus_old(scaled(alpha, s), beta, *c);
}

// Tail K-split: for tail item i (list entry tail_first + i) and each of its tiles, the stored triangle of C
// <- alpha * (sum of the slices' partial tiles, in slice order) + beta * C.  Unit (i, slice) has its 16 tile
// slots at partial + (i * slices + slice) * 16 * 1024.
__global__ void __launch_bounds__(256)
tail_reduce_f64_kernel(const WorkItem* __restrict__ items, int32_t tail_first, int32_t slices,
                       const double* __restrict__ partial, int64_t N, double* __restrict__ C, int64_t ldc,
                       double alpha, double beta) {
    const WorkItem* it = &items[tail_first + blockIdx.x];
    const int q = blockIdx.y;
    if (q >= it->n_tile) return;
    const int64_t row0 = int64_t(it->seg[it->tile_x[q]]) * kTile, col0 = int64_t(it->seg[it->tile_y[q]]) * kTile;
    const double* src = partial + (int64_t(blockIdx.x) * slices * kMmaWarps + q) * kPartTileElems;
    for (int e = threadIdx.x; e < kPartTileElems; e += blockDim.x) {
        const int64_t r = row0 + e / kTile, c = col0 + e % kTile;
        if (r >= N || c > r) continue;
        double s = 0.0;
        for (int32_t sl = 0; sl < slices; ++sl) s += src[int64_t(sl) * kPartUnitElems + e];
        double* dst = C + r * ldc + c;
        *dst = (beta == 0.0) ? scaled(alpha, s) : plus_old(scaled(alpha, s), beta, *dst);
    }
}

}  // namespace f64

namespace {
cudaError_t configure_f64_kernels() {
    // The shared-memory attribute belongs to a device's context: set it once per device.
    static bool configured[64] = {};
    static std::mutex configured_mu;                 // launchers are reached under different locks
    std::lock_guard<std::mutex> configured_lock(configured_mu);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        const void* kernels[16] = {reinterpret_cast<const void*>(&f64::syrk_f64_tbs_kernel<false, false, false, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_kernel<false, false, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_kernel<false, false>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_kernel<true, false>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_kernel<false, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_kernel<true, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<false, false>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<true, false>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<false, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<true, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeSyr2k>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeHerk>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeSyrk, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<true, false, f64::kModeSyrk, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeSyrk, false, true>),
                                  reinterpret_cast<const void*>(&f64::syrk_f64_tbs_persistent_kernel<true, false, f64::kModeSyrk, false, true>)};
        for (const void* fn : kernels) {
            bool persistent = false;
            for (int i = 6; i < 16; ++i) persistent = persistent || fn == kernels[i];
            cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 persistent ? f64::kPSmemBytes : f64::kSmemBytes);
            if (e != cudaSuccess) return e;
        }
        configured[dev] = true;
    }
    return cudaSuccess;
}
}  // namespace

cudaError_t launch_syrk_f64(const CUtensorMap& tmA, const CUtensorMap* tmC, const WorkItem* d_items,
                            int64_t n_items, int64_t N, int64_t M, double* C, int64_t ldc, double alpha,
                            double beta, int a_is_m_by_n, int* d_tickets, int n_blocks, int* d_status,
                            cudaStream_t stream, int64_t batch, int64_t c_batch_stride, int split_k,
                            double* d_partial, int upper, int64_t tail_first, int tail_slices) {
    cudaError_t e = configure_f64_kernels();
    if (e != cudaSuccess) return e;
    if (n_items == 0) return cudaSuccess;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 1) == 0 &&
                        (batch <= 0 || (c_batch_stride & 1) == 0)) ? 1 : 0;
    const int32_t n_ksteps = int32_t((M + f64::kBK - 1) / f64::kBK);
    const int c_tma = (tmC != nullptr && beta != 0.0 && vec_ok) ? 1 : 0;
    CUtensorMap none{};
    const dim3 threads(f64::kThreads);
    if (split_k > 1 && batch <= 0 && d_partial != nullptr) {
        // K-split: one block per (slice, item); slices write partial matrices (alpha = 1, beta = 0,
        // old C not read), summed afterwards in slice order.
        const int32_t slice_ksteps = (n_ksteps + split_k - 1) / split_k;
        const int32_t slices = (n_ksteps + slice_ksteps - 1) / slice_ksteps;       // none of them empty
        if (n_items * slices >= (int64_t(1) << 31)) return cudaErrorInvalidValue;
        auto kernel = upper ? (a_is_m_by_n ? f64::syrk_f64_tbs_kernel<true, true> : f64::syrk_f64_tbs_kernel<false, true>)
                            : (a_is_m_by_n ? f64::syrk_f64_tbs_kernel<true, false> : f64::syrk_f64_tbs_kernel<false, false>);
        kernel<<<dim3(unsigned(n_items * slices)), threads, f64::kSmemBytes, stream>>>(
            tmA, tmA, none, d_items, N, N, 0, n_ksteps, d_partial, N, 1.0, 0.0, (N & 1) == 0 ? 1 : 0, 0, d_status,
            n_items, N * N, slice_ksteps, 0, 1, nullptr);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        const dim3 rb(32, 8);
        f64::splitk_reduce_f64_kernel<<<dim3(unsigned((N + 31) / 32), unsigned((N + 7) / 8)), rb, 0, stream>>>(
            N, slices, d_partial, C, ldc, alpha, beta, upper);
        return cudaGetLastError();
    }
    if (batch > 0) {
        if (upper) return cudaErrorInvalidValue;
        if (d_tickets != nullptr && n_blocks > 0 && n_items * batch < (int64_t(1) << 30)) {
            // Strided batch on persistent blocks: tickets over the (matrix, item) pairs.
            const int64_t units = n_items * batch;
            const dim3 grid(unsigned(units < n_blocks ? units : int64_t(n_blocks)));
            auto pk = a_is_m_by_n ? f64::syrk_f64_tbs_persistent_kernel<true, false, f64::kModeSyrk, true>
                                  : f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeSyrk, true>;
            pk<<<grid, dim3(f64::kPThreads), f64::kPSmemBytes, stream>>>(tmA, tmA, d_items, units, d_tickets, N, n_ksteps, C, ldc, alpha,
                                                                     beta, vec_ok, d_status, n_items, c_batch_stride, 0, 1, nullptr);
            return cudaGetLastError();
        }
        // Strided batch (3-D tensor maps): one block per (matrix, item), matrix-major.
        if (n_items * batch >= (int64_t(1) << 31)) return cudaErrorInvalidValue;
        auto kernel = a_is_m_by_n ? f64::syrk_f64_tbs_kernel<true, false> : f64::syrk_f64_tbs_kernel<false, false>;
        kernel<<<dim3(unsigned(n_items * batch)), threads, f64::kSmemBytes, stream>>>(
            tmA, tmA, c_tma ? *tmC : none, d_items, N, N, 0, n_ksteps, C, ldc, alpha, beta, vec_ok, c_tma, d_status,
            n_items, c_batch_stride, 0, 0, 1, nullptr);
        return cudaGetLastError();
    }
    if (d_tickets != nullptr && n_blocks > 0 && n_items < (int64_t(1) << 30) && tail_slices > 1 && d_partial != nullptr && !upper &&
        tail_first >= 0 && tail_first < n_items) {
        // Persistent blocks with a tail K-split: the last n_items - tail_first items as tail_slices tickets each.
        const int64_t n_tail = n_items - tail_first;
        const int64_t units = tail_first + n_tail * tail_slices;
        if (units >= (int64_t(1) << 30) || n_tail >= 65536 || tail_slices > n_ksteps) return cudaErrorInvalidValue;
        const dim3 grid(unsigned(units < n_blocks ? units : int64_t(n_blocks)));
        auto pk = a_is_m_by_n ? f64::syrk_f64_tbs_persistent_kernel<true, false, f64::kModeSyrk, false, true>
                              : f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeSyrk, false, true>;
        pk<<<grid, dim3(f64::kPThreads), f64::kPSmemBytes, stream>>>(tmA, tmA, d_items, units, d_tickets, N, n_ksteps, C, ldc, alpha,
                                                                 beta, vec_ok, d_status, int64_t(0), int64_t(0), int32_t(tail_first),
                                                                 int32_t(tail_slices), d_partial);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        f64::tail_reduce_f64_kernel<<<dim3(unsigned(n_tail), f64::kMmaWarps), 256, 0, stream>>>(
            d_items, int32_t(tail_first), int32_t(tail_slices), d_partial, N, C, ldc, alpha, beta);
        return cudaGetLastError();
    }
    if (d_tickets != nullptr && n_blocks > 0 && n_items < (int64_t(1) << 30)) {
        const dim3 grid(unsigned(n_items < n_blocks ? n_items : int64_t(n_blocks)));
        auto kernel = upper ? (a_is_m_by_n ? f64::syrk_f64_tbs_persistent_kernel<true, true> : f64::syrk_f64_tbs_persistent_kernel<false, true>)
                            : (a_is_m_by_n ? f64::syrk_f64_tbs_persistent_kernel<true, false> : f64::syrk_f64_tbs_persistent_kernel<false, false>);
        kernel<<<grid, dim3(f64::kPThreads), f64::kPSmemBytes, stream>>>(tmA, tmA, d_items, n_items, d_tickets, N, n_ksteps, C,
                                                                         ldc, alpha, beta, vec_ok, d_status, int64_t(0), int64_t(0), 0, 1, nullptr);
        return cudaGetLastError();
    }
    auto kernel = upper ? (a_is_m_by_n ? f64::syrk_f64_tbs_kernel<true, true> : f64::syrk_f64_tbs_kernel<false, true>)
                        : (a_is_m_by_n ? f64::syrk_f64_tbs_kernel<true, false> : f64::syrk_f64_tbs_kernel<false, false>);
    if (tail_slices > 1 && d_partial != nullptr && !upper && tail_first >= 0 && tail_first < n_items) {
        // Tail K-split: the last n_items - tail_first items run as tail_slices blocks each (see the kernel).
        const int64_t n_tail = n_items - tail_first;
        const int64_t blocks = tail_first + n_tail * tail_slices;
        if (blocks >= (int64_t(1) << 31) || n_tail >= 65536 || tail_slices > n_ksteps) return cudaErrorInvalidValue;
        kernel<<<dim3(unsigned(blocks)), threads, f64::kSmemBytes, stream>>>(
            tmA, tmA, c_tma ? *tmC : none, d_items, N, N, 0, n_ksteps, C, ldc, alpha, beta, vec_ok, c_tma, d_status,
            int64_t(0), int64_t(0), 0, int32_t(tail_first), int32_t(tail_slices), d_partial);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        f64::tail_reduce_f64_kernel<<<dim3(unsigned(n_tail), f64::kMmaWarps), 256, 0, stream>>>(
            d_items, int32_t(tail_first), int32_t(tail_slices), d_partial, N, C, ldc, alpha, beta);
        return cudaGetLastError();
    }
    kernel<<<dim3(unsigned(n_items)), threads, f64::kSmemBytes, stream>>>(
        tmA, tmA, c_tma ? *tmC : none, d_items, N, N, 0, n_ksteps, C, ldc, alpha, beta, vec_ok, c_tma, d_status,
        int64_t(0), int64_t(0), 0, 0, 1, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_syr2k_f64(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap* tmC,
                             const WorkItem* d_items, int64_t n_items, int64_t N, int64_t M, double* C, int64_t ldc,
                             double alpha, double beta, int* d_status, cudaStream_t stream, int* d_tickets, int n_blocks) {
    cudaError_t e = configure_f64_kernels();
    if (e != cudaSuccess) return e;
    if (n_items == 0) return cudaSuccess;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 1) == 0) ? 1 : 0;
    const int32_t n_ksteps = int32_t((M + f64::kBK - 1) / f64::kBK);
    if (d_tickets != nullptr && n_blocks > 0 && n_items < (int64_t(1) << 30)) {
        const dim3 grid(unsigned(n_items < n_blocks ? n_items : int64_t(n_blocks)));
        f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeSyr2k><<<grid, dim3(f64::kPThreads), f64::kPSmemBytes, stream>>>(
            tmA, tmB, d_items, n_items, d_tickets, N, n_ksteps, C, ldc, alpha, beta, vec_ok, d_status, int64_t(0), int64_t(0), 0, 1, nullptr);
        return cudaGetLastError();
    }
    const int c_tma = (tmC != nullptr && beta != 0.0 && vec_ok) ? 1 : 0;
    CUtensorMap none{};
    f64::syrk_f64_tbs_kernel<false, false, true><<<dim3(unsigned(n_items)), dim3(f64::kThreads), f64::kSmemBytes, stream>>>(
        tmA, tmB, c_tma ? *tmC : none, d_items, N, N, 0, n_ksteps, C, ldc, alpha, beta, vec_ok, c_tma, d_status,
        int64_t(0), int64_t(0), 0, 0, 1, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_herk_f64(const CUtensorMap& tmA, const WorkItem* d_items, int64_t n_items, int64_t N, int64_t M,
                            double* C, int64_t ldc, double alpha, double beta, int* d_status, cudaStream_t stream,
                            int* d_tickets, int n_blocks) {
    cudaError_t e = configure_f64_kernels();
    if (e != cudaSuccess) return e;
    if (n_items == 0) return cudaSuccess;
    if ((reinterpret_cast<uintptr_t>(C) & 15) != 0) return cudaErrorInvalidValue;     // complex entries move as 16-byte words
    const int32_t n_ksteps = int32_t((2 * M + f64::kBK - 1) / f64::kBK);             // the real view has 2M columns
    if (d_tickets != nullptr && n_blocks > 0 && n_items < (int64_t(1) << 30)) {
        const dim3 grid(unsigned(n_items < n_blocks ? n_items : int64_t(n_blocks)));
        f64::syrk_f64_tbs_persistent_kernel<false, false, f64::kModeHerk><<<grid, dim3(f64::kPThreads), f64::kPSmemBytes, stream>>>(
            tmA, tmA, d_items, n_items, d_tickets, N, n_ksteps, C, ldc, alpha, beta, 1, d_status, int64_t(0), int64_t(0), 0, 1, nullptr);
        return cudaGetLastError();
    }
    CUtensorMap none{};
    f64::syrk_f64_tbs_kernel<false, false, false, true><<<dim3(unsigned(n_items)), dim3(f64::kThreads), f64::kSmemBytes, stream>>>(
        tmA, tmA, none, d_items, N, N, 0, n_ksteps, C, ldc, alpha, beta, 1, 0, d_status,
        int64_t(0), int64_t(0), 0, 0, 1, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_gemm_nt_f64(const CUtensorMap& tmP, const CUtensorMap& tmQ, const CUtensorMap* tmD,
                               int64_t nrows, int64_t ncols, int64_t K, double* D, int64_t ldd, double alpha,
                               double beta, int* d_status, cudaStream_t stream) {
    cudaError_t e = configure_f64_kernels();
    if (e != cudaSuccess) return e;
    if (nrows == 0 || ncols == 0) return cudaSuccess;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(D) & 15) == 0 && (ldd & 1) == 0) ? 1 : 0;
    const int32_t n_ksteps = int32_t((K + f64::kBK - 1) / f64::kBK);
    const int c_tma = (tmD != nullptr && beta != 0.0 && vec_ok) ? 1 : 0;
    const int64_t row_tiles = (nrows + f64::kTile - 1) / f64::kTile, col_tiles = (ncols + f64::kTile - 1) / f64::kTile;
    const int64_t blocks = ((row_tiles + 3) / 4) * ((col_tiles + 3) / 4);
    CUtensorMap none{};
    f64::syrk_f64_tbs_kernel<false, false><<<dim3(unsigned(blocks)), dim3(f64::kThreads), f64::kSmemBytes, stream>>>(
        tmP, tmQ, c_tma ? *tmD : none, nullptr, nrows, ncols, int32_t(col_tiles), n_ksteps, D, ldd, alpha, beta,
        vec_ok, c_tma, d_status, int64_t(0), int64_t(0), 0, 0, 1, nullptr);
    return cudaGetLastError();
}

int64_t f64_tail_partial_elems(int64_t n_tail_items, int tail_slices) {
    return n_tail_items * int64_t(tail_slices) * f64::kPartUnitElems;
}
int f64_tile() { return f64::kTile; }
int f64_bk() { return f64::kBK; }
int f64_stages() { return f64::kStages; }
int f64_persistent_stages() { return f64::kPStages; }

}  // namespace tbsyrk
