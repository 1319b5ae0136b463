// BF16-in (or FP16-in, TF32-in, FP8-E4M3-in) / FP32-accumulate triangle-block SYRK kernel for sm_100a
// (tcgen05 + TMEM).  A stage row is 128 bytes for every input kind: 64 bfloat16 or binary16 columns
// (kind::f16, K = 16 per MMA), 32 binary32 columns read as TF32 (kind::tf32, K = 8) or 128 FP8
// columns (kind::f8f6f4, K = 32); everything else is shared.
//
// Persistent kernel, one thread block per SM, work units dealt round-robin.  A work
// unit is one item of the tiled TBS schedule (Algorithm 4 / Section 5.1.4 of the
// paper) restricted to one K-slice.  An item names up to 3 row segments of A (128
// rows each) and up to 3 output tiles; for a triangle block (k = 3) the tiles are
// (s1,s0), (s2,s0), (s2,s1): three 128 x 128 accumulators fed by three segments per
// K-step, where a rectangle of the same staging footprint owns two.
//
//   warp 0   : producer - plain TMA tile loads (no multicast) of the item's segments,
//              64 columns of A per stage, 4-stage ring, 128-byte swizzle;
//   warp 1   : allocates tensor memory; one lane issues tcgen05.mma (M = 128,
//              N = 128 or 256, K = 16) from shared-memory descriptors into TMEM
//              accumulators and frees ring stages with tcgen05.commit;
//   warps 2-5: epilogue - tcgen05.ld of the accumulators, alpha/beta, and either
//              swizzled shared-memory staging + asynchronous TMA stores (tiles below the
//              diagonal, beta == 0) or masked direct stores of the entries with
//              col <= row (diagonal tiles, beta != 0), or raw partial tiles when M is split.
//
// TMEM holds four 128-column slots.  The N = 256 accumulator pair of an item always
// lives in slots 1-2; its N = 128 accumulator alternates between slot 0 and slot 3
// from one item to the next.  The epilogue drains the pair first, so the next item's
// MMAs start while the previous item's third tile is still being written out.
//
// Both MMA operands come from the same row-major A (K contiguous): segment x is the
// M-operand, segment y (or the adjacent pair y, y+1) the N-operand, both K-major.  When A is
// stored M x N (the Gram form) the stages hold boxes of k-rows by columns and both
// operands are MN-major (for every input kind; the boxes are then one stage's k-rows by 128 bytes
// of columns); everything after the MMA is the same.
#include <mutex>

#include "device_utils.cuh"
#include "kernels.h"
#include "tbs_plan.h"

namespace tbsyrk {
namespace bf16 {

constexpr int kTile = 128;                        // b
constexpr int kBK = 64;                           // columns of A per stage (128 bytes)
constexpr int kStages = 4;
constexpr int kSegSlots = 3;                      // segments per stage
constexpr int kSegBytes = kTile * kBK * 2;        // 16384
constexpr int kStageBytes = kSegSlots * kSegBytes;
constexpr int kMaxTiles = 3;                      // 3 x 128 TMEM columns of 512
constexpr int kTmemCols = 512;
constexpr int kThreads = 192;
constexpr int kStoreBox = 32;                      // rows and FP32 columns per TMA store
constexpr int kStageBufBytes = kStoreBox * kStoreBox * 4;   // 4096
constexpr int kStagingBytes = 4 * 2 * kStageBufBytes;        // 4 epilogue warps x 2 buffers
constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024 + 256;

// ---- tcgen05 wrappers -------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Input kinds of the kernel: what a 128-byte stage row holds and which MMA reads it.
constexpr int kKindBF16 = 0;    // 64 bfloat16 columns, kind::f16, K = 16 per instruction
constexpr int kKindTF32 = 1;    // 32 binary32 columns read as TF32, kind::tf32, K = 8
constexpr int kKindE4M3 = 2;    // 128 FP8 E4M3 columns, kind::f8f6f4, K = 32
constexpr int kKindF16 = 3;     // 64 IEEE binary16 columns, kind::f16, K = 16
template <int kKind> struct KindCols {
    static constexpr int value = (kKind == kKindBF16 || kKind == kKindF16) ? 64 : (kKind == kKindTF32 ? 32 : 128);
};

// D[tmem] (+)= A[smem] * B[smem]^T, FP32 accumulation, M = 128; 32 bytes of K per instruction for
// every kind.
template <int kKind>
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                       uint32_t accumulate) {
    if (kKind == kKindTF32)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    else if (kKind == kKindE4M3)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
            : "memory");
}
// 32 lanes x 32 consecutive 32-bit columns: thread i of the warp gets lane (base + i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
        "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128
// bytes, 8-row groups 1024 bytes apart; `addr` is the shared-memory byte address of
// the first row (+ 32 bytes per K = 16 step inside the swizzle atom).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    uint64_t d = 0;
    d |= uint64_t((addr & 0x3FFFF) >> 4);          // start address
    d |= uint64_t(1024 >> 4) << 32;                // stride byte offset (between 8-row groups)
    d |= uint64_t(1) << 46;                        // descriptor version of sm_100
    d |= uint64_t(2) << 61;                        // layout: 128-byte swizzle
    return d;
}
// The same for an MN-major operand (A stored M x N: a segment's 128 columns are contiguous in
// memory, one 128-byte row per k).  A 128-byte row holds 64 two-byte, 32 binary32 or 128 FP8
// columns, so a segment slot holds 2, 4 or 1 column groups, each a box of one stage's k-rows,
// `group_bytes` apart (leading byte offset; the N = 256 operand runs on into the next slot with
// the same stride); within a group, 8-row k groups are 1024 bytes apart (stride byte offset);
// `addr` advances by (k-rows per MMA) * 128 bytes per instruction.
// binary32 (TF32) operands in this order use the 128-byte swizzle with 32-byte atoms instead (layout
// code 1; the tensor map over A is encoded with the matching TMA mode): its pattern repeats every 4
// k-rows, so the k groups are 512 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_mn_sw128(uint32_t addr, uint32_t group_bytes, bool atom32) {
    uint64_t d = 0;
    d |= uint64_t((addr & 0x3FFFF) >> 4);
    d |= uint64_t(group_bytes >> 4) << 16;         // leading byte offset (between column groups)
    d |= uint64_t((atom32 ? 512 : 1024) >> 4) << 32;   // stride byte offset (between k groups of 4 or 8 rows)
    d |= uint64_t(1) << 46;
    d |= uint64_t(atom32 ? 1 : 2) << 61;
    return d;
}
// Instruction descriptor, kind::f16: D = FP32, A = B = BF16, M = 128; both operands K-major, or
// both MN-major (bits 15 and 16) when A is stored M x N.
// The other kinds have the same fields; the operand format code is 1 (BF16) or 0 (binary16) for
// kind::f16, 2 (TF32) for kind::tf32 and 0 (E4M3) for kind::f8f6f4.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, bool mn_major, int kind) {
    const uint32_t fmt = kind == kKindBF16 ? 1u : (kind == kKindTF32 ? 2u : 0u);
    return (1u << 4) | (fmt << 7) | (fmt << 10) | (mn_major ? (3u << 15) : 0u) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// ---- bulk-async (TMA) store helpers ---------------------------------------------------
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tmap, const void* smem_src, int32_t x, int32_t y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(smem_src)) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// The same into matrix z of a strided batch (3-D map, box depth 1).
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* tmap, const void* smem_src, int32_t x, int32_t y, int32_t z) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(smem_u32(smem_src)) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

struct Unit {       // one work unit: an item and a range of K-steps (or a matrix of a strided batch)
    int64_t item;
    int32_t slice;
    int32_t k0, k1;
    int32_t batch;      // matrix number, or -1 outside batched calls
};
__device__ __forceinline__ Unit unit_of(int64_t w, int64_t n_items, int32_t n_ksteps, int32_t split, int32_t n_batch) {
    Unit u;
    u.item = w % n_items;
    if (n_batch > 0) {                            // batched calls: matrix-major, whole inner dimension
        u.batch = int32_t(w / n_items); u.slice = 0; u.k0 = 0; u.k1 = n_ksteps;
        return u;
    }
    u.batch = -1;
    u.slice = int32_t(w / n_items);               // slice-major: a wave shares one K-slab of A
    u.k0 = int32_t(int64_t(n_ksteps) * u.slice / split);
    u.k1 = int32_t(int64_t(n_ksteps) * (u.slice + 1) / split);
    return u;
}

// Where an item's accumulators live.  Tiles t, t+1 with the same M-operand segment and
// adjacent N-operand segments form one N = 256 MMA group in TMEM slots 1-2; a lone tile
// is an N = 128 group in the single slot (0 or 3, alternating per item).  A valid item has
// at most one group of each kind.
struct Layout {
    int n_grp;
    int gx[2], gy[2], gn[2];
    uint32_t gcol[2];
    uint32_t tile_col[kMaxTiles];
    bool tile_in_pair[kMaxTiles];
};
__device__ __forceinline__ void layout_of(const WorkItem* it, int n_tile, uint32_t single_col, Layout& L) {
    L.n_grp = 0;
    for (int t = 0; t < n_tile && L.n_grp < 2;) {
        const int x = it->tile_x[t], y = it->tile_y[t];
        const bool pair = (t + 1 < n_tile) && it->tile_x[t + 1] == x && it->tile_y[t + 1] == y + 1;
        const int q = L.n_grp++;
        L.gx[q] = x; L.gy[q] = y; L.gn[q] = pair ? 256 : 128;
        L.gcol[q] = pair ? uint32_t(kTile) : single_col;
        L.tile_col[t] = L.gcol[q]; L.tile_in_pair[t] = pair;
        if (pair) { L.tile_col[t + 1] = L.gcol[q] + kTile; L.tile_in_pair[t + 1] = true; }
        t += pair ? 2 : 1;
    }
}

// kSyr2k: the rank-2k update alpha (A B^T + B A^T) + beta C on the same work list.  A stage then holds the
// item's segments of A in slots 0-2 and the same rows of B (second tensor map) in slots 3-5 - 96 KB, so the
// ring has two stages instead of four - and every accumulator group takes two MMAs per 32 bytes of K,
// A_x B_y^T and B_x A_y^T.  Operands stored N x M, lower triangle.
template <bool kTN, int kKind, bool kUpper, bool kSyr2k = false>
__global__ void __launch_bounds__(kThreads, 1)
syrk_bf16_tbs_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                     const __grid_constant__ CUtensorMap tmC,
                     const WorkItem* __restrict__ items, int64_t n_items, int64_t N, int32_t n_ksteps,
                     float* __restrict__ C, int64_t ldc, float alpha, float beta, int vec_ok, int tma_store_ok,
                     int32_t split, float* __restrict__ partial, const int64_t* __restrict__ tile_base,
                     int64_t total_tiles, const int64_t* __restrict__ cta_begin, int* __restrict__ status,
                     int32_t n_batch, int64_t c_batch_stride) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* staging = smem + kStages * kStageBytes;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(staging + kStagingBytes);
    uint64_t* empty_bar = full_bar + kStages;
    uint64_t* tmem_full_bar = empty_bar + kStages;
    uint64_t* pair_free_bar = tmem_full_bar + 1;
    uint64_t* single_free_bar = pair_free_bar + 1;     // [2]
    uint64_t* drain_bar = single_free_bar + 2;
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kCols = KindCols<kKind>::value;        // columns of A in a 128-byte stage row
    constexpr int kSt = kSyr2k ? kStages / 2 : kStages;                 // ring depth
    constexpr int kStB = kSyr2k ? 2 * kStageBytes : kStageBytes;        // bytes of a stage (same ring size either way)
    static_assert(!kSyr2k || (!kTN && !kUpper), "the rank-2k form takes N x M operands and the lower triangle");
    const int64_t n_units = n_items * split * (n_batch > 0 ? n_batch : 1);
    // This block's units: its own contiguous range of a list ordered block by block on the host,
    // or (K-split calls) every gridDim.x-th unit of the slice-major list.
    const int64_t w_first = cta_begin ? cta_begin[blockIdx.x] : int64_t(blockIdx.x);
    const int64_t w_last = cta_begin ? cta_begin[blockIdx.x + 1] : n_units;
    const int64_t w_stride = cta_begin ? 1 : int64_t(gridDim.x);

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < kSt; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(tmem_full_bar, 1);
        mbar_init(pair_free_bar, 4);
        mbar_init(&single_free_bar[0], 4);
        mbar_init(&single_free_bar[1], 4);
        mbar_init(drain_bar, 1);
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(&s_tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;

    if (warp == 0) {
        // ------------------------------ producer ------------------------------
        if (lane == 0) {
            prefetch_tensormap(&tmA);
            if (kSyr2k) prefetch_tensormap(&tmB);
            uint32_t g = 0;
            for (int64_t w = w_first; w < w_last && !s_abort; w += w_stride) {
                const Unit u = unit_of(w, n_items, n_ksteps, split, n_batch);
                const WorkItem* it = &items[u.item];
                const int n_seg = it->n_seg;
                int32_t rows[kSegSlots];
                for (int s = 0; s < kSegSlots; ++s) rows[s] = (s < n_seg) ? it->seg[s] * kTile : 0;
                for (int ks = u.k0; ks < u.k1; ++ks, ++g) {
                    const uint32_t st = g % kSt;
                    if (g >= kSt && !mbar_wait_bounded(&empty_bar[st], ((g / kSt) - 1) & 1, &s_abort)) {
                        s_abort = 1; atomicOr(status, kStatusWaitEmpty); break;
                    }
                    mbar_arrive_expect_tx(&full_bar[st], uint32_t(kSyr2k ? 2 * n_seg : n_seg) * kSegBytes);
                    uint8_t* dst = smem + st * kStB;
                    if (kSyr2k) {   // rows of A in slots 0-2, the same rows of B in slots 3-5
                        for (int s = 0; s < n_seg; ++s) {
                            tma_load_box(dst + s * kSegBytes, &tmA, ks * kCols, rows[s], u.batch, &full_bar[st]);
                            tma_load_box(dst + (kSegSlots + s) * kSegBytes, &tmB, ks * kCols, rows[s], u.batch, &full_bar[st]);
                        }
                    } else if (kTN) {   // A stored M x N: per segment, boxes of one stage's k-rows x 128 bytes of columns
                        constexpr int kGroupCols = kCols;                 // columns in a 128-byte row: 64, 32 or 128
                        constexpr int kGroups = kTile / kGroupCols;
                        for (int s = 0; s < n_seg; ++s)
                            for (int h = 0; h < kGroups; ++h)
                                tma_load_box(dst + s * kSegBytes + h * (kSegBytes / kGroups), &tmA, rows[s] + h * kGroupCols,
                                             ks * kCols, u.batch, &full_bar[st]);
                    } else {
                        for (int s = 0; s < n_seg; ++s)
                            tma_load_box(dst + s * kSegBytes, &tmA, ks * kCols, rows[s], u.batch, &full_bar[st]);
                    }
                }
            }
            if (s_abort) {   // winding down: let the copies still in flight land first
                volatile int dummy = 0;
                for (uint32_t i = (g > kSt ? g - kSt : 0); i < g; ++i)
                    mbar_wait_bounded(&full_bar[i % kSt], (i / kSt) & 1, &dummy);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------ MMA issuer ------------------------------
        if (lane == 0) {
            uint32_t g = 0, n_done = 0;
            const uint32_t smem_base = smem_u32(smem);
            // MN-major: a column group is one stage's k-rows (kCols) of 128 bytes; an MMA takes a quarter of them
            const uint64_t desc_hi = kTN ? smem_desc_mn_sw128(0, uint32_t(kCols) * 128u, kKind == kKindTF32) : smem_desc_sw128(0);
            constexpr uint32_t kk_step = kTN ? ((uint32_t(kCols) * 32u) >> 4) : (32u >> 4);   // descriptor advance per MMA
            for (int64_t w = w_first; w < w_last && !s_abort; w += w_stride, ++n_done) {
                const Unit u = unit_of(w, n_items, n_ksteps, split, n_batch);
                const WorkItem* it = &items[u.item];
                Layout L;
                layout_of(it, it->n_tile, (n_done & 1) ? 3u * kTile : 0u, L);
                uint32_t a_lo[2], b_lo[2], idesc[2], d_addr[2];
                for (int q = 0; q < 2; ++q) {
                    const int qq = q < L.n_grp ? q : 0;
                    a_lo[q] = (smem_base + uint32_t(L.gx[qq]) * kSegBytes) >> 4;
                    b_lo[q] = (smem_base + uint32_t(L.gy[qq]) * kSegBytes) >> 4;
                    idesc[q] = instr_desc(uint32_t(L.gn[qq]), kTN, kKind);
                    d_addr[q] = tmem_base + L.gcol[qq];
                }
                // accumulators of this item must have been drained by the epilogue
                if (n_done >= 1 && !mbar_wait_bounded(pair_free_bar, (n_done - 1) & 1, &s_abort)) {
                    s_abort = 1; atomicOr(status, kStatusWaitTmem); break;
                }
                if (n_done >= 2 && !mbar_wait_bounded(&single_free_bar[n_done & 1], ((n_done >> 1) - 1) & 1, &s_abort)) {
                    s_abort = 1; atomicOr(status, kStatusWaitTmem); break;
                }
                tc_fence_after();
                bool ok = true;
                for (int ks = u.k0; ks < u.k1; ++ks, ++g) {
                    const uint32_t st = g % kSt;
                    if (!mbar_wait_bounded(&full_bar[st], (g / kSt) & 1, &s_abort)) {
                        s_abort = 1; atomicOr(status, kStatusWaitFull); ok = false; break;
                    }
                    tc_fence_after();
                    const uint32_t st_off = (st * kStB) >> 4;
                    const uint32_t first = (ks > u.k0) ? 1u : 0u;
                    constexpr uint32_t kOther = (uint32_t(kSegSlots) * kSegBytes) >> 4;   // from a segment of A to the same rows of B
                    for (int q = 0; q < L.n_grp; ++q) {
#pragma unroll
                        for (int kk = 0; kk < kBK / 16; ++kk) {
                            if (kSyr2k) {   // A_x B_y^T, then B_x A_y^T into the same accumulator
                                tc_mma<kKind>(d_addr[q], desc_hi | uint64_t(a_lo[q] + st_off + kk_step * kk),
                                              desc_hi | uint64_t(b_lo[q] + kOther + st_off + kk_step * kk), idesc[q],
                                              (kk > 0) ? 1u : first);
                                tc_mma<kKind>(d_addr[q], desc_hi | uint64_t(a_lo[q] + kOther + st_off + kk_step * kk),
                                              desc_hi | uint64_t(b_lo[q] + st_off + kk_step * kk), idesc[q], 1u);
                            } else {
                                tc_mma<kKind>(d_addr[q], desc_hi | uint64_t(a_lo[q] + st_off + kk_step * kk),
                                              desc_hi | uint64_t(b_lo[q] + st_off + kk_step * kk), idesc[q],
                                              (kk > 0) ? 1u : first);
                            }
                        }
                    }
                    tc_commit(&empty_bar[st]);    // stage reusable once these MMAs have read it
                }
                if (!ok) break;
                tc_commit(tmem_full_bar);         // accumulators complete
            }
            if (s_abort) {                        // let issued MMAs finish before TMEM is freed
                volatile int dummy = 0;
                tc_commit(drain_bar);
                mbar_wait_bounded(drain_bar, 0, &dummy);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------ epilogue ------------------------------
        const int quarter = warp & 3;                     // TMEM lanes this warp may read
        const int row_in_tile = quarter * 32 + lane;
        uint8_t* my_staging = staging + (warp - 2) * 2 * kStageBufBytes;
        uint32_t n_done = 0, n_stores = 0;
        for (int64_t w = w_first; w < w_last && !s_abort; w += w_stride, ++n_done) {
            const Unit u = unit_of(w, n_items, n_ksteps, split, n_batch);
            const WorkItem* it = &items[u.item];
            const int n_tile = it->n_tile;
            Layout L;
            layout_of(it, n_tile, (n_done & 1) ? 3u * kTile : 0u, L);
            int64_t trow[kMaxTiles], tcol[kMaxTiles];
            for (int t = 0; t < kMaxTiles; ++t) {
                trow[t] = (t < n_tile) ? it->seg[it->tile_x[t]] : 0;
                tcol[t] = (t < n_tile) ? it->seg[it->tile_y[t]] : 0;
            }
            const int64_t slot0 = (split > 1) ? tile_base[u.item] : 0;
            float* Cb = (u.batch > 0) ? C + int64_t(u.batch) * c_batch_stride : C;     // this unit's matrix
            if (!mbar_wait_bounded(tmem_full_bar, n_done & 1, &s_abort)) {
                s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitMma); break;
            }
            tc_fence_after();
            for (int pass = 0; pass < 2; ++pass) {        // the N = 256 pair first, then the lone tile
                for (int t = 0; t < n_tile; ++t) {
                    if (L.tile_in_pair[t] != (pass == 0)) continue;
                    const int64_t r = trow[t] * kTile + row_in_tile;
                    const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + L.tile_col[t];
                    const bool staged = tma_store_ok && split == 1 && beta == 0.f && trow[t] != tcol[t] &&
                                        trow[t] * kTile + quarter * 32 < N;
#pragma unroll 1
                    for (int cb = 0; cb < kTile; cb += 32) {
                        uint32_t v[32];
                        tmem_ld_32x32(taddr + cb, v);
                        if (split > 1) {
                            float4* dst = reinterpret_cast<float4*>(
                                partial + ((int64_t(u.slice) * total_tiles + slot0 + t) * kTile + row_in_tile) * kTile + cb);
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                     __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                            continue;
                        }
                        const int64_t c0 = tcol[t] * kTile + cb;
                        if (staged) {
                            // 32 x 32 block -> swizzled staging buffer -> asynchronous TMA store
                            uint8_t* buf = my_staging + (n_stores & 1) * kStageBufBytes;
                            if (lane == 0) tma_store_wait_read_1();   // the store that last used `buf` has read it
                            __syncwarp();
#pragma unroll
                            for (int j = 0; j < 8; ++j)
                                *reinterpret_cast<float4*>(buf + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                    make_float4(alpha * __uint_as_float(v[4 * j]), alpha * __uint_as_float(v[4 * j + 1]),
                                                alpha * __uint_as_float(v[4 * j + 2]), alpha * __uint_as_float(v[4 * j + 3]));
                            fence_async_smem();
                            __syncwarp();
                            if (lane == 0) {
                                if (u.batch < 0) tma_store_2d(&tmC, buf, int32_t(c0), int32_t(trow[t] * kTile + quarter * 32));
                                else tma_store_3d(&tmC, buf, int32_t(c0), int32_t(trow[t] * kTile + quarter * 32), u.batch);
                            }
                            ++n_stores;
                            continue;
                        }
                        if (r >= N) continue;
                        float* crow = Cb + r * ldc + c0;
                        // entries this row keeps: columns <= r (lower form) or r .. N-1 (upper form)
                        const bool whole = kUpper ? (c0 >= r && c0 + 31 < N) : (c0 + 31 <= r);
                        if (whole && vec_ok) {
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                float4 o = make_float4(alpha * __uint_as_float(v[4 * j]), alpha * __uint_as_float(v[4 * j + 1]),
                                                       alpha * __uint_as_float(v[4 * j + 2]), alpha * __uint_as_float(v[4 * j + 3]));
                                float4* p = reinterpret_cast<float4*>(crow) + j;
                                if (beta != 0.f) {
                                    const float4 old = *p;
                                    o.x += beta * old.x; o.y += beta * old.y; o.z += beta * old.z; o.w += beta * old.w;
                                }
                                *p = o;
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                if (kUpper ? (c0 + j >= r && c0 + j < N) : (c0 + j <= r)) {
                                    float o = alpha * __uint_as_float(v[j]);
                                    if (beta != 0.f) o += beta * crow[j];
                                    crow[j] = o;
                                }
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(pass == 0 ? pair_free_bar : &single_free_bar[n_done & 1]);
            }
        }
        if (lane == 0) tma_store_wait_all();              // staged tiles are in global memory
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// Sum of the K-slices' partial tiles in slice order, then alpha/beta and the triangle mask
// (col <= row, or col >= row for the upper form).
__global__ void __launch_bounds__(256)
splitk_reduce_kernel(const WorkItem* __restrict__ items, const int64_t* __restrict__ tile_base,
                     int64_t total_tiles, int32_t split, const float* __restrict__ partial, int64_t N,
                     float* __restrict__ C, int64_t ldc, float alpha, float beta, int upper) {
    const WorkItem* it = &items[blockIdx.x];
    const int t = blockIdx.y;
    if (t >= it->n_tile) return;
    const int64_t slot = tile_base[blockIdx.x] + t;
    const int64_t row0 = int64_t(it->seg[it->tile_x[t]]) * kTile, col0 = int64_t(it->seg[it->tile_y[t]]) * kTile;
    for (int e = threadIdx.x; e < kTile * kTile / 4; e += blockDim.x) {
        const int rr = e / (kTile / 4), cc = (e % (kTile / 4)) * 4;
        const int64_t r = row0 + rr;
        if (r >= N) continue;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sl = 0; sl < split; ++sl) {
            const float4 p = *reinterpret_cast<const float4*>(
                partial + ((int64_t(sl) * total_tiles + slot) * kTile + rr) * kTile + cc);
            s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
        }
        const float vals[4] = {s.x, s.y, s.z, s.w};
        float* crow = C + r * ldc + col0 + cc;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t c = col0 + cc + j;
            if (upper ? (c >= r && c < N) : (c <= r)) {
                float o = alpha * vals[j];
                if (beta != 0.f) o += beta * crow[j];
                crow[j] = o;
            }
        }
    }
}

// The instantiation for an input kind, a storage order of A and a stored triangle of C.
using KernelFn = void (*)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const WorkItem*, int64_t, int64_t, int32_t,
                          float*, int64_t, float, float, int, int, int32_t, float*, const int64_t*, int64_t, const int64_t*, int*,
                          int32_t, int64_t);
template <int kKind>
KernelFn kernel_of_kind(int tn, int upper) {
    return tn ? (upper ? syrk_bf16_tbs_kernel<true, kKind, true> : syrk_bf16_tbs_kernel<true, kKind, false>)
              : (upper ? syrk_bf16_tbs_kernel<false, kKind, true> : syrk_bf16_tbs_kernel<false, kKind, false>);
}
KernelFn kernel_for(int kind, int tn, int upper) {
    switch (kind) {
        case kKindTF32: return kernel_of_kind<kKindTF32>(tn, upper);
        case kKindE4M3: return kernel_of_kind<kKindE4M3>(tn, upper);
        case kKindF16: return kernel_of_kind<kKindF16>(tn, upper);
        default: return kernel_of_kind<kKindBF16>(tn, upper);
    }
}
KernelFn syr2k_kernel_for(int kind) {
    switch (kind) {
        case kKindTF32: return syrk_bf16_tbs_kernel<false, kKindTF32, false, true>;
        case kKindE4M3: return syrk_bf16_tbs_kernel<false, kKindE4M3, false, true>;
        case kKindF16: return syrk_bf16_tbs_kernel<false, kKindF16, false, true>;
        default: return syrk_bf16_tbs_kernel<false, kKindBF16, false, true>;
    }
}

}  // namespace bf16

cudaError_t launch_syrk_bf16(const CUtensorMap& tmA, const CUtensorMap* tmC, const WorkItem* d_items,
                             int64_t n_items, int64_t N, int64_t M, float* C, int64_t ldc, float alpha,
                             float beta, int split_k, float* d_partial, const int64_t* d_tile_base,
                             int64_t total_tiles, const int64_t* d_cta_begin, int n_ctas, int a_is_m_by_n,
                             int a_kind, int* d_status, int sm_count, cudaStream_t stream, int64_t batch,
                             int64_t c_batch_stride, int upper, const CUtensorMap* tmB) {
    // The shared-memory attribute belongs to a device's context: set it once per device.
    static bool configured[64] = {};
    static std::mutex configured_mu;                 // launchers are reached under different locks
    std::lock_guard<std::mutex> configured_lock(configured_mu);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return cudaErrorInvalidDevice;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        const void* kernels[20];
        for (int i = 0; i < 16; ++i) kernels[i] = reinterpret_cast<const void*>(bf16::kernel_for(i >> 2, (i >> 1) & 1, i & 1));
        for (int i = 0; i < 4; ++i) kernels[16 + i] = reinterpret_cast<const void*>(bf16::syr2k_kernel_for(i));
        for (const void* fn : kernels) {
            cudaError_t e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, bf16::kSmemBytes);
            if (e != cudaSuccess) return e;
        }
        configured[dev] = true;
    }
    if (n_items == 0) return cudaSuccess;
    const bool two_byte = a_kind == bf16::kKindBF16 || a_kind == bf16::kKindF16;
    if (a_kind < 0 || a_kind > 3) return cudaErrorInvalidValue;   // no such kernel
    const int bk = two_byte ? 64 : (a_kind == bf16::kKindTF32 ? 32 : 128);
    const int32_t n_ksteps = int32_t((M + bk - 1) / bk);
    const int split = split_k < 1 ? 1 : (split_k > n_ksteps ? n_ksteps : split_k);
    if (batch > 0 && (split != 1 || upper || batch >= (int64_t(1) << 31))) return cudaErrorInvalidValue;
    if (tmB != nullptr && (a_is_m_by_n || upper || batch > 0)) return cudaErrorInvalidValue;   // rank-2k: N x M operands, lower triangle
    const int64_t n_units = n_items * split * (batch > 0 ? batch : 1);
    const bool ranges = (d_cta_begin != nullptr && split == 1 && n_ctas > 0 && batch <= 0);
    const unsigned grid = ranges ? unsigned(n_ctas) : unsigned(n_units < sm_count ? n_units : sm_count);
    const int vec_ok = ((reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 3) == 0 &&
                        (batch <= 0 || (c_batch_stride & 3) == 0)) ? 1 : 0;
    CUtensorMap none{};
    auto kernel = tmB ? bf16::syr2k_kernel_for(a_kind) : bf16::kernel_for(a_kind, a_is_m_by_n, upper);
    kernel<<<grid, bf16::kThreads, bf16::kSmemBytes, stream>>>(
        tmA, tmB ? *tmB : none, tmC ? *tmC : none, d_items, n_items, N, n_ksteps, C, ldc, alpha, beta, vec_ok, tmC ? 1 : 0, split,
        d_partial, d_tile_base, total_tiles, ranges ? d_cta_begin : nullptr, d_status, int32_t(batch > 0 ? batch : 0),
        c_batch_stride);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || split == 1) return e;
    bf16::splitk_reduce_kernel<<<dim3(unsigned(n_items), bf16::kMaxTiles), 256, 0, stream>>>(
        d_items, d_tile_base, total_tiles, split, d_partial, N, C, ldc, alpha, beta, upper);
    return cudaGetLastError();
}

int bf16_tile() { return bf16::kTile; }
int bf16_bk() { return bf16::kBK; }
int bf16_stages() { return bf16::kStages; }
int bf16_seg_slots() { return bf16::kSegSlots; }
int bf16_store_box() { return bf16::kStoreBox; }

}  // namespace tbsyrk
