// Square-block comparison kernel on CTA pairs (tcgen05 cta_group::2) for the tcgen05 input types
// (bfloat16, binary16, binary32 read as TF32, FP8 E4M3; a stage row is 128 bytes for all of them).
//
// The triangle-block kernel (syrk_bf16.cu) is bound by shared-memory traffic: one SM feeds both
// MMA operands from its own shared memory.  A CTA pair halves the N-operand traffic: the pair
// computes a 256 x 256 block of C (tile rows X0, X1 against tile rows Y0, Y1, all strictly below
// the diagonal) with one M = 256, N = 256 MMA per K = 16, each CTA staging 128 rows of the
// M-operand (its own X) and 128 rows of the N-operand (its own Y); the tensor cores of both SMs read
// the N-operand halves of both.  This shape does not fit triangle blocks (a pair shares its
// N-operand; the left-over pairs of a triangle block have none in common), so the kernel runs the
// square-block schedule of the paper's comparison algorithm (Section 5, the blocks of the generic
// out-of-core scheme of Algorithm 3): 256 x 256 squares, those on the diagonal included (a quarter of
// such a block is computed in vain; they are one block in sixty-odd at the sizes this schedule is for).
//
// Per CTA: warp 0 = TMA producer (2 loads of 16 KB per stage, 6 stages, completion counted on the
// LEADER CTA's full barrier), warp 1 = TMEM allocation (both CTAs) and, in the leader CTA (cluster
// rank 0), the MMA issuer for the pair, warps 2-5 = epilogue of the CTA's own 128 x 256 half.
// TMEM holds two accumulator stages of 256 columns, so a block's write-out overlaps the next
// block's MMAs completely.  No multicast loads anywhere; tcgen05.commit multicasts the barrier
// arrivals to both CTAs.
#include "device_utils.cuh"
#include "kernels.h"

namespace tbsyrk {
namespace pair {

constexpr int kTile = 128;
constexpr int kStages = 6;
constexpr int kSegBytes = kTile * 128;             // 128 rows of 128 bytes: 64 two-byte, 32 binary32 or 128 FP8 columns
constexpr int kStageBytes = 2 * kSegBytes;         // own X rows + own Y rows
constexpr int kThreads = 192;
constexpr int kStoreBox = 32;
constexpr int kStageBufBytes = kStoreBox * kStoreBox * 4;
constexpr int kStagingBytes = 4 * 2 * kStageBufBytes;
constexpr int kSmemBytes = kStages * kStageBytes + kStagingBytes + 1024 + 256;
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;                      // one accumulator stage: 128 lanes x 256 columns

__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Shared::cluster address of `local` (a shared::cta address of this CTA) in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(local), "r"(rank));
    return a;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void remote_arrive(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void remote_arrive_expect_tx(uint32_t cluster_addr, uint32_t bytes) {
    // default semantics (not release at cluster scope: that fence costs about a microsecond per stage and the
    // bytes are counted by the copies themselves)
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(cluster_addr), "r"(bytes) : "memory");
}
// TMA tile load of this CTA whose completion is counted on a barrier of the pair's leader CTA.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* tmap, int32_t x, int32_t y,
                                                 uint32_t leader_bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(leader_bar)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t* smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_dst)), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Arrive on the barrier at the same shared-memory offset in both CTAs of the pair once the MMAs
// issued so far have completed.
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(mask) : "memory");
}
// Input kinds as in the triangle-block kernel: 0 bfloat16, 1 TF32, 2 FP8 E4M3, 3 binary16.
template <int kKind>
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    if (kKind == 1)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    else if (kKind == 2)
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    else
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
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
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {   // K-major, 128-byte swizzle, 8-row groups 1024 B apart
    uint64_t d = 0;
    d |= uint64_t((addr & 0x3FFFF) >> 4);
    d |= uint64_t(1024 >> 4) << 32;
    d |= uint64_t(1) << 46;
    d |= uint64_t(2) << 61;
    return d;
}
// Instruction descriptor for the pair: D = FP32, A = B = format code `fmt` (kind::f16: 1 bfloat16, 0 binary16;
// kind::tf32: 2; kind::f8f6f4: 0 = E4M3), both K-major, N = 256, M = 256 (128 rows per CTA).
__device__ __forceinline__ uint32_t instr_desc_pair(uint32_t fmt) {
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* tmap, const void* smem_src, int32_t x, int32_t y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(smem_src)) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
__device__ __forceinline__ void tma_store_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// blocks[i] = {X0, X1, Y0, Y1}: tile rows of the 256 x 256 block i, below the diagonal (X0 > Y1) or on it
// (X = Y: the two diagonal tiles are stored with the triangle mask, the tile above the diagonal is
// computed but not stored).  The pair with index p runs blocks p, p + pairs, p + 2 pairs, ...
template <int kKind>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
syrk_pair_square_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmC,
                        const int4* __restrict__ blocks, int32_t n_blocks, int64_t N, int32_t n_ksteps,
                        float* __restrict__ C, int64_t ldc, float alpha, float beta, int vec_ok, int tma_store_ok,
                        uint32_t fmt, int* __restrict__ status, int32_t split, float* __restrict__ partial) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* staging = smem + kStages * kStageBytes;
    uint64_t* full_bar = reinterpret_cast<uint64_t*>(staging + kStagingBytes);   // used in the leader CTA
    uint64_t* empty_bar = full_bar + kStages;                                     // one per CTA
    uint64_t* tmem_full_bar = empty_bar + kStages;                                // [2], one set per CTA
    uint64_t* tmem_empty_bar = tmem_full_bar + 2;                                 // [2], used in the leader CTA
    uint64_t* drain_bar = tmem_empty_bar + 2;
    __shared__ uint32_t s_tmem_base;
    __shared__ volatile int s_abort;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kCols = kKind == 1 ? 32 : (kKind == 2 ? 128 : 64);   // columns of A in a 128-byte stage row
    const uint32_t rank = cluster_rank();                  // 0 = leader of the pair
    const int32_t pair_id = int32_t(blockIdx.x >> 1), n_pairs = int32_t(gridDim.x >> 1);
    // Units: (block, K-slice) pairs, slice-major (split == 1: the blocks themselves).  Unit w is block
    // w % n_blocks restricted to K-steps [n_ksteps * s / split, n_ksteps * (s + 1) / split), s = w / n_blocks.
    const int32_t n_units = n_blocks * split;

    if (tid == 0) {
        s_abort = 0;
        for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 2); mbar_init(&empty_bar[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tmem_full_bar[a], 1); mbar_init(&tmem_empty_bar[a], 8); }
        mbar_init(drain_bar, 1);
        mbar_fence_init();
    }
    __syncthreads();
    if (warp == 1) tmem_alloc2(&s_tmem_base, kTmemCols);   // the same warp of both CTAs
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                    // barriers of both CTAs are initialised, TMEM is allocated
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;

    if (warp == 0) {
        // ------------------------------ producer (each CTA) ------------------------------
        if (lane == 0) {
            prefetch_tensormap(&tmA);
            uint32_t g = 0;
            for (int32_t w = pair_id; w < n_units && !s_abort; w += n_pairs) {
                const int4 blk = blocks[w % n_blocks];
                const int32_t sl = w / n_blocks;
                const int32_t k0 = int32_t(int64_t(n_ksteps) * sl / split), k1 = int32_t(int64_t(n_ksteps) * (sl + 1) / split);
                const int32_t row_x = (rank == 0 ? blk.x : blk.y) * kTile;       // this CTA's M-operand rows
                const int32_t row_y = (rank == 0 ? blk.z : blk.w) * kTile;       // this CTA's half of the N-operand
                for (int ks = k0; ks < k1; ++ks, ++g) {
                    const uint32_t st = g % kStages;
                    if (g >= kStages && !mbar_wait_bounded(&empty_bar[st], ((g / kStages) - 1) & 1, &s_abort)) {
                        s_abort = 1; atomicOr(status, kStatusWaitEmpty); break;
                    }
                    const uint32_t leader_full = map_to_cta(smem_u32(&full_bar[st]), 0);
                    remote_arrive_expect_tx(leader_full, uint32_t(kStageBytes));
                    uint8_t* dst = smem + st * kStageBytes;
                    tma_load_2d_pair(dst, &tmA, ks * kCols, row_x, leader_full);
                    tma_load_2d_pair(dst + kSegBytes, &tmA, ks * kCols, row_y, leader_full);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------ MMA issuer (leader CTA only) ------------------------------
        if (lane == 0 && rank == 0) {
            uint32_t g = 0, n_done = 0;
            const uint32_t smem_base = smem_u32(smem);
            const uint64_t desc_hi = smem_desc_sw128(0);
            const uint32_t idesc = instr_desc_pair(fmt);
            for (int32_t w = pair_id; w < n_units && !s_abort; w += n_pairs, ++n_done) {
                const int32_t sl = w / n_blocks;
                const int32_t k0 = int32_t(int64_t(n_ksteps) * sl / split), k1 = int32_t(int64_t(n_ksteps) * (sl + 1) / split);
                const uint32_t acc = n_done & 1;
                if (n_done >= 2 && !mbar_wait_bounded(&tmem_empty_bar[acc], ((n_done >> 1) - 1) & 1, &s_abort)) {
                    s_abort = 1; atomicOr(status, kStatusWaitTmem); break;
                }
                tc_fence_after();
                const uint32_t d_addr = tmem_base + acc * kAccCols;
                bool ok = true;
                for (int ks = k0; ks < k1; ++ks, ++g) {
                    const uint32_t st = g % kStages;
                    if (!mbar_wait_bounded(&full_bar[st], (g / kStages) & 1, &s_abort)) {
                        s_abort = 1; atomicOr(status, kStatusWaitFull); ok = false; break;
                    }
                    tc_fence_after();
                    const uint32_t a_lo = (smem_base + st * kStageBytes) >> 4, b_lo = a_lo + (kSegBytes >> 4);
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)            // 32 bytes of K per instruction for every kind
                        tc_mma_pair<kKind>(d_addr, desc_hi | uint64_t(a_lo + 2 * kk), desc_hi | uint64_t(b_lo + 2 * kk), idesc,
                                    (kk > 0 || ks > k0) ? 1u : 0u);
                    tc_commit_pair(&empty_bar[st]);          // both CTAs may refill the stage
                }
                if (!ok) break;
                tc_commit_pair(&tmem_full_bar[acc]);         // both halves of the accumulator are complete
            }
            if (s_abort) {                                   // let issued MMAs finish before TMEM is freed
                volatile int dummy = 0;
                tc_commit_pair(drain_bar);
                mbar_wait_bounded(drain_bar, 0, &dummy);
            }
        }
        __syncwarp();
    } else {
        // ------------------------------ epilogue (each CTA: its 128 rows x 256 columns) ------------------------------
        const int quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        uint8_t* my_staging = staging + (warp - 2) * 2 * kStageBufBytes;
        uint32_t n_done = 0, n_stores = 0;
        for (int32_t w = pair_id; w < n_units && !s_abort; w += n_pairs, ++n_done) {
            const int32_t b = w % n_blocks, sl = w / n_blocks;
            const int4 blk = blocks[b];
            const uint32_t acc = n_done & 1;
            const int64_t trow = rank == 0 ? blk.x : blk.y;
            if (!mbar_wait_bounded(&tmem_full_bar[acc], (n_done >> 1) & 1, &s_abort)) {
                s_abort = 1; if (lane == 0) atomicOr(status, kStatusWaitMma); break;
            }
            tc_fence_after();
            const int64_t r = trow * kTile + row_in_tile;
            for (int t = 0; t < 2; ++t) {
                const int64_t tcol = t == 0 ? blk.z : blk.w;
                const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + acc * kAccCols + uint32_t(t) * kTile;
                if (tcol > trow) continue;                          // diagonal block: the tile above the diagonal is not stored
                const bool on_diag = tcol == trow;
                const bool staged = tma_store_ok && split == 1 && !on_diag && beta == 0.f && trow * kTile + quarter * 32 < N;
                // K-split: raw partial tile (slice, block, rank, t), 128 x 128 binary32
                float* part = split > 1 ? partial + (((int64_t(sl) * n_blocks + b) * 4 + int64_t(rank) * 2 + t) * kTile + row_in_tile) * kTile
                                        : nullptr;
#pragma unroll 1
                for (int cb = 0; cb < kTile; cb += 32) {
                    uint32_t v[32];
                    tmem_ld_32x32(taddr + cb, v);
                    if (split > 1) {
                        float4* dst = reinterpret_cast<float4*>(part + cb);
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            dst[j] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]),
                                                 __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
                        continue;
                    }
                    const int64_t c0 = tcol * kTile + cb;
                    if (staged) {
                        uint8_t* buf = my_staging + (n_stores & 1) * kStageBufBytes;
                        if (lane == 0) tma_store_wait_read_1();
                        __syncwarp();
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<float4*>(buf + lane * 128 + ((j ^ (lane & 7)) << 4)) =
                                make_float4(alpha * __uint_as_float(v[4 * j]), alpha * __uint_as_float(v[4 * j + 1]),
                                            alpha * __uint_as_float(v[4 * j + 2]), alpha * __uint_as_float(v[4 * j + 3]));
                        fence_async_smem();
                        __syncwarp();
                        if (lane == 0) tma_store_2d(&tmC, buf, int32_t(c0), int32_t(trow * kTile + quarter * 32));
                        ++n_stores;
                        continue;
                    }
                    if (r >= N) continue;
                    float* crow = C + r * ldc + c0;                  // below the diagonal every column is kept
                    if (on_diag && c0 + 31 > r) {                    // diagonal tile: columns <= row only
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            if (c0 + j <= r) {
                                float o = alpha * __uint_as_float(v[j]);
                                if (beta != 0.f) o += beta * crow[j];
                                crow[j] = o;
                            }
                        }
                    } else if (vec_ok) {
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
                            float o = alpha * __uint_as_float(v[j]);
                            if (beta != 0.f) o += beta * crow[j];
                            crow[j] = o;
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) remote_arrive(map_to_cta(smem_u32(&tmem_empty_bar[acc]), 0));   // this warp's half is drained
        }
        if (lane == 0) tma_store_wait_all();
        __syncwarp();
    }

    // Both CTAs stay until the other is done with their shared memory and barriers.
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc2(tmem_base, kTmemCols);
    }
}

// K-split calls: stored entries of tile (rank, t) of block blockIdx.x <- alpha * (sum of the slices' partial
// tiles, in slice order) + beta * C.
__global__ void __launch_bounds__(256)
pair_splitk_reduce_kernel(const int4* __restrict__ blocks, int32_t n_blocks, int32_t split, const float* __restrict__ partial,
                          int64_t N, float* __restrict__ C, int64_t ldc, float alpha, float beta) {
    const int4 blk = blocks[blockIdx.x];
    const int rank = blockIdx.y >> 1, t = blockIdx.y & 1;
    const int64_t trow = rank == 0 ? blk.x : blk.y, tcol = t == 0 ? blk.z : blk.w;
    if (tcol > trow) return;
    for (int e = threadIdx.x; e < kTile * kTile / 4; e += blockDim.x) {
        const int rr = e / (kTile / 4), cc = (e % (kTile / 4)) * 4;
        const int64_t r = trow * kTile + rr;
        if (r >= N) continue;
        float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int sl = 0; sl < split; ++sl) {
            const float4 p = *reinterpret_cast<const float4*>(
                partial + (((int64_t(sl) * n_blocks + blockIdx.x) * 4 + blockIdx.y) * kTile + rr) * kTile + cc);
            s.x += p.x; s.y += p.y; s.z += p.z; s.w += p.w;
        }
        const float vals[4] = {s.x, s.y, s.z, s.w};
        float* crow = C + r * ldc + tcol * kTile + cc;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (tcol * kTile + cc + j <= r) {
                float o = alpha * vals[j];
                if (beta != 0.f) o += beta * crow[j];
                crow[j] = o;
            }
        }
    }
}

}  // namespace pair

namespace {
template <int kKind>
cudaError_t launch_pair_kind(const CUtensorMap& tmA, const CUtensorMap* tmC, const int4* d_blocks, int32_t n_blocks, int64_t N,
                             int32_t n_ksteps, float* C, int64_t ldc, float alpha, float beta, int vec_ok, uint32_t fmt,
                             int* d_status, int pairs, int split, float* d_partial, cudaStream_t stream) {
    static bool configured[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (!configured[dev]) {
        cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void*>(&pair::syrk_pair_square_kernel<kKind>),
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, pair::kSmemBytes);
        if (e != cudaSuccess) return e;
        configured[dev] = true;
    }
    CUtensorMap none{};
    pair::syrk_pair_square_kernel<kKind><<<dim3(unsigned(2 * pairs)), pair::kThreads, pair::kSmemBytes, stream>>>(
        tmA, tmC ? *tmC : none, d_blocks, n_blocks, N, n_ksteps, C, ldc, alpha, beta, vec_ok, tmC ? 1 : 0, fmt, d_status,
        split, d_partial);
    return cudaGetLastError();
}
}  // namespace

cudaError_t launch_syrk_pair_square(const CUtensorMap& tmA, const CUtensorMap* tmC, const int4* d_blocks, int32_t n_blocks,
                                    int64_t N, int64_t M, float* C, int64_t ldc, float alpha, float beta, int a_kind,
                                    int* d_status, int sm_count, cudaStream_t stream, int split_k, float* d_partial) {
    if (n_blocks <= 0) return cudaSuccess;
    if (a_kind < 0 || a_kind > 3) return cudaErrorInvalidValue;
    const int cols = a_kind == 1 ? 32 : (a_kind == 2 ? 128 : 64);
    const int32_t n_ksteps = int32_t((M + cols - 1) / cols);
    const int split = (split_k < 1 || d_partial == nullptr) ? 1 : (split_k > n_ksteps ? n_ksteps : split_k);
    int pairs = sm_count / 2;
    if (int64_t(pairs) > int64_t(n_blocks) * split) pairs = n_blocks * split;
    const int vec_ok = ((reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 3) == 0) ? 1 : 0;
    const uint32_t fmt = a_kind == 0 ? 1u : (a_kind == 1 ? 2u : 0u);
    cudaError_t e;
    if (a_kind == 1) e = launch_pair_kind<1>(tmA, tmC, d_blocks, n_blocks, N, n_ksteps, C, ldc, alpha, beta, vec_ok, fmt, d_status, pairs, split, d_partial, stream);
    else if (a_kind == 2) e = launch_pair_kind<2>(tmA, tmC, d_blocks, n_blocks, N, n_ksteps, C, ldc, alpha, beta, vec_ok, fmt, d_status, pairs, split, d_partial, stream);
    else e = launch_pair_kind<0>(tmA, tmC, d_blocks, n_blocks, N, n_ksteps, C, ldc, alpha, beta, vec_ok, fmt, d_status, pairs, split, d_partial, stream);
    if (e != cudaSuccess || split == 1) return e;
    pair::pair_splitk_reduce_kernel<<<dim3(unsigned(n_blocks), 4), 256, 0, stream>>>(d_blocks, n_blocks, split, d_partial, N, C,
                                                                                     ldc, alpha, beta);
    return cudaGetLastError();
}

}  // namespace tbsyrk
