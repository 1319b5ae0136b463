// Small sm_100a building blocks shared by the kernels: mbarrier, TMA tile loads,
// bounded waits.  Every wait in this library has an iteration/time limit; when it
// runs out the waiter records an error and the kernel winds down instead of
// spinning forever.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_runtime.h>

namespace tbsyrk {

// Error bits written to the device status word.
constexpr int kStatusWaitFull = 1;    // consumer gave up waiting for a TMA stage
constexpr int kStatusWaitEmpty = 2;   // producer gave up waiting for a free stage
constexpr int kStatusWaitMma = 4;     // epilogue gave up waiting for the tensor core
constexpr int kStatusWaitTmem = 8;    // MMA issuer gave up waiting for a drained accumulator
constexpr int kStatusBadItem = 16;    // a work item failed its bounds check

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Wait for a phase of `bar` with a limit of about two seconds.  `abort_flag` is a
// shared-memory word that any role of the thread block raises when it gives up,
// so that the others stop waiting too.  Returns false when the wait was abandoned.
constexpr uint64_t kWaitLimitNs = 2000000000ull;

__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity,
                                                  volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0x3FFu) == 0) {
            if (*abort_flag != 0) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) return false;
        }
    }
    return true;
}

// 2-D tiled TMA load (no multicast): box at element coordinates (x = column,
// y = row) of the tensor map into shared memory, completion counted in bytes on
// `bar`.  x * element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* tmap, int32_t x,
                                            int32_t y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y),
          "r"(smem_u32(bar))
        : "memory");
}

// The same for a 3-D tensor map whose outermost coordinate z selects one matrix of a strided
// batch (box depth 1): the box lands in shared memory exactly as a 2-D box would.
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* tmap, int32_t x,
                                            int32_t y, int32_t z, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes "
        "[%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z),
          "r"(smem_u32(bar))
        : "memory");
}

// Box load from a 2-D map (z < 0) or from matrix z of a batched 3-D map.
__device__ __forceinline__ void tma_load_box(void* smem_dst, const CUtensorMap* tmap, int32_t x,
                                             int32_t y, int32_t z, uint64_t* bar) {
    if (z < 0) tma_load_2d(smem_dst, tmap, x, y, bar);
    else tma_load_3d(smem_dst, tmap, x, y, z, bar);
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* tmap) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(tmap)) : "memory");
}

}  // namespace tbsyrk
