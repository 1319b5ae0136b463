// syrk_lower_bf16_static: the K-split BF16 path for callers that must not allocate.
//
// Some callers of this library cannot let it call cudaMalloc: code running between
// other libraries' pool allocations that must not see the device heap move, services
// that pin the device memory budget at start-up, or a latency-critical loop where an
// allocation (an implicit device synchronisation) is not acceptable.  The regular
// entry point creates its work list and K-split workspace with cudaMalloc on first
// use; this variant keeps both in fixed arrays that are part of the library image,
// so every GPU that loads the library holds them (about 34 MiB) until the process
// exits.
//
// It runs the same two kernels as syrk_lower does for a K-split BF16 call (the
// tcgen05 kernel writing one partial tile set per K-slice, then the fixed-order
// reduction), with the workspace, the work list and the status word taken from the
// arrays below.  All calls share these arrays: the work list is rewritten and the
// partial tiles are overwritten by every call (nothing has to start at zero), so
// two calls whose GPU work overlaps - different streams, or different host
// threads - race and must be serialised by the caller.
#include <algorithm>
#include <cstring>
#include <mutex>
#include <vector>

#include "../../include/tbsyrk.h"
#include "kernels.h"
#include "runtime.h"

namespace {

using namespace tbsyrk;

constexpr int64_t kStaticMaxItems = 1024;                       // work items (80 bytes each)
constexpr int64_t kStaticMaxSliceTiles = SYRK_STATIC_MAX_SLICE_TILES;   // slices x 128x128 output tiles
constexpr int64_t kTileFloats = 128 * 128;

// The scratch itself.  In host code these names are only stand-ins for the device
// symbols; their device addresses are fetched once per device with
// cudaGetSymbolAddress (below) and only those addresses are handed to kernels.
static __device__ __align__(256) float g_static_partial[kStaticMaxSliceTiles * kTileFloats];
static __device__ __align__(256) unsigned char g_static_items[kStaticMaxItems * sizeof(WorkItem)];
static __device__ __align__(256) long long g_static_tile_base[kStaticMaxItems + 1];
static __device__ __align__(256) int g_static_status[64];

struct StaticAddrs {
    bool ready = false;
    float* partial = nullptr;
    WorkItem* items = nullptr;
    int64_t* tile_base = nullptr;
    int* status = nullptr;
    int sm_count = 0;
    int64_t uploaded_tiles = -1;    // tile rows of the work list the device arrays hold (-1: none yet)
};

std::mutex g_mu;
StaticAddrs g_addrs[64];   // per device ordinal
// Host copies of the work list and of its tile offsets, the source of the upload: fixed storage that
// outlives the call (the copy engine may read it after the call has returned).  Guarded by g_mu.
WorkItem g_host_items[kStaticMaxItems];
int64_t g_host_tile_base[kStaticMaxItems + 1];

// Set-up, once per device, with that device current: resolve the device addresses of
// the arrays above.  Happens inside the first call on a device.
int setup_device(int dev, StaticAddrs** out) {
    if (dev < 0 || dev >= 64) return SYRK_ERR_NO_DEVICE;
    StaticAddrs& a = g_addrs[dev];
    if (!a.ready) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&a.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            cudaGetLastError();
            return SYRK_ERR_NO_DEVICE;
        }
        if (major != 10) return SYRK_ERR_NO_DEVICE;
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_partial) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
        a.partial = static_cast<float*>(p);
        if (cudaGetSymbolAddress(&p, g_static_items) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
        a.items = static_cast<WorkItem*>(p);
        if (cudaGetSymbolAddress(&p, g_static_tile_base) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
        a.tile_base = static_cast<int64_t*>(p);
        if (cudaGetSymbolAddress(&p, g_static_status) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
        a.status = static_cast<int*>(p);
        a.ready = true;
    }
    *out = &a;
    return SYRK_OK;
}

}  // namespace

extern "C" int syrk_lower_bf16_static(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc,
                                      double alpha, double beta, int slices, void* stream) {
    if (N < 0 || M < 0 || N >= (int64_t(1) << 31) - 256 || M >= (int64_t(1) << 31) - 256) return SYRK_ERR_SIZE;
    if (slices < 2) return SYRK_ERR_SIZE;
    if (N == 0) return SYRK_OK;
    if (lda < (M > 1 ? M : 1) || ldc < N) return SYRK_ERR_LD;
    if (!A || !C) return SYRK_ERR_NULL;
    if (M == 0 || alpha == 0.0) return SYRK_ERR_SIZE;                 // nothing to split: use syrk_lower
    if ((reinterpret_cast<uintptr_t>(A) & 15) != 0 || (lda * 2) % 16 != 0) return SYRK_ERR_LD;   // TMA rules

    const int64_t n_ksteps = (M + bf16_bk() - 1) / bf16_bk();
    if (slices > n_ksteps) return SYRK_ERR_SIZE;
    const int64_t n_tiles = (N + bf16_tile() - 1) / bf16_tile();
    // every output tile belongs to exactly one item, so the list has n_tiles (n_tiles + 1) / 2 tiles
    if (n_tiles * (n_tiles + 1) / 2 * slices > kStaticMaxSliceTiles) return SYRK_ERR_STATIC_LIMIT;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // The call copies its work list from host memory and shares device arrays with every other call:
    // neither belongs in a captured graph, which would replay both at times of its own.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
    if (cap != cudaStreamCaptureStatusNone) return SYRK_ERR_CUDA;

    std::lock_guard<std::mutex> lock(g_mu);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_NO_DEVICE; }
    StaticAddrs* a = nullptr;
    int rc = setup_device(dev, &a);
    if (rc != SYRK_OK) return rc;

    // Host-side work list (the same generator and ordering as the regular path); it depends on the
    // number of tile rows only, so a call that finds the device arrays holding that list already
    // uploads nothing.
    int64_t n_items = 0, total_tiles = 0;
    {
        Plan plan;
        if (!build_host_plan(N, SYRK_DTYPE_BF16_F32, SYRK_SCHEDULE_TBS, &plan)) return SYRK_ERR_PLAN;
        n_items = int64_t(plan.items.size());
        if (n_items > kStaticMaxItems) return SYRK_ERR_STATIC_LIMIT;
        if (!items_fit_kernel(plan.items, SYRK_DTYPE_BF16_F32)) return SYRK_ERR_PLAN;   // the kernel does not check items
        for (int64_t i = 0; i < n_items; ++i) total_tiles += plan.items[size_t(i)].n_tile;
        if (total_tiles * slices > kStaticMaxSliceTiles) return SYRK_ERR_STATIC_LIMIT;   // workspace beyond the fixed array
        if (a->uploaded_tiles != n_tiles) {
            g_host_tile_base[0] = 0;
            for (int64_t i = 0; i < n_items; ++i) {
                g_host_items[i] = plan.items[size_t(i)];
                g_host_tile_base[i + 1] = g_host_tile_base[i] + plan.items[size_t(i)].n_tile;
            }
        }
    }
    if (a->uploaded_tiles != n_tiles) {
        // The work list travels on the caller's stream, ahead of the kernels that read it.
        a->uploaded_tiles = -1;
        if (cudaMemcpyAsync(a->items, g_host_items, size_t(n_items) * sizeof(WorkItem), cudaMemcpyHostToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(a->tile_base, g_host_tile_base, (size_t(n_items) + 1) * sizeof(int64_t), cudaMemcpyHostToDevice, st) != cudaSuccess) {
            cudaGetLastError();
            return SYRK_ERR_CUDA;
        }
        // The copies above are from pageable memory: the runtime has staged them before returning,
        // so the host arrays may be rewritten by the next call.
        a->uploaded_tiles = n_tiles;
    }
    CUtensorMap tm;
    rc = encode_tensor_map_2d(&tm, SYRK_DTYPE_BF16_F32, A, N, M, lda, bf16_tile(), bf16_bk());
    if (rc != SYRK_OK) return rc;
    const cudaError_t e = launch_syrk_bf16(tm, nullptr, a->items, n_items, N, M, static_cast<float*>(C), ldc,
                                           float(alpha), float(beta), slices, a->partial, a->tile_base,
                                           total_tiles, nullptr, 0, 0, 0, a->status, a->sm_count, st);
    return e == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}

extern "C" int syrk_lower_bf16_static_status(void) {
    std::lock_guard<std::mutex> lock(g_mu);
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_NO_DEVICE; }
    if (dev < 0 || dev >= 64) return SYRK_ERR_NO_DEVICE;
    const StaticAddrs& a = g_addrs[dev];
    if (!a.ready) return SYRK_OK;                                    // no call on this device yet
    int flag = 0;
    if (cudaMemcpy(&flag, a.status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
    if (flag == 0) return SYRK_OK;
    if (cudaMemset(a.status, 0, sizeof(int)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
    return SYRK_ERR_DEVICE_WAIT;
}
