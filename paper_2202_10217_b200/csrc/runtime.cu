// Host-side runtime: device state, work-list cache, TMA descriptors.
#include "runtime.h"

#include <cstdio>
#include <cstdlib>
#include <algorithm>
#include <vector>

#include "../../include/tbsyrk.h"
#include "kernels.h"

namespace tbsyrk {

Runtime& runtime() {
    static Runtime r;
    return r;
}

KernelShape kernel_shape(int dtype) {
    KernelShape s{};
    if (dtype == SYRK_DTYPE_F64) {
        // 32-row segments; k = 6 gives 15 of the 16 accumulator tiles a block can hold.
        s.tile = f64_tile(); s.k = 6; s.rect_rows = 4; s.rect_cols = 4; s.diag_side = 4;
        s.bk = f64_bk(); s.stages = f64_stages();
        s.s_acc = int64_t(16) * s.tile * s.tile;
    } else {
        // 128-row segments, three per pipeline stage and three 128 x 128 FP32 accumulators in
        // TMEM: a triangle block with k = 3, or a 1 x 2 rectangle, or two diagonal tile rows.
        // A stage row is 128 bytes: 64 bfloat16, 32 binary32 (TF32) or 128 FP8 columns.
        s.tile = bf16_tile(); s.k = 3; s.rect_rows = 1; s.rect_cols = 2; s.diag_side = 2;
        s.bk = 128 / int(a_elem_size(dtype)); s.stages = bf16_stages();
        s.s_acc = int64_t(3) * s.tile * s.tile;
    }
    return s;
}

bool build_host_plan(int64_t N, int dtype, int schedule, Plan* out, int upper) {
    const KernelShape ks = kernel_shape(dtype);
    PlanParams p;
    p.n_tiles = (N + ks.tile - 1) / ks.tile;
    p.k = ks.k;
    // The upper-triangle form runs the mirror image of a lower-triangle list: a rectangle of r x c
    // tiles below the diagonal becomes one of c x r above it, so the list is built with the
    // rectangle's sides exchanged (the tcgen05 kernel wants one M-operand and two adjacent N-operands).
    p.rect_rows = upper ? ks.rect_cols : ks.rect_rows;
    p.rect_cols = upper ? ks.rect_rows : ks.rect_cols;
    if (upper && ks.diag_side < p.rect_rows) return false;
    p.diag_side = ks.diag_side;
    p.schedule = schedule;
    if (!build_plan(p, out)) return false;
    // FP64: one thread block per item, dispatched in list order, heaviest first (no rectangles are
    // cut into quarters for the last round: measured over a dozen shapes, the four-tile items that
    // gives keep a quarter of the MMA warps busy and cost 0-4 % more than they even out); the
    // tcgen05 kernel is persistent and deals items to blocks by a cost model, heaviest first.
    if (dtype == SYRK_DTYPE_F64) balance_for_slots(out, 0);
    else std::stable_sort(out->items.begin(), out->items.end(),
                          [](const WorkItem& a, const WorkItem& b) { return a.n_tile > b.n_tile; });
    if (upper) {
        for (WorkItem& it : out->items) {
            for (int t = 0; t < it.n_tile; ++t) std::swap(it.tile_x[t], it.tile_y[t]);     // tile (x, y) -> (y, x)
            if (dtype != SYRK_DTYPE_F64) {
                // tcgen05 layout: tiles with the same M-operand and adjacent N-operands must follow each other
                for (int a = 1; a < it.n_tile; ++a)
                    for (int b = a; b > 0 && (it.tile_x[b] < it.tile_x[b - 1] ||
                                              (it.tile_x[b] == it.tile_x[b - 1] && it.tile_y[b] < it.tile_y[b - 1])); --b) {
                        std::swap(it.tile_x[b], it.tile_x[b - 1]);
                        std::swap(it.tile_y[b], it.tile_y[b - 1]);
                    }
            }
        }
    }
    return true;
}

int get_device_state(DeviceState** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_NO_DEVICE; }
    Runtime& rt = runtime();
    auto it = rt.devices.find(dev);
    if (it == rt.devices.end()) {
        DeviceState ds;
        ds.device = dev;
        cudaDeviceProp prop;
        if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_NO_DEVICE; }
        ds.sm_count = prop.multiProcessorCount;
        ds.cc_major = prop.major;
        if (prop.major != 10) return SYRK_ERR_NO_DEVICE;  // kernels are built for sm_100a only
        if (cudaMalloc(&ds.d_status, (kStreamSlots + 1) * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_ALLOC; }
        if (cudaMemset(ds.d_status, 0, (kStreamSlots + 1) * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
        if (cudaMalloc(&ds.d_tickets, 2 * kStreamSlots * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_ALLOC; }
        if (cudaMemset(ds.d_tickets, 0, 2 * kStreamSlots * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_CUDA; }
        ds.workspaces.resize(kStreamSlots);
        it = rt.devices.emplace(dev, std::move(ds)).first;
    }
    *out = &it->second;
    return SYRK_OK;
}

int slot_for_stream(DeviceState* ds, cudaStream_t stream) {
    auto it = ds->stream_slot.find(stream);
    if (it == ds->stream_slot.end()) {
        if (int(ds->stream_slot.size()) >= kStreamSlots) return -1;
        it = ds->stream_slot.emplace(stream, int(ds->stream_slot.size())).first;
    }
    return it->second;
}

int* status_for_stream(DeviceState* ds, cudaStream_t stream) {
    const int slot = slot_for_stream(ds, stream);
    return ds->d_status + (slot >= 0 ? slot : kStreamSlots);
}

namespace {
bool stream_is_capturing(cudaStream_t stream) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) != cudaSuccess) { cudaGetLastError(); return true; }   // be careful
    return cap != cudaStreamCaptureStatusNone;
}
}  // namespace

int* tickets_for_stream(DeviceState* ds, cudaStream_t stream) {
    if (stream_is_capturing(stream)) return nullptr;
    const int slot = slot_for_stream(ds, stream);
    return slot >= 0 ? ds->d_tickets + 2 * slot : nullptr;
}

int workspace_for_stream(DeviceState* ds, cudaStream_t stream, size_t want, void** out) {
    const int slot = slot_for_stream(ds, stream);
    if (slot < 0) return SYRK_ERR_ALLOC;
    StreamWorkspace& ws = ds->workspaces[size_t(slot)];
    if (ws.bytes < want || !ws.d_partial) {
        if (stream_is_capturing(stream)) return SYRK_ERR_ALLOC;
        const int rc = ensure_device_bytes(&ws.d_partial, &ws.bytes, want);
        if (rc != SYRK_OK) return rc;
    }
    *out = ws.d_partial;
    return SYRK_OK;
}

int read_and_clear_status(DeviceState* ds, cudaStream_t stream, bool all) {
    int words[kStreamSlots + 1];
    const int first = all ? 0 : int(status_for_stream(ds, stream) - ds->d_status);
    const int count = all ? kStreamSlots + 1 : 1;
    if (cudaMemcpy(words, ds->d_status + first, size_t(count) * sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) {
        cudaGetLastError();
        return SYRK_ERR_CUDA;
    }
    int flag = 0;
    for (int i = 0; i < count; ++i) flag |= words[i];
    if (flag == 0) return SYRK_OK;
    cudaMemset(ds->d_status + first, 0, size_t(count) * sizeof(int));
    return SYRK_ERR_DEVICE_WAIT;
}

bool items_fit_kernel(const std::vector<WorkItem>& items, int dtype) {
    const int max_seg = (dtype == SYRK_DTYPE_F64) ? kMaxSeg : bf16_seg_slots();
    const int max_tile = (dtype == SYRK_DTYPE_F64) ? kMaxTile : 3;
    for (const WorkItem& it : items) {
        if (it.n_seg < 1 || it.n_tile < 1 || it.n_seg > max_seg || it.n_tile > max_tile) return false;
        for (int t = 0; t < it.n_tile; ++t)
            if (it.tile_x[t] >= it.n_seg || it.tile_y[t] >= it.n_seg) return false;
        if (is_tcgen05_dtype(dtype)) {   // TMEM layout: at most one lone tile and one adjacent pair
            int lone = 0, pairs = 0;
            for (int t = 0; t < it.n_tile;) {
                const bool pair = t + 1 < it.n_tile && it.tile_x[t + 1] == it.tile_x[t] &&
                                  it.tile_y[t + 1] == it.tile_y[t] + 1;
                pair ? ++pairs : ++lone;
                t += pair ? 2 : 1;
            }
            if (lone > 1 || pairs > 1) return false;
        }
    }
    return true;
}

int get_device_plan(DeviceState* ds, int64_t N, int dtype, DevicePlan** out, int upper) {
    const KernelShape ks = kernel_shape(dtype);
    const int64_t n_tiles = (N + ks.tile - 1) / ks.tile;
    const auto key = std::make_tuple(n_tiles, dtype, runtime().schedule + (upper ? 16 : 0));
    auto it = ds->plans.find(key);
    if (it == ds->plans.end()) {
        DevicePlan dp;
        if (!build_host_plan(N, dtype, runtime().schedule, &dp.plan, upper)) return SYRK_ERR_PLAN;
        if (!items_fit_kernel(dp.plan.items, dtype)) return SYRK_ERR_PLAN;
        std::vector<int64_t> cta_begin;
        if (is_tcgen05_dtype(dtype) && !dp.plan.items.empty()) {
            // Persistent kernel: items go to thread blocks (one per SM) longest first, each to the
            // block with the least work so far.  The kernel is bound by shared-memory traffic, so
            // an item costs, per K-step, 16 KB per segment written by TMA plus the operand reads of
            // its MMAs (16 KB for the M-operand and 16 KB per 128 columns of N), and about 600 KB
            // worth of time per tile for the write-out.  K-steps are not known here; 64 (M = 4096)
            // weighs the two terms.
            const int n_ctas = int(std::min<size_t>(dp.plan.items.size(), size_t(ds->sm_count)));
            auto cost = [](const WorkItem& it) {
                int64_t kb = 16 * it.n_seg;
                for (int t = 0; t < it.n_tile;) {
                    const bool pair = t + 1 < it.n_tile && it.tile_x[t + 1] == it.tile_x[t] &&
                                      it.tile_y[t + 1] == it.tile_y[t] + 1;
                    kb += pair ? 48 : 32;
                    t += pair ? 2 : 1;
                }
                return 64 * kb + 600 * int64_t(it.n_tile);
            };
            std::vector<WorkItem> sorted = dp.plan.items;
            std::stable_sort(sorted.begin(), sorted.end(),
                             [&](const WorkItem& a, const WorkItem& b) { return cost(a) > cost(b); });
            std::vector<std::vector<WorkItem>> per_block(static_cast<size_t>(n_ctas));
            std::vector<int64_t> load(size_t(n_ctas), 0);
            for (const WorkItem& it : sorted) {
                const size_t b = size_t(std::min_element(load.begin(), load.end()) - load.begin());
                per_block[b].push_back(it);
                load[b] += cost(it);
            }
            dp.plan.items.clear();
            cta_begin.push_back(0);
            for (int b = 0; b < n_ctas; ++b) {
                dp.plan.items.insert(dp.plan.items.end(), per_block[size_t(b)].begin(), per_block[size_t(b)].end());
                cta_begin.push_back(int64_t(dp.plan.items.size()));
            }
            dp.n_ctas = n_ctas;
        }
        const size_t n = dp.plan.items.size();
        std::vector<int64_t> base(n + 1, 0);
        for (size_t i = 0; i < n; ++i) base[i + 1] = base[i] + dp.plan.items[i].n_tile;
        dp.total_tiles = base[n];
        if (n > 0) {
            if (cudaMalloc(&dp.d_items, n * sizeof(WorkItem)) != cudaSuccess ||
                cudaMalloc(&dp.d_tile_base, (n + 1) * sizeof(int64_t)) != cudaSuccess) {
                cudaGetLastError();
                if (dp.d_items) cudaFree(dp.d_items);
                return SYRK_ERR_ALLOC;
            }
            if (cudaMemcpy(dp.d_items, dp.plan.items.data(), n * sizeof(WorkItem), cudaMemcpyHostToDevice) != cudaSuccess ||
                cudaMemcpy(dp.d_tile_base, base.data(), (n + 1) * sizeof(int64_t), cudaMemcpyHostToDevice) != cudaSuccess) {
                cudaGetLastError();
                cudaFree(dp.d_items); cudaFree(dp.d_tile_base);
                return SYRK_ERR_CUDA;
            }
        }
        if (!cta_begin.empty()) {
            if (cudaMalloc(&dp.d_cta_begin, cta_begin.size() * sizeof(int64_t)) != cudaSuccess) {
                cudaGetLastError(); cudaFree(dp.d_items); cudaFree(dp.d_tile_base); return SYRK_ERR_ALLOC;
            }
            if (cudaMemcpy(dp.d_cta_begin, cta_begin.data(), cta_begin.size() * sizeof(int64_t), cudaMemcpyHostToDevice) != cudaSuccess) {
                cudaGetLastError(); cudaFree(dp.d_items); cudaFree(dp.d_tile_base); cudaFree(dp.d_cta_begin); return SYRK_ERR_CUDA;
            }
        }
        it = ds->plans.emplace(key, std::move(dp)).first;
    }
    *out = &it->second;
    return SYRK_OK;
}

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            p = nullptr;
        }
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}
}  // namespace

int encode_tensor_map_2d(CUtensorMap* tm, int dtype, const void* A, int64_t N, int64_t M,
                         int64_t lda, int box_rows, int box_cols, int swizzle_atom_32b) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SYRK_ERR_CUDA;
    const size_t es = a_elem_size(dtype);
    const cuuint64_t dims[2] = {cuuint64_t(M), cuuint64_t(N)};
    const cuuint64_t strides[1] = {cuuint64_t(lda) * es};
    const cuuint32_t box[2] = {cuuint32_t(box_cols), cuuint32_t(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    // TF32 operands travel as plain binary32 (bits untouched; the tensor core ignores the low 13).
    const CUtensorMapDataType dt =
        (dtype == SYRK_DTYPE_F64) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT64
        : (dtype == SYRK_DTYPE_TF32_F32) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
        : (dtype == SYRK_DTYPE_E4M3_F32) ? CU_TENSOR_MAP_DATA_TYPE_UINT8
        : (dtype == SYRK_DTYPE_F16_F32) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult r = fn(tm, dt, 2, const_cast<void*>(A), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE,
                          swizzle_atom_32b ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SYRK_OK : SYRK_ERR_CUDA;
}

int encode_tensor_map_c_f32(CUtensorMap* tm, const void* C, int64_t N, int64_t ldc, int box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SYRK_ERR_CUDA;
    const cuuint64_t dims[2] = {cuuint64_t(N), cuuint64_t(N)};
    const cuuint64_t strides[1] = {cuuint64_t(ldc) * 4};
    const cuuint32_t bx[2] = {cuuint32_t(box), cuuint32_t(box)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(C), dims, strides, bx, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SYRK_OK : SYRK_ERR_CUDA;
}

// Strided batch: a third dimension of `batch` matrices `stride` elements apart (box depth 1).
int encode_tensor_map_batched(CUtensorMap* tm, int dtype, const void* A, int64_t N, int64_t M, int64_t lda,
                              int64_t stride, int64_t batch, int box_rows, int box_cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SYRK_ERR_CUDA;
    const size_t es = a_elem_size(dtype);
    const cuuint64_t dims[3] = {cuuint64_t(M), cuuint64_t(N), cuuint64_t(batch)};
    const cuuint64_t strides[2] = {cuuint64_t(lda) * es, cuuint64_t(stride) * es};
    const cuuint32_t box[3] = {cuuint32_t(box_cols), cuuint32_t(box_rows), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUtensorMapDataType dt =
        (dtype == SYRK_DTYPE_F64) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT64
        : (dtype == SYRK_DTYPE_TF32_F32) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32
        : (dtype == SYRK_DTYPE_E4M3_F32) ? CU_TENSOR_MAP_DATA_TYPE_UINT8
        : (dtype == SYRK_DTYPE_F16_F32) ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    const CUresult r = fn(tm, dt, 3, const_cast<void*>(A), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SYRK_OK : SYRK_ERR_CUDA;
}

// C of a strided batch: square boxes of `box` elements, 128-byte swizzle for binary32 (the store
// path of the tcgen05 kernel), none for binary64 (old-C tiles of the FP64 kernel).
int encode_tensor_map_c_batched(CUtensorMap* tm, int is_f64, const void* C, int64_t N, int64_t ldc,
                                int64_t stride, int64_t batch, int box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SYRK_ERR_CUDA;
    const size_t es = is_f64 ? 8 : 4;
    const cuuint64_t dims[3] = {cuuint64_t(N), cuuint64_t(N), cuuint64_t(batch)};
    const cuuint64_t strides[2] = {cuuint64_t(ldc) * es, cuuint64_t(stride) * es};
    const cuuint32_t bx[3] = {cuuint32_t(box), cuuint32_t(box), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(tm, is_f64 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT64 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3,
                          const_cast<void*>(C), dims, strides, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                          is_f64 ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B,
                          is_f64 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SYRK_OK : SYRK_ERR_CUDA;
}

int encode_tensor_map_f64_plain(CUtensorMap* tm, const void* p, int64_t rows, int64_t cols, int64_t ld,
                                int box_rows, int box_cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SYRK_ERR_CUDA;
    const cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(ld) * 8};
    const cuuint32_t bx[2] = {cuuint32_t(box_cols), cuuint32_t(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 2, const_cast<void*>(p), dims, strides, bx, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SYRK_OK : SYRK_ERR_CUDA;
}

int encode_tensor_map_c_f64(CUtensorMap* tm, const void* C, int64_t N, int64_t ldc, int box) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return SYRK_ERR_CUDA;
    const cuuint64_t dims[2] = {cuuint64_t(N), cuuint64_t(N)};
    const cuuint64_t strides[1] = {cuuint64_t(ldc) * 8};
    const cuuint32_t bx[2] = {cuuint32_t(box), cuuint32_t(box)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT64, 2, const_cast<void*>(C), dims, strides, bx, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? SYRK_OK : SYRK_ERR_CUDA;
}

int ensure_device_bytes(void** p, size_t* have, size_t want) {
    if (*have >= want && *p) return SYRK_OK;
    if (*p) { cudaFree(*p); *p = nullptr; *have = 0; }
    if (cudaMalloc(p, want) != cudaSuccess) { cudaGetLastError(); *p = nullptr; return SYRK_ERR_ALLOC; }
    *have = want;
    return SYRK_OK;
}

int ensure_pinned_bytes(void** p, size_t* have, size_t want) {
    if (*have >= want && *p) return SYRK_OK;
    if (*p) { cudaFreeHost(*p); *p = nullptr; *have = 0; }
    if (cudaMallocHost(p, want) != cudaSuccess) { cudaGetLastError(); *p = nullptr; return SYRK_ERR_ALLOC; }
    *have = want;
    return SYRK_OK;
}

void release_all() {
    release_cholesky_workspaces();
    Runtime& rt = runtime();
    int prev = -1;
    cudaGetDevice(&prev);
    for (auto& kv : rt.devices) {
        DeviceState& ds = kv.second;
        cudaSetDevice(ds.device);
        for (auto& pk : ds.plans) {
            if (pk.second.d_items) cudaFree(pk.second.d_items);
            if (pk.second.d_tile_base) cudaFree(pk.second.d_tile_base);
            if (pk.second.d_cta_begin) cudaFree(pk.second.d_cta_begin);
        }
        for (auto& pp : ds.pair_plans) {
            if (pp.second.d_blocks) cudaFree(pp.second.d_blocks);
        }
        if (ds.d_status) cudaFree(ds.d_status);
        if (ds.d_tickets) cudaFree(ds.d_tickets);
        for (StreamWorkspace& ws : ds.workspaces) if (ws.d_partial) cudaFree(ws.d_partial);
        if (ds.d_a) cudaFree(ds.d_a);
        if (ds.d_c) cudaFree(ds.d_c);
        if (ds.d_packed) cudaFree(ds.d_packed);
        if (ds.h_packed) cudaFreeHost(ds.h_packed);
        if (ds.host_stream) cudaStreamDestroy(ds.host_stream);
        if (ds.copy_stream) cudaStreamDestroy(ds.copy_stream);
        if (ds.down_stream) cudaStreamDestroy(ds.down_stream);
        for (cudaStream_t bs : ds.band_streams) if (bs) cudaStreamDestroy(bs);
        for (auto& bk : ds.banded) if (bk.second.d_items) cudaFree(bk.second.d_items);
        for (cudaEvent_t ev : ds.host_events) if (ev) cudaEventDestroy(ev);
    }
    rt.devices.clear();
    if (prev >= 0) cudaSetDevice(prev);
    cudaGetLastError();
}

}  // namespace tbsyrk
