// Host-side runtime of the library: per-device state, the cache of device-resident
// work lists, TMA descriptor encoding.  Internal.
#pragma once
#include <cstdint>
#include <map>
#include <mutex>
#include <tuple>
#include <utility>
#include <vector>

#include <cuda.h>
#include <cuda_runtime.h>

#include "tbs_plan.h"

namespace tbsyrk {

// Schedule parameters per dtype (tile side b, block side k, leftover shapes).
struct KernelShape {
    int tile;        // b
    int k;           // segments per triangle block
    int rect_rows, rect_cols, diag_side;
    int bk, stages;  // staging: columns per stage, pipeline depth
    int64_t s_acc;   // accumulator elements a thread block may hold
};
KernelShape kernel_shape(int dtype);
// Element sizes of A and C, and whether the dtype runs on the tcgen05 kernel (BF16, TF32 or FP8 inputs).
inline size_t a_elem_size(int dtype) { return dtype == 0 ? 8 : ((dtype == 1 || dtype == 4) ? 2 : (dtype == 2 ? 4 : 1)); }
inline size_t c_elem_size(int dtype) { return dtype == 0 ? 8 : 4; }
inline bool is_tcgen05_dtype(int dtype) { return dtype >= 1 && dtype <= 4; }
inline bool known_dtype(int dtype) { return dtype >= 0 && dtype <= 4; }

struct DevicePlan {
    Plan plan;
    WorkItem* d_items = nullptr;
    int64_t* d_tile_base = nullptr;  // first output-tile slot of each item (K-split workspace)
    int64_t total_tiles = 0;
    int64_t* d_cta_begin = nullptr;  // BF16: first item of each persistent thread block (n_ctas + 1)
    int n_ctas = 0;
    std::map<int64_t, int> auto_split;   // tcgen05: modelled number of K-slices by inner dimension (the model
                                         // walks every unit of every candidate: too slow to redo on every call)
    std::map<int64_t, std::pair<int64_t, int>> tail_split;   // FP64: (first tail item, slices) by number of K-steps
};

// Square-block work list in row order for the host-buffer entry point: band j owns the rows
// [j * band_rows, (j + 1) * band_rows) of C and the items [item_end[j-1], item_end[j]).
struct BandedPlan {
    std::vector<WorkItem> items;
    WorkItem* d_items = nullptr;
    int64_t band_rows = 0;
    std::vector<int64_t> item_end;
};

// Work list of the CTA-pair square-block schedule: the 256 x 256 blocks below and on the diagonal.
struct PairPlan {
    int4* d_blocks = nullptr;
    int32_t n_blocks = 0;
};

// K-split workspace of one stream slot (grow-only).
struct StreamWorkspace {
    void* d_partial = nullptr;
    size_t bytes = 0;
};

struct DeviceState {
    int device = -1;
    int sm_count = 0;
    int cc_major = 0;
    // Per-stream state.  Work enqueued on one stream runs in order, so it can share a status word,
    // a K-split workspace and a ticket pair; work on different streams may overlap on the GPU and
    // must not.  Every stream the library sees gets a slot (first come, kStreamSlots per device).
    // d_status holds one word per slot plus a last one shared by the streams that found no slot.
    int* d_status = nullptr;
    // FP64 persistent launches: a pair of tickets per slot.
    int* d_tickets = nullptr;
    std::map<cudaStream_t, int> stream_slot;
    std::vector<StreamWorkspace> workspaces;   // K-split partial tiles, by slot
    std::map<int64_t, PairPlan> pair_plans;   // by number of tile rows
    // staging for the host-buffer entry point (grow-only)
    void* d_a = nullptr; size_t d_a_bytes = 0;
    void* d_c = nullptr; size_t d_c_bytes = 0;
    void* d_packed = nullptr; size_t d_packed_bytes = 0;
    void* h_packed = nullptr; size_t h_packed_bytes = 0;
    cudaStream_t host_stream = nullptr;      // compute stream of the host-buffer entry point
    cudaStream_t copy_stream = nullptr;      // its upload stream
    cudaStream_t down_stream = nullptr;      // its download stream
    cudaStream_t band_streams[4] = {};       // its compute streams when C is produced band by band
    cudaEvent_t host_events[48] = {};        // block-landed / band-computed / band-packed events of that entry point
    std::map<std::pair<int64_t, int>, BandedPlan> banded;  // (n_tiles, dtype)
    std::map<std::tuple<int64_t, int, int>, DevicePlan> plans;  // (n_tiles, dtype, schedule)
};

struct Runtime {
    std::mutex mu;
    std::map<int, DeviceState> devices;
    int schedule = 0;
    bool pair_square = false;   // SYRK_SCHEDULE_PAIR_SQUARE: square blocks, CTA-pair kernel where it applies
    bool auto_pair = true;      // SYRK_SCHEDULE_AUTO (default): triangle blocks, but the pair kernel for short work lists
    int split_k = 0;
    int f64_launch = 0;
    int host_pipeline = 0;      // syrk_set_host_pipeline
    int f64_tail_slices = 0;    // syrk_set_f64_tail_split: 0 automatic, 1 off, >= 2 forced
    int64_t f64_tail_items = 0; //   forced number of tail items
};
constexpr int kStreamSlots = 256;

// Slot of `stream` on this device (assigned on first sight), or -1 when all slots are taken.
int slot_for_stream(DeviceState* ds, cudaStream_t stream);
// The status word kernels launched on `stream` report to (the shared last word without a slot).
int* status_for_stream(DeviceState* ds, cudaStream_t stream);
// The ticket pair of `stream` on this device, or null when the persistent form must not be used
// (no slot left, or the stream is being captured into a graph, whose replays may overlap).
int* tickets_for_stream(DeviceState* ds, cudaStream_t stream);
// K-split workspace of at least `want` bytes for work enqueued on `stream`.  SYRK_ERR_ALLOC when the
// stream has no slot, when the allocation fails, or when the buffer would have to grow while the
// stream is being captured (growing frees the old buffer, which synchronises the device).
int workspace_for_stream(DeviceState* ds, cudaStream_t stream, size_t want, void** out);
// Reads and clears the status word of `stream`, or of every stream when `all` is set; the caller
// has synchronised.  Returns SYRK_OK, SYRK_ERR_DEVICE_WAIT or SYRK_ERR_CUDA.
int read_and_clear_status(DeviceState* ds, cudaStream_t stream, bool all);
Runtime& runtime();

// Current device's state, created on first use.  Returns a SYRK_* code.
int get_device_state(DeviceState** out);

// Plan for (N, dtype) under the current schedule, built and uploaded on first use.
int get_device_plan(DeviceState* ds, int64_t N, int dtype, DevicePlan** out, int upper = 0);

// Whether every item of a list can be run by the kernel of `dtype`: segment and tile counts, tile
// indices, and for the tcgen05 kernel its accumulator layout (at most one lone tile and one pair of
// tiles with the same M-operand and adjacent N-operands).  That kernel does not check items itself.
bool items_fit_kernel(const std::vector<WorkItem>& items, int dtype);

// Host-only plan (no device).
bool build_host_plan(int64_t N, int dtype, int schedule, Plan* out, int upper = 0);

// 2-D row-major tensor map over A (N x M, pitch lda elements) with a box of
// box_rows x box_cols elements and 128-byte swizzle (16-byte atoms, or 32-byte atoms with
// `swizzle_atom_32b`: the form MN-major binary32 operands of the tensor core need).
int encode_tensor_map_2d(CUtensorMap* tm, int dtype, const void* A, int64_t N, int64_t M,
                         int64_t lda, int box_rows, int box_cols, int swizzle_atom_32b = 0);

// 2-D row-major FP32 tensor map over C (N x N, pitch ldc) with box x box boxes, 128-byte swizzle.
int encode_tensor_map_batched(CUtensorMap* tm, int dtype, const void* A, int64_t N, int64_t M, int64_t lda,
                              int64_t stride, int64_t batch, int box_rows, int box_cols);
int encode_tensor_map_c_batched(CUtensorMap* tm, int is_f64, const void* C, int64_t N, int64_t ldc,
                                int64_t stride, int64_t batch, int box);
int encode_tensor_map_c_f32(CUtensorMap* tm, const void* C, int64_t N, int64_t ldc, int box);
// The same over an FP64 C, without swizzle (a box row of 32 doubles is 256 bytes).
int encode_tensor_map_c_f64(CUtensorMap* tm, const void* C, int64_t N, int64_t ldc, int box);

// Plain (unswizzled) FP64 tensor map over a rows x cols row-major matrix with pitch ld.
int encode_tensor_map_f64_plain(CUtensorMap* tm, const void* p, int64_t rows, int64_t cols, int64_t ld,
                                int box_rows, int box_cols);

// The device path of syrk_lower (arguments already validated; the caller holds the runtime lock).
// `f64_launch` >= 0 overrides the process-wide FP64 launch form for this call.  `a_is_m_by_n`: A is
// stored M x N row-major (pitch lda >= N) and the call computes alpha * A^T A + beta * C.
// `upper`: the entries with col >= row are updated instead of those with col <= row.
// `prepare_only`: take the call's decisions (schedule, K-split) and create what it would allocate (work
// lists, the stream's workspace) for an aligned operand, launch nothing; A and C are not looked at.
int syrk_run_device(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc, double alpha,
                    double beta, int dtype, cudaStream_t stream, int f64_launch = -1, int a_is_m_by_n = 0,
                    int upper = 0, bool prepare_only = false);

void release_cholesky_workspaces();

// Grow-only device / pinned-host buffers.
int ensure_device_bytes(void** p, size_t* have, size_t want);
int ensure_pinned_bytes(void** p, size_t* have, size_t want);

void release_all();

}  // namespace tbsyrk
