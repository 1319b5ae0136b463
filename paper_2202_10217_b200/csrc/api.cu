// C ABI of libtbsyrk.so (see include/tbsyrk.h for the contract of every call).
#include <algorithm>
#include <cmath>
#include <cstring>
#include <thread>
#include <vector>

#include "../../include/tbsyrk.h"
#include "kernels.h"
#include "runtime.h"

using namespace tbsyrk;

namespace {

int validate(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc, int dtype,
             bool a_is_m_by_n = false) {
    if (!known_dtype(dtype)) return SYRK_ERR_DTYPE;
    if (N < 0 || M < 0 || N >= (int64_t(1) << 31) - 256 || M >= (int64_t(1) << 31) - 256) return SYRK_ERR_SIZE;
    if (N == 0) return SYRK_OK;
    if (lda < std::max<int64_t>(1, a_is_m_by_n ? N : M) || ldc < N) return SYRK_ERR_LD;
    if (!C || (M > 0 && !A)) return SYRK_ERR_NULL;
    return SYRK_OK;
}

size_t a_elem(int dtype) { return a_elem_size(dtype); }
size_t c_elem(int dtype) { return c_elem_size(dtype); }

bool tma_ok(const void* A, int64_t lda, int dtype) {
    return (reinterpret_cast<uintptr_t>(A) & 15) == 0 && (size_t(lda) * a_elem(dtype)) % 16 == 0;
}

// K-slices for a BF16 call.  The persistent kernel deals its units (item x K-slice) round-robin
// to min(units, SMs) thread blocks; with few items the inner dimension is cut so that every SM
// has work.  The number of slices is the one with the smallest modelled makespan, in units of
// one 128 x 128 x 64 tile step: a unit costs tiles x its K-steps plus about 20 per tile for the
// write-out, and the reduction pass adds about 0.2 per partial tile.
int auto_split_k(const std::vector<WorkItem>& items, int64_t M, int bk, int sm_count, int forced) {
    const int64_t ksteps = (M + bk - 1) / bk;
    if (forced > 0) return int(std::max<int64_t>(1, std::min<int64_t>(forced, ksteps)));
    const int64_t n = int64_t(items.size());
    if (n == 0 || n >= 4 * int64_t(sm_count) || ksteps < 16) return 1;
    int64_t total_tiles = 0;
    for (const WorkItem& it : items) total_tiles += it.n_tile;
    int best = 1;
    double best_cost = 0.0;
    std::vector<double> load;
    for (int s = 1; s <= 32 && s <= ksteps / 8; ++s) {
        const int64_t units = n * s;
        const int64_t grid = std::min<int64_t>(units, sm_count);
        load.assign(size_t(grid), 0.0);
        for (int64_t w = 0; w < units; ++w) {
            const WorkItem& it = items[size_t(w % n)];
            const int64_t slice = w / n;
            const int64_t kk = ksteps * (slice + 1) / s - ksteps * slice / s;
            load[size_t(w % grid)] += double(it.n_tile) * double(kk + 20);
        }
        double cost = *std::max_element(load.begin(), load.end());
        if (s > 1) cost += 0.2 * double(s) * double(total_tiles) + 40.0;
        if (s == 1 || cost < best_cost) { best = s; best_cost = cost; }
    }
    return best;
}

// The automatic choice of the FP64 launch form.  Persistent blocks hide every item's start-up and write-out behind
// the next item's M loop (for beta == 0 and beta == 1, see the kernel) and take the tail K-split as the other form does.
// Measured on 2048 to 16384 rows and 256 to 8192 columns, they win or tie wherever the list has an item per SM; shorter
// lists run one block per (item, K-slice).
bool f64_persistent_pays(int64_t n_items, double beta, int sm_count) {
    return (beta == 0.0 || beta == 1.0) && n_items >= int64_t(sm_count);
}

// K-slices for an FP64 call (one block per item).  With fewer items than SMs the inner
// dimension is cut so that more blocks run at once; the slices' partial matrices are
// summed by a second kernel.  Model, in microseconds, fitted to measured calls of 512 to 1024 rows and 256 to
// 1024 columns under 1 to 16 slices: 4 for the launch; per round of blocks 4.3 plus 2.14 per K-step of a
// slice; for the reduction 3 plus 0.25 per slice and 512 x 512 entries.  A slice keeps at least 2 K-steps.
int auto_split_k_f64(int64_t n_items, int64_t N, int64_t M, int bk, int sm_count, int forced) {
    const int64_t ksteps = (M + bk - 1) / bk;
    if (forced > 0) return int(std::max<int64_t>(1, std::min<int64_t>(forced, ksteps)));
    if (n_items == 0 || n_items >= int64_t(sm_count) || ksteps < 4) return 1;
    int best = 1;
    double best_cost = 0.0;
    for (int s = 1; s <= 16 && s <= ksteps / 2; ++s) {
        if (s > 1 && double(s) * double(N) * double(N) * 8.0 > 512e6) break;        // workspace cap
        const int64_t rounds = (n_items * s + sm_count - 1) / sm_count;
        double cost = 4.0 + double(rounds) * (2.14 * double((ksteps + s - 1) / s) + 4.3);
        if (s > 1) cost += 3.0 + 0.25 * double(s) * double(N) * double(N) / (512.0 * 512.0);
        if (s == 1 || cost < best_cost) { best = s; best_cost = cost; }
    }
    return best;
}

// Tail K-split of an FP64 call in the one-block-per-item form.  The hardware hands the blocks to SMs in
// list order as SMs free up, so a call lasts as long as its most loaded SM; with long items (many K-steps)
// and a list of only a few rounds, the last round leaves SMs idle for up to an item's duration.  Cutting
// the last items along the inner dimension gives the last round smaller units.  This replays that
// dispatch for the whole list and for a few (number of tail items, slices) candidates with a cost model -
// an item takes 3 us plus, per K-step, 2.17 us times the share of the busiest of the SM's four DMMA pipes
// (16 tiles = 1), a slice 1 us more for its partial tiles; fitted to forty measured (shape, tail, slices)
// triples within 1 % - and returns the best candidate when it is modelled at least 1.5 % faster, else {n, 1}.
struct TailSplit { int64_t first; int slices; };
TailSplit plan_tail_split_f64(const std::vector<WorkItem>& items, int64_t ksteps, int sm_count) {
    const int64_t n = int64_t(items.size());
    TailSplit none{n, 1};
    if (n < sm_count || n > 16 * int64_t(sm_count) || ksteps < 64) return none;
    auto weight = [](const WorkItem& it) {
        if (it.kind == kTri && it.n_tile == 15) return 15.0 / 16.0;        // the 16th warp evens the pipes out
        return double((it.n_tile + 3) / 4) / 4.0;
    };
    constexpr double kFixedUs = 3.0, kStepUs = 2.17, kPartialUs = 1.0;
    std::vector<double> free_at;
    auto makespan = [&](int64_t first, int slices) {
        free_at.assign(size_t(sm_count), 0.0);
        std::make_heap(free_at.begin(), free_at.end(), std::greater<double>());
        double end = 0.0;
        auto run = [&](double cost) {
            std::pop_heap(free_at.begin(), free_at.end(), std::greater<double>());
            free_at.back() += cost;
            end = std::max(end, free_at.back());
            std::push_heap(free_at.begin(), free_at.end(), std::greater<double>());
        };
        for (int64_t i = 0; i < first; ++i) run(kFixedUs + kStepUs * double(ksteps) * weight(items[size_t(i)]));
        for (int64_t i = first; i < n; ++i)
            for (int sl = 0; sl < slices; ++sl) {
                const int64_t kk = ksteps * (sl + 1) / slices - ksteps * sl / slices;
                run(kFixedUs + kPartialUs + kStepUs * double(kk) * weight(items[size_t(i)]));
            }
        if (slices > 1) end += 5.0 + double(n - first) * double(slices) * 16.0 * 8192.0 / 4e6;   // the reduction pass
        return end;
    };
    const double whole = makespan(n, 1);
    TailSplit best = none;
    double best_t = whole;
    for (int slices = 2; slices <= 6 && ksteps / slices >= 16; ++slices)
        for (int64_t tail = sm_count / 4; tail <= 3 * int64_t(sm_count) && tail <= n; tail += sm_count / 4) {
            const double t = makespan(n - tail, slices);
            if (t < best_t) { best_t = t; best = TailSplit{n - tail, slices}; }
        }
    return best_t < 0.985 * whole ? best : none;
}

int pick_split_k(const DeviceState* ds, DevicePlan* dp, int64_t M, int bk) {
    if (runtime().split_k > 0) return auto_split_k(dp->plan.items, M, bk, ds->sm_count, runtime().split_k);
    auto it = dp->auto_split.find(M);
    if (it == dp->auto_split.end()) it = dp->auto_split.emplace(M, auto_split_k(dp->plan.items, M, bk, ds->sm_count, 0)).first;
    return it->second;
}

// One launch of the item kernels over a list (the whole plan, or the items of one band of rows).
int launch_items(DeviceState* ds, int dtype, const CUtensorMap& tm, const WorkItem* d_items, int64_t n_items,
                 int64_t N, int64_t M, void* C, int64_t ldc, double alpha, double beta, int split,
                 const int64_t* d_tile_base, int64_t total_tiles, const int64_t* d_cta_begin, int n_ctas,
                 int f64_launch, int a_is_m_by_n, cudaStream_t stream, int upper = 0, void* d_partial = nullptr,
                 int64_t tail_first = 0, int tail_slices = 1) {
    cudaError_t e;
    int* d_status = status_for_stream(ds, stream);
    if (dtype == SYRK_DTYPE_F64) {
        CUtensorMap tmc;
        const bool c_tma = beta != 0.0 && (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 1) == 0 &&
                           encode_tensor_map_c_f64(&tmc, C, N, ldc, f64_tile()) == SYRK_OK;
        // Persistent blocks hide each item's start-up and write-out behind the next item's M loop
        // (see f64_persistent_pays for when that is the faster form).
        const int mode = f64_launch >= 0 ? f64_launch : runtime().f64_launch;
        const bool persistent = mode == SYRK_F64_LAUNCH_PERSISTENT ||
                                (mode == SYRK_F64_LAUNCH_AUTO && f64_persistent_pays(n_items, beta, ds->sm_count));
        int* tickets = (persistent && split <= 1) ? tickets_for_stream(ds, stream) : nullptr;
        e = launch_syrk_f64(tm, c_tma ? &tmc : nullptr, d_items, n_items, N, M, static_cast<double*>(C), ldc,
                            alpha, beta, a_is_m_by_n, tickets, ds->sm_count, d_status, stream, 0, 0, split,
                            static_cast<double*>(d_partial), upper, tail_first, tail_slices);
    } else {
        CUtensorMap tmc;
        const bool c_tma = (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 3) == 0 &&
                           encode_tensor_map_c_f32(&tmc, C, N, ldc, bf16_store_box()) == SYRK_OK;
        e = launch_syrk_bf16(tm, c_tma ? &tmc : nullptr, d_items, n_items, N, M, static_cast<float*>(C), ldc, float(alpha),
                             float(beta), split, static_cast<float*>(d_partial), d_tile_base, total_tiles, d_cta_begin, n_ctas,
                             a_is_m_by_n, dtype - SYRK_DTYPE_BF16_F32, d_status, ds->sm_count, stream, 0, 0, upper);
    }
    return e == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}

// The row-ordered square-block list of (N, dtype), built and uploaded on first use.  Returns
// SYRK_ERR_PLAN when the list cannot be cut into bands (the caller then takes another path).
int get_banded_plan(DeviceState* ds, int64_t N, int dtype, int max_bands, BandedPlan** out) {
    const KernelShape ks = kernel_shape(dtype);
    const int64_t n_tiles = (N + ks.tile - 1) / ks.tile;
    auto key = std::make_pair(n_tiles, dtype);
    auto it = ds->banded.find(key);
    if (it == ds->banded.end()) {
        PlanParams p;
        p.n_tiles = n_tiles; p.k = ks.k; p.rect_rows = ks.rect_rows; p.rect_cols = ks.rect_cols;
        p.diag_side = ks.diag_side; p.schedule = SYRK_SCHEDULE_SQUARE;
        Plan plan;
        if (!build_plan(p, &plan) || plan.items.empty()) return SYRK_ERR_PLAN;
        // Items come strip by strip (diag_side tile rows each, top to bottom); a band is a whole
        // number of strips.
        const int64_t n_strips = (n_tiles + ks.diag_side - 1) / ks.diag_side;
        const int64_t n_bands = std::max<int64_t>(1, std::min<int64_t>(max_bands, n_strips));
        const int64_t strips_per_band = (n_strips + n_bands - 1) / n_bands;
        BandedPlan bp;
        bp.band_rows = strips_per_band * ks.diag_side * ks.tile;
        bp.items = plan.items;
        int64_t band = 0;
        for (size_t i = 0; i < bp.items.size(); ++i) {
            const WorkItem& w = bp.items[i];
            int64_t lo = INT64_MAX, hi = -1;
            for (int t = 0; t < w.n_tile; ++t) {
                lo = std::min<int64_t>(lo, w.seg[w.tile_x[t]]);
                hi = std::max<int64_t>(hi, w.seg[w.tile_x[t]]);
            }
            const int64_t b_lo = lo * ks.tile / bp.band_rows, b_hi = hi * ks.tile / bp.band_rows;
            if (b_lo != b_hi || b_hi < band) return SYRK_ERR_PLAN;      // straddles a boundary or out of order
            while (band < b_hi) { bp.item_end.push_back(int64_t(i)); ++band; }
        }
        bp.item_end.push_back(int64_t(bp.items.size()));
        if (cudaMalloc(&bp.d_items, bp.items.size() * sizeof(WorkItem)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_ALLOC; }
        if (cudaMemcpy(bp.d_items, bp.items.data(), bp.items.size() * sizeof(WorkItem), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaGetLastError(); cudaFree(bp.d_items); return SYRK_ERR_CUDA;
        }
        it = ds->banded.emplace(key, std::move(bp)).first;
    }
    *out = &it->second;
    return SYRK_OK;
}

}  // namespace

namespace {
// The CTA-pair square-block schedule for (N, M): number of 256 x 256 blocks and K-slices.  Returns false
// when the problem, even cut along the inner dimension, has fewer units than half the GPU's pairs (the
// caller then runs a single-CTA list).
bool pair_square_shape(int64_t N, int64_t M, int dtype, int sm_count, int forced_split, int64_t* n_blk_out, int* split_out) {
    const int tile = bf16_tile();
    const int64_t n_tiles = (N + tile - 1) / tile, n_super = (n_tiles + 1) / 2;
    const int64_t n_blk = n_super * (n_super + 1) / 2, pairs = sm_count / 2;
    const int64_t bk = 128 / int64_t(a_elem(dtype));              // columns in a 128-byte stage row
    const int64_t n_ksteps = (M + bk - 1) / bk;
    if (n_tiles >= (int64_t(1) << 15)) return false;
    // K-slices: with fewer blocks than a few rounds of pairs the inner dimension is cut so that every pair
    // has work; the number of slices minimises rounds x (K-steps per slice + 20) plus the partial traffic.
    int split = 1;
    if (forced_split > 0) split = int(std::max<int64_t>(1, std::min<int64_t>(forced_split, n_ksteps)));
    else if (n_blk < 4 * pairs) {
        double best = 0.0;
        for (int sp = 1; sp <= 32 && sp <= n_ksteps / 8; ++sp) {
            const int64_t rounds = (n_blk * sp + pairs - 1) / pairs;
            double cost = double(rounds) * (double((n_ksteps + sp - 1) / sp) + 20.0);
            if (sp > 1) cost += 0.1 * double(sp) * double(n_blk) * 2.0 + 40.0;
            if (sp == 1 || cost < best) { best = cost; split = sp; }
        }
    }
    if (2 * n_blk * split < pairs) return false;               // still fewer units than half the pairs
    *n_blk_out = n_blk;
    *split_out = split;
    return true;
}

// SYRK_SCHEDULE_PAIR_SQUARE for tcgen05-type operands stored N x M, lower triangle: the 256 x 256
// blocks below and on the diagonal on the CTA-pair kernel.  Returns SYRK_ERR_PLAN when the problem has
// fewer blocks than the GPU has pairs.  `launch` false: only create what the call would allocate.
int run_pair_square(DeviceState* ds, int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc,
                    double alpha, double beta, int dtype, cudaStream_t stream, bool launch = true) {
    const int tile = bf16_tile();
    const int64_t n_tiles = (N + tile - 1) / tile, n_super = (n_tiles + 1) / 2;
    const int64_t bk = 128 / int64_t(a_elem(dtype));
    int64_t n_blk = 0;
    int split = 1;
    if (!pair_square_shape(N, M, dtype, ds->sm_count, runtime().split_k, &n_blk, &split)) return SYRK_ERR_PLAN;
    void* d_partial = nullptr;
    if (split > 1) {
        const int rc2 = workspace_for_stream(ds, stream, size_t(split) * size_t(n_blk) * 4 * tile * tile * sizeof(float), &d_partial);
        if (rc2 != SYRK_OK) return rc2;
    }
    auto it = ds->pair_plans.find(n_tiles);
    if (it == ds->pair_plans.end()) {
        // heaviest first is moot (all blocks cost the same); the diagonal blocks go last
        std::vector<int4> blocks;
        for (int64_t I = 0; I < n_super; ++I)
            for (int64_t J = 0; J < I; ++J)
                blocks.push_back(make_int4(int(2 * I), int(2 * I + 1), int(2 * J), int(2 * J + 1)));
        for (int64_t I = 0; I < n_super; ++I)
            blocks.push_back(make_int4(int(2 * I), int(2 * I + 1), int(2 * I), int(2 * I + 1)));
        PairPlan pp;
        pp.n_blocks = int32_t(blocks.size());
        bool ok = cudaMalloc(&pp.d_blocks, blocks.size() * sizeof(int4)) == cudaSuccess;
        ok = ok && cudaMemcpy(pp.d_blocks, blocks.data(), blocks.size() * sizeof(int4), cudaMemcpyHostToDevice) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            if (pp.d_blocks) cudaFree(pp.d_blocks);
            return SYRK_ERR_ALLOC;
        }
        it = ds->pair_plans.emplace(n_tiles, pp).first;
    }
    if (!launch) return SYRK_OK;
    const PairPlan& pp = it->second;
    CUtensorMap tm, tmc;
    int rc = encode_tensor_map_2d(&tm, dtype, A, N, M, lda, tile, int(bk));
    if (rc != SYRK_OK) return rc;
    const bool c_tma = (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 3) == 0 &&
                       encode_tensor_map_c_f32(&tmc, C, N, ldc, bf16_store_box()) == SYRK_OK;
    cudaError_t e = launch_syrk_pair_square(tm, c_tma ? &tmc : nullptr, pp.d_blocks, pp.n_blocks, N, M, static_cast<float*>(C),
                                            ldc, float(alpha), float(beta), dtype - SYRK_DTYPE_BF16_F32,
                                            status_for_stream(ds, stream), ds->sm_count, stream, split,
                                            static_cast<float*>(d_partial));
    return e == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}
}  // namespace

int tbsyrk::syrk_run_device(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc, double alpha,
                            double beta, int dtype, cudaStream_t stream, int f64_launch, int a_is_m_by_n, int upper,
                            bool prepare_only) {
    DeviceState* ds = nullptr;
    int rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    if (alpha == 0.0 || M == 0) {
        if (beta == 1.0 || prepare_only) return SYRK_OK;
        return launch_scale_lower(dtype, N, C, ldc, beta, stream, upper) == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
    }
    if (!prepare_only && !tma_ok(A, lda, dtype))
        return launch_syrk_plain(dtype, N, M, A, lda, C, ldc, alpha, beta, a_is_m_by_n, stream, upper) == cudaSuccess
                   ? SYRK_OK : SYRK_ERR_CUDA;
    const bool pair_form = is_tcgen05_dtype(dtype) && !a_is_m_by_n && !upper;    // what the CTA-pair kernel covers
    if (runtime().pair_square && pair_form) {
        rc = run_pair_square(ds, N, M, A, lda, C, ldc, alpha, beta, dtype, stream, !prepare_only);
        if (rc != SYRK_ERR_PLAN) return rc;          // SYRK_ERR_PLAN: too few blocks for the pairs - the square list below
    }
    DevicePlan* dp = nullptr;
    rc = get_device_plan(ds, N, dtype, &dp, upper);
    if (rc != SYRK_OK) return rc;
    // SYRK_SCHEDULE_AUTO (the default): a triangle-block list shorter than a few rounds of SMs fills the GPU
    // unevenly or only through a K-split of many short units; square blocks on CTA pairs (their own
    // K-split, equal units) are the faster form there (measured 1.0-1.5x from 1024 to 7168 rows, never slower).
    if (runtime().auto_pair && pair_form && int64_t(dp->plan.items.size()) < 4 * int64_t(ds->sm_count)) {
        rc = run_pair_square(ds, N, M, A, lda, C, ldc, alpha, beta, dtype, stream, !prepare_only);
        if (rc != SYRK_ERR_PLAN) return rc;
    }
    const KernelShape ks = kernel_shape(dtype);
    int split = 1, tail_slices = 1;
    int64_t tail_first = 0;
    void* d_partial = nullptr;
    if (is_tcgen05_dtype(dtype)) {
        split = pick_split_k(ds, dp, M, ks.bk);
        if (split > 1) {
            const size_t want = size_t(split) * size_t(dp->total_tiles) * ks.tile * ks.tile * sizeof(float);
            if ((rc = workspace_for_stream(ds, stream, want, &d_partial)) != SYRK_OK) return rc;
        }
    } else {
        // FP64 K-split for lists shorter than the SM count (every stream has its own workspace, so the
        // Cholesky driver's two streams may both use it)
        split = auto_split_k_f64(int64_t(dp->plan.items.size()), N, M, ks.bk, ds->sm_count, runtime().split_k);
        if (split > 1 &&
            (rc = workspace_for_stream(ds, stream, size_t(split) * size_t(N) * size_t(N) * sizeof(double), &d_partial)) != SYRK_OK)
            return rc;
        // Otherwise: the last round's items in slices (tail K-split), in either launch form.
        const int64_t n_items = int64_t(dp->plan.items.size());
        if (split == 1 && !upper && runtime().f64_tail_slices != 1) {
            TailSplit ts{n_items, 1};
            const int64_t ksteps = (M + ks.bk - 1) / ks.bk;
            if (runtime().f64_tail_slices >= 2) {                    // forced (tests, measurements)
                const int64_t tail = std::min<int64_t>(n_items, std::max<int64_t>(1, runtime().f64_tail_items));
                if (runtime().f64_tail_slices <= ksteps) ts = TailSplit{n_items - tail, runtime().f64_tail_slices};
            } else {
                auto it = dp->tail_split.find(ksteps);
                if (it == dp->tail_split.end()) {
                    const TailSplit t = plan_tail_split_f64(dp->plan.items, ksteps, ds->sm_count);
                    it = dp->tail_split.emplace(ksteps, std::make_pair(t.first, t.slices)).first;
                }
                ts = TailSplit{it->second.first, it->second.second};
            }
            if (ts.slices > 1) {
                const size_t want = size_t(f64_tail_partial_elems(n_items - ts.first, ts.slices)) * sizeof(double);
                if ((rc = workspace_for_stream(ds, stream, want, &d_partial)) != SYRK_OK) return rc;
                tail_first = ts.first; tail_slices = ts.slices;
            }
        }
    }
    if (prepare_only) return SYRK_OK;
    CUtensorMap tm;
    // A stored M x N: boxes of one stage's k-rows x 128 bytes of columns (16 doubles, 64 bf16)
    if (a_is_m_by_n) rc = encode_tensor_map_2d(&tm, dtype, A, M, N, lda, ks.bk, 128 / int(a_elem(dtype)),
                                               dtype == SYRK_DTYPE_TF32_F32);
    else rc = encode_tensor_map_2d(&tm, dtype, A, N, M, lda, ks.tile, ks.bk);
    if (rc != SYRK_OK) return rc;
    return launch_items(ds, dtype, tm, dp->d_items, int64_t(dp->plan.items.size()), N, M, C, ldc, alpha, beta, split,
                        dp->d_tile_base, dp->total_tiles, dp->d_cta_begin, dp->n_ctas, f64_launch, a_is_m_by_n, stream, upper,
                        d_partial, tail_first, tail_slices);
}

namespace {

// Rows [row0, row1) of the lower triangles of the diagonal blocks of side band_h of C (row pitch
// ldc), packed: block b
// starts at element b * band_h (band_h + 1) / 2 and its local row l has l + 1 entries starting at
// l (l + 1) / 2.
template <typename T>
__global__ void pack_diag_blocks_kernel(int64_t row0, int64_t row1, int64_t band_h, const T* __restrict__ C,
                                        int64_t ldc, T* __restrict__ packed) {
    const int64_t full = band_h * (band_h + 1) / 2;
    for (int64_t i = row0 + blockIdx.y; i < row1; i += gridDim.y) {
        const int64_t b = i / band_h, l = i - b * band_h;
        const T* src = C + i * ldc + b * band_h;
        T* dst = packed + b * full + l * (l + 1) / 2;
        for (int64_t j = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; j <= l; j += int64_t(gridDim.x) * blockDim.x)
            dst[j] = src[j];
    }
}

// Entries [first, first + count) of the packed lower triangle (row i starts at i (i + 1) / 2):
// C[i][j] <- packed[idx - first] + beta * C[i][j]  (C not read when beta == 0).
template <typename T>
__global__ void unpack_lower_axpby_kernel(int64_t first, int64_t count, const T* __restrict__ packed, double beta,
                                          T* __restrict__ C, int64_t ldc) {
    for (int64_t e = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; e < count; e += int64_t(gridDim.x) * blockDim.x) {
        const int64_t idx = first + e;
        int64_t i = int64_t((sqrt(8.0 * double(idx) + 1.0) - 1.0) * 0.5);
        while (i * (i + 1) / 2 > idx) --i;                 // the square root may be off by one either way
        while ((i + 1) * (i + 2) / 2 <= idx) ++i;
        const int64_t j = idx - i * (i + 1) / 2;
        T* c = C + i * ldc + j;
        *c = (beta == 0.0) ? packed[e] : T(double(packed[e]) + beta * double(*c));
    }
}

// The launch form of the rank-2k and Hermitian updates: as set by syrk_set_f64_launch, the automatic rule being
// that of the rank-k update.
bool two_warp_form_is_persistent(int64_t n_items, double beta, int sm_count) {
    const int mode = runtime().f64_launch;
    return mode == SYRK_F64_LAUNCH_PERSISTENT ||
           (mode == SYRK_F64_LAUNCH_AUTO && f64_persistent_pays(n_items, beta, sm_count));
}

// Work list of Algorithm 4 for the kernels' forms in which two warps share a tile (rank-2k and Hermitian
// updates): triangle blocks with k = 4 (6 tiles; for the rank-2k update a stage holds the four segments of A
// and the same rows of B), 2 x 2 rectangles, diagonal blocks of two rows.  Cached per device.
int get_two_warp_plan(DeviceState* ds, int64_t N, DevicePlan** out) {
    const int64_t n_tiles = (N + f64_tile() - 1) / f64_tile();
    const auto key = std::make_tuple(n_tiles, 64, runtime().schedule);       // 64: this list
    auto it = ds->plans.find(key);
    if (it == ds->plans.end()) {
        DevicePlan dp;
        PlanParams p;
        p.n_tiles = n_tiles; p.k = 4; p.rect_rows = 2; p.rect_cols = 2; p.diag_side = 2; p.schedule = runtime().schedule;
        if (!build_plan(p, &dp.plan)) return SYRK_ERR_PLAN;
        std::stable_sort(dp.plan.items.begin(), dp.plan.items.end(),
                         [](const WorkItem& a, const WorkItem& b) { return a.n_tile > b.n_tile; });
        const size_t n = dp.plan.items.size();
        if (n > 0) {
            if (cudaMalloc(&dp.d_items, n * sizeof(WorkItem)) != cudaSuccess) { cudaGetLastError(); return SYRK_ERR_ALLOC; }
            if (cudaMemcpy(dp.d_items, dp.plan.items.data(), n * sizeof(WorkItem), cudaMemcpyHostToDevice) != cudaSuccess) {
                cudaGetLastError(); cudaFree(dp.d_items); return SYRK_ERR_CUDA;
            }
        }
        it = ds->plans.emplace(key, std::move(dp)).first;
    }
    *out = &it->second;
    return SYRK_OK;
}

}  // namespace

extern "C" {

int syrk_pack_lower(int64_t N, const void* C, int64_t ldc, int dtype, void* packed, void* stream) {
    if (!known_dtype(dtype)) return SYRK_ERR_DTYPE;
    if (N < 0) return SYRK_ERR_SIZE;
    if (N == 0) return SYRK_OK;
    if (ldc < N) return SYRK_ERR_LD;
    if (!C || !packed) return SYRK_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dim3 grid(unsigned(std::min<int64_t>(64, (N + 255) / 256)), unsigned(std::min<int64_t>(N, 32768)));
    if (dtype == SYRK_DTYPE_F64)
        pack_diag_blocks_kernel<double><<<grid, 256, 0, st>>>(0, N, N, static_cast<const double*>(C), ldc, static_cast<double*>(packed));
    else
        pack_diag_blocks_kernel<float><<<grid, 256, 0, st>>>(0, N, N, static_cast<const float*>(C), ldc, static_cast<float*>(packed));
    return cudaGetLastError() == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}

int syrk_unpack_lower_axpby(int64_t N, int64_t first, int64_t count, const void* packed, double beta, void* C,
                            int64_t ldc, int dtype, void* stream) {
    if (!known_dtype(dtype)) return SYRK_ERR_DTYPE;
    if (N < 0 || first < 0 || count < 0 || first + count > N * (N + 1) / 2) return SYRK_ERR_SIZE;
    if (count == 0) return SYRK_OK;
    if (ldc < N) return SYRK_ERR_LD;
    if (!C || !packed) return SYRK_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned grid = unsigned(std::min<int64_t>((count + 255) / 256, 148 * 16));
    if (dtype == SYRK_DTYPE_F64)
        unpack_lower_axpby_kernel<double><<<grid, 256, 0, st>>>(first, count, static_cast<const double*>(packed), beta,
                                                                static_cast<double*>(C), ldc);
    else
        unpack_lower_axpby_kernel<float><<<grid, 256, 0, st>>>(first, count, static_cast<const float*>(packed), beta,
                                                               static_cast<float*>(C), ldc);
    return cudaGetLastError() == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}

int syrk_lower(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc, double alpha,
               double beta, int dtype, void* stream) {
    int rc = validate(N, M, A, lda, C, ldc, dtype);
    if (rc != SYRK_OK || N == 0) return rc;
    std::lock_guard<std::mutex> lock(runtime().mu);
    return syrk_run_device(N, M, A, lda, C, ldc, alpha, beta, dtype, static_cast<cudaStream_t>(stream));
}

int syrk_lower_tn(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc, double alpha,
                  double beta, int dtype, void* stream) {
    int rc = validate(N, M, A, lda, C, ldc, dtype, true);
    if (rc != SYRK_OK || N == 0) return rc;
    std::lock_guard<std::mutex> lock(runtime().mu);
    return syrk_run_device(N, M, A, lda, C, ldc, alpha, beta, dtype, static_cast<cudaStream_t>(stream), -1, 1);
}

int syrk_ex(int uplo, int trans, int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc,
            double alpha, double beta, int dtype, void* stream) {
    if ((uplo != SYRK_UPLO_LOWER && uplo != SYRK_UPLO_UPPER) || (trans != SYRK_OP_N && trans != SYRK_OP_T))
        return SYRK_ERR_SIZE;
    int rc = validate(N, M, A, lda, C, ldc, dtype, trans == SYRK_OP_T);
    if (rc != SYRK_OK || N == 0) return rc;
    std::lock_guard<std::mutex> lock(runtime().mu);
    return syrk_run_device(N, M, A, lda, C, ldc, alpha, beta, dtype, static_cast<cudaStream_t>(stream), -1,
                           trans == SYRK_OP_T ? 1 : 0, uplo == SYRK_UPLO_UPPER ? 1 : 0);
}

int syr2k_lower(int64_t N, int64_t M, const void* A, int64_t lda, const void* B, int64_t ldb, void* C, int64_t ldc,
                double alpha, double beta, void* stream) {
    int rc = validate(N, M, A, lda, C, ldc, SYRK_DTYPE_F64);
    if (rc != SYRK_OK || N == 0) return rc;
    if (ldb < std::max<int64_t>(1, M)) return SYRK_ERR_LD;
    if (M > 0 && !B) return SYRK_ERR_NULL;
    std::lock_guard<std::mutex> lock(runtime().mu);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceState* ds = nullptr;
    rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    if (alpha == 0.0 || M == 0) {
        if (beta == 1.0) return SYRK_OK;
        return launch_scale_lower(SYRK_DTYPE_F64, N, C, ldc, beta, st) == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
    }
    if (!tma_ok(A, lda, SYRK_DTYPE_F64) || !tma_ok(B, ldb, SYRK_DTYPE_F64))
        return launch_syr2k_plain(N, M, static_cast<const double*>(A), lda, static_cast<const double*>(B), ldb,
                                  static_cast<double*>(C), ldc, alpha, beta, st) == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
    DevicePlan* dp = nullptr;
    if ((rc = get_two_warp_plan(ds, N, &dp)) != SYRK_OK) return rc;
    CUtensorMap ta, tb, tmc;
    if ((rc = encode_tensor_map_2d(&ta, SYRK_DTYPE_F64, A, N, M, lda, f64_tile(), f64_bk())) != SYRK_OK) return rc;
    if ((rc = encode_tensor_map_2d(&tb, SYRK_DTYPE_F64, B, N, M, ldb, f64_tile(), f64_bk())) != SYRK_OK) return rc;
    const bool c_tma = beta != 0.0 && (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 1) == 0 &&
                       encode_tensor_map_c_f64(&tmc, C, N, ldc, f64_tile()) == SYRK_OK;
    const int64_t n_items = int64_t(dp->plan.items.size());
    int* tickets = two_warp_form_is_persistent(n_items, beta, ds->sm_count) ? tickets_for_stream(ds, st) : nullptr;
    return launch_syr2k_f64(ta, tb, c_tma ? &tmc : nullptr, dp->d_items, n_items, N, M, static_cast<double*>(C), ldc, alpha,
                            beta, status_for_stream(ds, st), st, tickets, ds->sm_count) == cudaSuccess
               ? SYRK_OK : SYRK_ERR_CUDA;
}

int herk_lower(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc, double alpha, double beta,
               void* stream) {
    if (N < 0 || M < 0) return SYRK_ERR_SIZE;
    if (lda < std::max<int64_t>(1, M) || ldc < std::max<int64_t>(1, N)) return SYRK_ERR_LD;
    if (N == 0) return SYRK_OK;
    if (!C || (M > 0 && !A)) return SYRK_ERR_NULL;
    std::lock_guard<std::mutex> lock(runtime().mu);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceState* ds = nullptr;
    int rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    if ((alpha == 0.0 || M == 0) && beta == 1.0) return SYRK_OK;
    // Scale-only calls and operands that are not 16-byte aligned take the plain-load kernel.
    if (alpha == 0.0 || M == 0 || (reinterpret_cast<uintptr_t>(A) & 15) != 0 || (reinterpret_cast<uintptr_t>(C) & 15) != 0)
        return launch_herk_plain(N, M, static_cast<const double*>(A), lda, static_cast<double*>(C), ldc, alpha, beta, st) ==
                       cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
    DevicePlan* dp = nullptr;
    if ((rc = get_two_warp_plan(ds, N, &dp)) != SYRK_OK) return rc;
    CUtensorMap ta;          // the real view of A: N rows of 2M values, pitch 2 lda
    if ((rc = encode_tensor_map_2d(&ta, SYRK_DTYPE_F64, A, N, 2 * M, 2 * lda, f64_tile(), f64_bk())) != SYRK_OK) return rc;
    const int64_t n_items = int64_t(dp->plan.items.size());
    int* tickets = two_warp_form_is_persistent(n_items, beta, ds->sm_count) ? tickets_for_stream(ds, st) : nullptr;
    return launch_herk_f64(ta, dp->d_items, n_items, N, M, static_cast<double*>(C), ldc, alpha, beta, status_for_stream(ds, st),
                           st, tickets, ds->sm_count) == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}

int syr2k_lower_ex(int64_t N, int64_t M, const void* A, int64_t lda, const void* B, int64_t ldb, void* C, int64_t ldc,
                   double alpha, double beta, int dtype, void* stream) {
    if (dtype == SYRK_DTYPE_F64) return syr2k_lower(N, M, A, lda, B, ldb, C, ldc, alpha, beta, stream);
    int rc = validate(N, M, A, lda, C, ldc, dtype);
    if (rc != SYRK_OK || N == 0) return rc;
    if (ldb < std::max<int64_t>(1, M)) return SYRK_ERR_LD;
    if (M > 0 && !B) return SYRK_ERR_NULL;
    std::lock_guard<std::mutex> lock(runtime().mu);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DeviceState* ds = nullptr;
    rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    if (alpha == 0.0 || M == 0) {
        if (beta == 1.0) return SYRK_OK;
        return launch_scale_lower(dtype, N, C, ldc, beta, st) == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
    }
    if (!tma_ok(A, lda, dtype) || !tma_ok(B, ldb, dtype))
        return launch_syr2k_plain_f32(dtype, N, M, A, lda, B, ldb, static_cast<float*>(C), ldc, float(alpha), float(beta), st) ==
                       cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
    // The work list of the rank-k update under the current setting (triangle blocks k = 3, or squares): same
    // items, each stage carrying the items' rows of both operands.  The CTA-pair kernel has no rank-2k form.
    DevicePlan* dp = nullptr;
    rc = get_device_plan(ds, N, dtype, &dp);
    if (rc != SYRK_OK) return rc;
    const KernelShape ks = kernel_shape(dtype);
    const int split = pick_split_k(ds, dp, M, ks.bk);
    void* d_partial = nullptr;
    if (split > 1) {
        const size_t want = size_t(split) * size_t(dp->total_tiles) * ks.tile * ks.tile * sizeof(float);
        if ((rc = workspace_for_stream(ds, st, want, &d_partial)) != SYRK_OK) return rc;
    }
    CUtensorMap ta, tb, tmc;
    if ((rc = encode_tensor_map_2d(&ta, dtype, A, N, M, lda, ks.tile, ks.bk)) != SYRK_OK) return rc;
    if ((rc = encode_tensor_map_2d(&tb, dtype, B, N, M, ldb, ks.tile, ks.bk)) != SYRK_OK) return rc;
    const bool c_tma = (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (ldc & 3) == 0 &&
                       encode_tensor_map_c_f32(&tmc, C, N, ldc, bf16_store_box()) == SYRK_OK;
    return launch_syrk_bf16(ta, c_tma ? &tmc : nullptr, dp->d_items, int64_t(dp->plan.items.size()), N, M,
                            static_cast<float*>(C), ldc, float(alpha), float(beta), split, static_cast<float*>(d_partial),
                            dp->d_tile_base, dp->total_tiles, dp->d_cta_begin, dp->n_ctas, 0, dtype - SYRK_DTYPE_BF16_F32,
                            status_for_stream(ds, st), ds->sm_count, st, 0, 0, 0, &tb) == cudaSuccess
               ? SYRK_OK : SYRK_ERR_CUDA;
}

int syrk_lower_batched(int64_t batch, int64_t N, int64_t M, const void* A, int64_t lda, int64_t stride_a,
                       void* C, int64_t ldc, int64_t stride_c, double alpha, double beta, int dtype, void* stream) {
    if (batch < 0 || batch >= (int64_t(1) << 31)) return SYRK_ERR_SIZE;
    int rc = validate(N, M, A, lda, C, ldc, dtype);
    if (rc != SYRK_OK || N == 0 || batch == 0) return rc;
    if (batch > 1 && ((M > 0 && stride_a < (N - 1) * lda + M) || stride_c < (N - 1) * ldc + N)) return SYRK_ERR_LD;
    std::lock_guard<std::mutex> lock(runtime().mu);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t ea = a_elem(dtype), ec = c_elem(dtype);
    // One launch over all matrices needs 3-D tensor maps: base and both pitches of A multiples of 16
    // bytes.  Otherwise (and for the quick returns) the matrices are enqueued one by one.
    const bool one_launch = alpha != 0.0 && M > 0 && batch > 1 && tma_ok(A, lda, dtype) && (size_t(stride_a) * ea) % 16 == 0;
    if (!one_launch) {
        for (int64_t b = 0; b < batch; ++b) {
            rc = syrk_run_device(N, M, static_cast<const char*>(A) + size_t(b) * size_t(stride_a) * ea, lda,
                                 static_cast<char*>(C) + size_t(b) * size_t(stride_c) * ec, ldc, alpha, beta, dtype, st);
            if (rc != SYRK_OK) return rc;
        }
        return SYRK_OK;
    }
    DeviceState* ds = nullptr;
    rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    DevicePlan* dp = nullptr;
    rc = get_device_plan(ds, N, dtype, &dp);
    if (rc != SYRK_OK) return rc;
    const KernelShape ks = kernel_shape(dtype);
    const int64_t n_items = int64_t(dp->plan.items.size());
    if (n_items * batch >= (int64_t(1) << 31)) return SYRK_ERR_SIZE;
    CUtensorMap tm, tmc;
    rc = encode_tensor_map_batched(&tm, dtype, A, N, M, lda, stride_a, batch, ks.tile, ks.bk);
    if (rc != SYRK_OK) return rc;
    const bool c_aligned = (reinterpret_cast<uintptr_t>(C) & 15) == 0 && (size_t(ldc) * ec) % 16 == 0 &&
                           (size_t(stride_c) * ec) % 16 == 0;
    cudaError_t e;
    if (dtype == SYRK_DTYPE_F64) {
        const bool c_tma = beta != 0.0 && c_aligned &&
                           encode_tensor_map_c_batched(&tmc, 1, C, N, ldc, stride_c, batch, f64_tile()) == SYRK_OK;
        // persistent blocks over the (matrix, item) pairs when the launch-form rule says so for that many units
        const int mode = runtime().f64_launch;
        const bool persistent = mode == SYRK_F64_LAUNCH_PERSISTENT ||
                                (mode == SYRK_F64_LAUNCH_AUTO && f64_persistent_pays(n_items * batch, beta, ds->sm_count));
        int* tickets = persistent ? tickets_for_stream(ds, st) : nullptr;
        e = launch_syrk_f64(tm, c_tma ? &tmc : nullptr, dp->d_items, n_items, N, M, static_cast<double*>(C), ldc, alpha,
                            beta, 0, tickets, ds->sm_count, status_for_stream(ds, st), st, batch, stride_c);
    } else {
        const bool c_tma = c_aligned &&
                           encode_tensor_map_c_batched(&tmc, 0, C, N, ldc, stride_c, batch, bf16_store_box()) == SYRK_OK;
        e = launch_syrk_bf16(tm, c_tma ? &tmc : nullptr, dp->d_items, n_items, N, M, static_cast<float*>(C), ldc,
                             float(alpha), float(beta), 1, nullptr, dp->d_tile_base, dp->total_tiles, nullptr, 0, 0,
                             dtype - SYRK_DTYPE_BF16_F32, status_for_stream(ds, st), ds->sm_count, st, batch, stride_c);
    }
    return e == cudaSuccess ? SYRK_OK : SYRK_ERR_CUDA;
}

int syrk_lower_host(int64_t N, int64_t M, const void* A, int64_t lda, void* C, int64_t ldc, double alpha,
                    double beta, int dtype) {
    int rc = validate(N, M, A, lda, C, ldc, dtype);
    if (rc != SYRK_OK || N == 0) return rc;
    std::lock_guard<std::mutex> lock(runtime().mu);
    DeviceState* ds = nullptr;
    rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    constexpr int kMaxChunks = 8, kBands = 16;
    if (!ds->host_stream) {
        bool ok = cudaStreamCreateWithFlags(&ds->host_stream, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&ds->copy_stream, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&ds->down_stream, cudaStreamNonBlocking) == cudaSuccess;
        for (cudaStream_t& bs : ds->band_streams) ok = ok && cudaStreamCreateWithFlags(&bs, cudaStreamNonBlocking) == cudaSuccess;
        for (cudaEvent_t& ev : ds->host_events) ok = ok && cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) { cudaGetLastError(); return SYRK_ERR_CUDA; }
    }
    cudaStream_t st = ds->host_stream, cp = ds->copy_stream;
    const size_t ea = a_elem(dtype), ec = c_elem(dtype);
    // device pitch of A rounded up so that the TMA path applies to any M
    const int64_t dlda = (std::max<int64_t>(M, 1) * int64_t(ea) + 15) / 16 * 16 / int64_t(ea);
    const int64_t dldc = (N + 1) / 2 * 2;
    // packed lower triangles of the diagonal blocks of the download bands (see below)
    cudaPointerAttributes c_attr{};
    const bool c_pinned = cudaPointerGetAttributes(&c_attr, C) == cudaSuccess && c_attr.type == cudaMemoryTypeHost;
    cudaGetLastError();
    // Large problems with a page-locked C are produced band by band (see below); the bands are then
    // those of the row-ordered work list.
    BandedPlan* bp = nullptr;
    const bool banded = c_pinned && M > 0 && alpha != 0.0 && N >= 4096 && runtime().host_pipeline != SYRK_HOST_COLUMN_BLOCKS &&
                        get_banded_plan(ds, N, dtype, kBands, &bp) == SYRK_OK && bp->item_end.size() > 1;
    const int64_t pk_h = banded ? bp->band_rows
                                : (c_pinned ? (N + std::max<int64_t>(1, std::min<int64_t>(kBands, N / 256)) - 1) /
                                                  std::max<int64_t>(1, std::min<int64_t>(kBands, N / 256))
                                            : N);
    const int64_t pk_bands = (N + pk_h - 1) / pk_h;
    const size_t packed_bytes = size_t(pk_bands) * size_t(pk_h) * size_t(pk_h + 1) / 2 * ec;
    if ((rc = ensure_device_bytes(&ds->d_a, &ds->d_a_bytes, size_t(N) * dlda * ea)) != SYRK_OK) return rc;
    if ((rc = ensure_device_bytes(&ds->d_c, &ds->d_c_bytes, size_t(N) * dldc * ec)) != SYRK_OK) return rc;
    if ((rc = ensure_device_bytes(&ds->d_packed, &ds->d_packed_bytes, packed_bytes)) != SYRK_OK) return rc;
    if ((rc = ensure_pinned_bytes(&ds->h_packed, &ds->h_packed_bytes, packed_bytes)) != SYRK_OK) return rc;
    auto chk = [](cudaError_t e) { if (e != cudaSuccess) { cudaGetLastError(); return false; } return true; };

    if (banded) {
        // Row-band pipeline.  Rows [r0, r1) of C need rows [0, r1) of A only, and in the row-ordered
        // square-block list the items of band j write rows of band j only.  So A goes up band by band
        // (copy stream), band j's items run as soon as its rows have landed (four compute streams in
        // turn, so that short lists of long items overlap), and band j of C goes down (download
        // stream) while later bands are still being uploaded and computed: the rectangle left of the
        // diagonal block straight into C, the diagonal block packed.
        const int64_t band_h = bp->band_rows, n_bands = int64_t(bp->item_end.size());
        cudaStream_t dl = ds->down_stream;
        const KernelShape ks = kernel_shape(dtype);
        CUtensorMap tm;
        if ((rc = encode_tensor_map_2d(&tm, dtype, ds->d_a, N, M, dlda, ks.tile, ks.bk)) != SYRK_OK) return rc;
        cudaEvent_t* ev_up = ds->host_events;
        cudaEvent_t* ev_done = ds->host_events + kBands;
        cudaEvent_t* ev_packed = ds->host_events + 2 * kBands;
        const size_t full = size_t(band_h) * size_t(band_h + 1) / 2;
        for (int64_t j = 0; j < n_bands; ++j) {
            const int64_t r0 = j * band_h, r1 = std::min(N, r0 + band_h);
            cudaStream_t cs = ds->band_streams[j % 4];
            bool ok = chk(cudaMemcpy2DAsync(static_cast<char*>(ds->d_a) + size_t(r0) * dlda * ea, dlda * ea,
                                            static_cast<const char*>(A) + size_t(r0) * lda * ea, lda * ea, M * ea, r1 - r0,
                                            cudaMemcpyHostToDevice, cp));
            if (beta != 0.0)
                ok = ok && chk(cudaMemcpy2DAsync(static_cast<char*>(ds->d_c) + size_t(r0) * dldc * ec, dldc * ec,
                                                 static_cast<const char*>(C) + size_t(r0) * ldc * ec, ldc * ec, r1 * ec, r1 - r0,
                                                 cudaMemcpyHostToDevice, cp));
            ok = ok && chk(cudaEventRecord(ev_up[j], cp)) && chk(cudaStreamWaitEvent(cs, ev_up[j], 0));
            if (!ok) return SYRK_ERR_CUDA;
            const int64_t i0 = j == 0 ? 0 : bp->item_end[size_t(j - 1)], i1 = bp->item_end[size_t(j)];
            if (i1 > i0) {
                rc = launch_items(ds, dtype, tm, bp->d_items + i0, i1 - i0, N, M, ds->d_c, dldc, alpha, beta, 1, nullptr, 0,
                                  nullptr, 0, -1, 0, cs);
                if (rc != SYRK_OK) return rc;
            }
            ok = chk(cudaEventRecord(ev_done[j], cs)) && chk(cudaStreamWaitEvent(dl, ev_done[j], 0));
            if (ok && r0 > 0)
                ok = chk(cudaMemcpy2DAsync(static_cast<char*>(C) + size_t(r0) * ldc * ec, size_t(ldc) * ec,
                                           static_cast<const char*>(ds->d_c) + size_t(r0) * dldc * ec, size_t(dldc) * ec,
                                           size_t(r0) * ec, size_t(r1 - r0), cudaMemcpyDeviceToHost, dl));
            if (!ok) return SYRK_ERR_CUDA;
            const dim3 grid(unsigned(std::min<int64_t>(64, (band_h + 255) / 256)), unsigned(std::min<int64_t>(r1 - r0, 32768)));
            if (dtype == SYRK_DTYPE_F64)
                pack_diag_blocks_kernel<double><<<grid, 256, 0, dl>>>(r0, r1, band_h, static_cast<const double*>(ds->d_c), dldc,
                                                                      static_cast<double*>(ds->d_packed));
            else
                pack_diag_blocks_kernel<float><<<grid, 256, 0, dl>>>(r0, r1, band_h, static_cast<const float*>(ds->d_c), dldc,
                                                                     static_cast<float*>(ds->d_packed));
            const size_t h = size_t(r1 - r0);
            if (!chk(cudaGetLastError()) ||
                !chk(cudaMemcpyAsync(static_cast<char*>(ds->h_packed) + size_t(j) * full * ec,
                                     static_cast<const char*>(ds->d_packed) + size_t(j) * full * ec, h * (h + 1) / 2 * ec,
                                     cudaMemcpyDeviceToHost, dl)) ||
                !chk(cudaEventRecord(ev_packed[j], dl)))
                return SYRK_ERR_CUDA;
        }
        const char* psrc = static_cast<const char*>(ds->h_packed);
        char* pdst = static_cast<char*>(C);
        for (int64_t j = 0; j < n_bands; ++j) {
            if (!chk(cudaEventSynchronize(ev_packed[j]))) return SYRK_ERR_CUDA;
            const int64_t r0 = j * band_h, r1 = std::min(N, r0 + band_h);
            for (int64_t i = r0; i < r1; ++i) {
                const int64_t l = i - r0;
                std::memcpy(pdst + (size_t(i) * ldc + size_t(r0)) * ec,
                            psrc + (size_t(j) * full + size_t(l) * size_t(l + 1) / 2) * ec, size_t(l + 1) * ec);
            }
        }
        if (!chk(cudaStreamSynchronize(dl))) return SYRK_ERR_CUDA;
        int worst = SYRK_OK;                               // the band streams ran the kernels
        for (cudaStream_t bs : ds->band_streams) {
            const int r = read_and_clear_status(ds, bs, false);
            if (r != SYRK_OK) worst = r;
        }
        return worst;
    }

    // Upload and compute overlap: A goes up in column blocks on the copy stream and each block's
    // rank-update C <- alpha A_c A_c^T + (beta or 1) C runs on the compute stream as soon as its
    // block has landed.  Blocks are multiples of 256 columns (16-byte aligned for every dtype, whole
    // pipeline stages) and at least 32 MB of A each, so short inputs stay one call.
    int64_t n_chunks = 1;
    if (M > 0) {
        const size_t a_bytes = size_t(N) * size_t(M) * ea;
        n_chunks = std::max<int64_t>(1, std::min<int64_t>({int64_t(kMaxChunks), int64_t(a_bytes >> 25), M / 256}));
    }
    const int64_t chunk_cols = M > 0 ? ((M + n_chunks - 1) / n_chunks + 255) / 256 * 256 : 0;
    if (beta != 0.0 && !chk(cudaMemcpy2DAsync(ds->d_c, dldc * ec, C, ldc * ec, N * ec, N, cudaMemcpyHostToDevice, cp)))
        return SYRK_ERR_CUDA;
    if (M == 0) {
        if (!chk(cudaEventRecord(ds->host_events[0], cp)) || !chk(cudaStreamWaitEvent(st, ds->host_events[0], 0)))
            return SYRK_ERR_CUDA;
        rc = syrk_run_device(N, 0, ds->d_a, dlda, ds->d_c, dldc, alpha, beta, dtype, st);
        if (rc != SYRK_OK) return rc;
    }
    for (int64_t c = 0, col0 = 0; col0 < M; ++c, col0 += chunk_cols) {
        const int64_t cols = std::min<int64_t>(chunk_cols, M - col0);
        const char* src = static_cast<const char*>(A) + size_t(col0) * ea;
        char* dst = static_cast<char*>(ds->d_a) + size_t(col0) * ea;
        if (!chk(cudaMemcpy2DAsync(dst, dlda * ea, src, lda * ea, cols * ea, N, cudaMemcpyHostToDevice, cp)) ||
            !chk(cudaEventRecord(ds->host_events[c], cp)) || !chk(cudaStreamWaitEvent(st, ds->host_events[c], 0)))
            return SYRK_ERR_CUDA;
        rc = syrk_run_device(N, cols, dst, dlda, ds->d_c, dldc, alpha, c == 0 ? beta : 1.0, dtype, st);
        if (rc != SYRK_OK) return rc;
    }

    // Download: C is cut into bands of `band_h` rows.  The part of a band left of its diagonal block
    // (rows [r0, r1) x columns [0, r0)) is a rectangle below the diagonal and is copied straight into
    // the caller's C; the diagonal blocks' lower triangles (a few percent of the entries) come back
    // packed and are put in place by the host while the rectangles are still being copied.
    // (Copying straight into C pays only when C is page-locked; otherwise there is one band, i.e.
    // the whole triangle comes back packed as one block.)
    const int64_t n_bands = pk_bands;
    const int64_t band_h = pk_h;
    auto pack_rows = [&](int64_t r0, int64_t r1) {
        const dim3 grid(unsigned(std::min<int64_t>(64, (band_h + 255) / 256)), unsigned(std::min<int64_t>(r1 - r0, 32768)));
        if (dtype == SYRK_DTYPE_F64)
            pack_diag_blocks_kernel<double><<<grid, 256, 0, st>>>(r0, r1, band_h, static_cast<const double*>(ds->d_c), dldc,
                                                                  static_cast<double*>(ds->d_packed));
        else
            pack_diag_blocks_kernel<float><<<grid, 256, 0, st>>>(r0, r1, band_h, static_cast<const float*>(ds->d_c), dldc,
                                                                 static_cast<float*>(ds->d_packed));
        return cudaGetLastError() == cudaSuccess;
    };
    const char* psrc = static_cast<const char*>(ds->h_packed);
    char* pdst = static_cast<char*>(C);
    const size_t full = size_t(band_h) * size_t(band_h + 1) / 2;              // entries of a full diagonal block
    auto unpack_rows = [=](int64_t i0, int64_t i1) {
        for (int64_t i = i0; i < i1; ++i) {
            const int64_t bnd = i / band_h, l = i - bnd * band_h;
            std::memcpy(pdst + (size_t(i) * ldc + size_t(bnd) * band_h) * ec,
                        psrc + (size_t(bnd) * full + size_t(l) * size_t(l + 1) / 2) * ec, size_t(l + 1) * ec);
        }
    };
    const unsigned hw = std::thread::hardware_concurrency();
    auto unpack_parallel = [&](int64_t i0, int64_t i1, size_t bytes, bool by_bytes) {
        // a few host threads, about 4 MB each; `by_bytes`: shares of equal bytes of a triangle's rows
        const int T = int(std::max<int64_t>(1, std::min<int64_t>({int64_t(hw ? hw : 1), int64_t(8), int64_t(bytes >> 22)})));
        std::vector<std::thread> pool;
        int64_t lo = i0;
        for (int t = 0; t < T; ++t) {
            int64_t hi = i0 + (i1 - i0) * (t + 1) / T;
            if (by_bytes) hi = int64_t(std::sqrt(double(i0) * i0 + (double(i1) * i1 - double(i0) * i0) * (t + 1) / T));
            if (t == T - 1) hi = i1;
            hi = std::min(std::max(hi, lo), i1);
            if (t == T - 1) unpack_rows(lo, hi);
            else pool.emplace_back(unpack_rows, lo, hi);
            lo = hi;
        }
        for (std::thread& th : pool) th.join();
    };
    if (n_bands > 1) {
        // page-locked C: diagonal blocks packed (one copy), rectangles copied in place
        if (!pack_rows(0, N) ||
            !chk(cudaMemcpyAsync(ds->h_packed, ds->d_packed, packed_bytes, cudaMemcpyDeviceToHost, st)) ||
            !chk(cudaEventRecord(ds->host_events[0], st)))
            return SYRK_ERR_CUDA;
        for (int64_t r0 = band_h; r0 < N; r0 += band_h) {
            const int64_t r1 = std::min(N, r0 + band_h);
            if (!chk(cudaMemcpy2DAsync(static_cast<char*>(C) + size_t(r0) * ldc * ec, size_t(ldc) * ec,
                                       static_cast<const char*>(ds->d_c) + size_t(r0) * dldc * ec, size_t(dldc) * ec,
                                       size_t(r0) * ec, size_t(r1 - r0), cudaMemcpyDeviceToHost, st)))
                return SYRK_ERR_CUDA;
        }
        if (!chk(cudaEventSynchronize(ds->host_events[0]))) return SYRK_ERR_CUDA;
        unpack_parallel(0, N, packed_bytes, false);
    } else {
        // one block = the whole triangle, packed; it comes back in four groups of rows of about equal
        // bytes, and host threads move group q into C while group q + 1 is copied
        constexpr int kGroups = 4;
        int64_t grp[kGroups + 1];
        for (int q = 0; q <= kGroups; ++q) grp[q] = (q == kGroups) ? N : int64_t(double(N) * std::sqrt(double(q) / kGroups));
        for (int q = 0; q < kGroups; ++q) {
            grp[q + 1] = std::max(grp[q + 1], grp[q]);
            const int64_t r0 = grp[q], r1 = grp[q + 1];
            if (r1 > r0) {
                const size_t off = size_t(r0) * size_t(r0 + 1) / 2 * ec, end = size_t(r1) * size_t(r1 + 1) / 2 * ec;
                if (!pack_rows(r0, r1) ||
                    !chk(cudaMemcpyAsync(static_cast<char*>(ds->h_packed) + off, static_cast<char*>(ds->d_packed) + off,
                                         end - off, cudaMemcpyDeviceToHost, st)))
                    return SYRK_ERR_CUDA;
            }
            if (!chk(cudaEventRecord(ds->host_events[q], st))) return SYRK_ERR_CUDA;
        }
        for (int q = 0; q < kGroups; ++q) {
            if (!chk(cudaEventSynchronize(ds->host_events[q]))) return SYRK_ERR_CUDA;
            if (grp[q + 1] > grp[q])
                unpack_parallel(grp[q], grp[q + 1], size_t(grp[q + 1] - grp[q]) * size_t(grp[q + 1] + grp[q]) / 2 * ec, true);
        }
    }
    if (!chk(cudaStreamSynchronize(st))) return SYRK_ERR_CUDA;
    return read_and_clear_status(ds, st, false);
}

int syrk_plan_prepare_stream(int64_t N, int64_t M, int dtype, void* stream) {
    if (!known_dtype(dtype)) return SYRK_ERR_DTYPE;
    if (N < 0 || M < 0) return SYRK_ERR_SIZE;
    if (N == 0) return SYRK_OK;
    std::lock_guard<std::mutex> lock(runtime().mu);
    // The decisions of a syrk_lower call (schedule, K-split) with everything they allocate, nothing launched.
    return syrk_run_device(N, M, nullptr, M, nullptr, N, 1.0, 0.0, dtype, static_cast<cudaStream_t>(stream), -1, 0, 0, true);
}

int syrk_plan_prepare(int64_t N, int64_t M, int dtype) { return syrk_plan_prepare_stream(N, M, dtype, nullptr); }

void syrk_shutdown(void) {
    std::lock_guard<std::mutex> lock(runtime().mu);
    release_all();
}

int syrk_last_status(void* stream) {
    std::lock_guard<std::mutex> lock(runtime().mu);
    DeviceState* ds = nullptr;
    int rc = get_device_state(&ds);
    if (rc != SYRK_OK) return rc;
    return read_and_clear_status(ds, static_cast<cudaStream_t>(stream), stream == nullptr);
}

const char* syrk_strerror(int code) {
    switch (code) {
        case SYRK_OK: return "success";
        case SYRK_ERR_NULL: return "a required pointer is null";
        case SYRK_ERR_SIZE: return "negative or too large size";
        case SYRK_ERR_LD: return "leading dimension smaller than the row length";
        case SYRK_ERR_DTYPE: return "unknown dtype";
        case SYRK_ERR_ALLOC: return "allocation failed";
        case SYRK_ERR_CUDA: return "a CUDA call failed";
        case SYRK_ERR_PLAN: return "invalid schedule parameters";
        case SYRK_ERR_DEVICE_WAIT: return "a bounded wait inside a kernel ran out";
        case SYRK_ERR_NO_DEVICE: return "no usable sm_100 CUDA device";
        case SYRK_ERR_NOT_SPD: return "matrix is not positive definite";
        case SYRK_ERR_STATIC_LIMIT: return "problem too large for the fixed arrays of syrk_lower_bf16_static (work items or slices x tiles)";
        default: return "unknown error code";
    }
}

int syrk_set_schedule(int schedule) {
    if (schedule != SYRK_SCHEDULE_TBS && schedule != SYRK_SCHEDULE_SQUARE && schedule != SYRK_SCHEDULE_PAIR_SQUARE &&
        schedule != SYRK_SCHEDULE_AUTO)
        return SYRK_ERR_PLAN;
    std::lock_guard<std::mutex> lock(runtime().mu);
    runtime().pair_square = schedule == SYRK_SCHEDULE_PAIR_SQUARE;
    runtime().auto_pair = schedule == SYRK_SCHEDULE_AUTO;
    runtime().schedule = runtime().pair_square ? SYRK_SCHEDULE_SQUARE : (runtime().auto_pair ? SYRK_SCHEDULE_TBS : schedule);
    return SYRK_OK;
}

namespace {
// What syrk_lower(N, M, ..., dtype) runs on a device with `sm_count` SMs under the current settings, for an
// aligned N x M operand and the lower triangle: the schedule and its number of K-slices.
int effective_schedule_of(int64_t N, int64_t M, int dtype, int sm_count, int* split_out) {
    int schedule, forced_split;
    bool pair_square, auto_pair;
    {
        std::lock_guard<std::mutex> lock(runtime().mu);
        schedule = runtime().schedule; forced_split = runtime().split_k;
        pair_square = runtime().pair_square; auto_pair = runtime().auto_pair;
    }
    *split_out = 1;
    if (N == 0 || M == 0) return schedule;
    const KernelShape ks = kernel_shape(dtype);
    Plan plan;
    if (!build_host_plan(N, dtype, schedule, &plan)) return SYRK_ERR_PLAN;
    if (is_tcgen05_dtype(dtype)) {
        int64_t n_blk = 0;
        int split = 1;
        const bool pairs_fit = pair_square_shape(N, M, dtype, sm_count, forced_split, &n_blk, &split);
        if (pairs_fit && (pair_square || (auto_pair && int64_t(plan.items.size()) < 4 * int64_t(sm_count)))) {
            *split_out = split;
            return SYRK_SCHEDULE_PAIR_SQUARE;
        }
        *split_out = auto_split_k(plan.items, M, ks.bk, sm_count, forced_split);
    } else {
        *split_out = auto_split_k_f64(int64_t(plan.items.size()), N, M, ks.bk, sm_count, forced_split);
    }
    return schedule;
}
}  // namespace

int syrk_effective_schedule(int64_t N, int64_t M, int dtype) {
    if (!known_dtype(dtype)) return SYRK_ERR_DTYPE;
    if (N < 0 || M < 0) return SYRK_ERR_SIZE;
    int split = 1;
    return effective_schedule_of(N, M, dtype, 148, &split);
}

int syrk_set_host_pipeline(int mode) {
    if (mode != SYRK_HOST_AUTO && mode != SYRK_HOST_COLUMN_BLOCKS) return SYRK_ERR_PLAN;
    std::lock_guard<std::mutex> lock(runtime().mu);
    runtime().host_pipeline = mode;
    return SYRK_OK;
}

int syrk_host_pipeline_for(int64_t N, int64_t M, int c_is_page_locked) {
    if (N < 0 || M < 0) return SYRK_ERR_SIZE;
    std::lock_guard<std::mutex> lock(runtime().mu);
    return (c_is_page_locked && M > 0 && N >= 4096 && runtime().host_pipeline != SYRK_HOST_COLUMN_BLOCKS)
               ? SYRK_HOST_ROW_BANDS : SYRK_HOST_COLUMN_BLOCKS;
}

int syrk_set_f64_launch(int mode) {
    if (mode != SYRK_F64_LAUNCH_AUTO && mode != SYRK_F64_LAUNCH_PER_ITEM && mode != SYRK_F64_LAUNCH_PERSISTENT)
        return SYRK_ERR_PLAN;
    std::lock_guard<std::mutex> lock(runtime().mu);
    runtime().f64_launch = mode;
    return SYRK_OK;
}

int syrk_set_f64_tail_split(int slices, int64_t tail_items) {
    if (slices < 0 || slices > 64 || tail_items < 0) return SYRK_ERR_PLAN;
    std::lock_guard<std::mutex> lock(runtime().mu);
    runtime().f64_tail_slices = slices;
    runtime().f64_tail_items = tail_items;
    return SYRK_OK;
}

int syrk_set_split_k(int slices) {
    if (slices < 0 || slices > 1024) return SYRK_ERR_PLAN;
    std::lock_guard<std::mutex> lock(runtime().mu);
    runtime().split_k = slices;
    return SYRK_OK;
}

int syrk_get_schedule_stats(int64_t N, int64_t M, int dtype, syrk_schedule_stats* out) {
    if (!out) return SYRK_ERR_NULL;
    if (!known_dtype(dtype)) return SYRK_ERR_DTYPE;
    if (N < 0 || M < 0) return SYRK_ERR_SIZE;
    int schedule;
    { std::lock_guard<std::mutex> lock(runtime().mu); schedule = runtime().schedule; }
    Plan plan;
    if (!build_host_plan(N, dtype, schedule, &plan)) return SYRK_ERR_PLAN;
    const KernelShape ks = kernel_shape(dtype);
    const SimResult sim = simulate_plan(plan, N, M, ks.tile);
    std::memset(out, 0, sizeof(*out));
    out->tile = ks.tile;
    out->k = ks.k;
    out->c = int32_t(plan.c_top);
    int split = 1;
    out->effective_schedule = effective_schedule_of(N, M, dtype, 148, &split);
    out->split_k = split;
    out->launches = split > 1 ? 2 : 1;
    bool f64_persistent = false;
    if (dtype == SYRK_DTYPE_F64 && split == 1 && out->effective_schedule != SYRK_SCHEDULE_PAIR_SQUARE) {
        // the tail K-split (either launch form) adds its reduction kernel; the launch form is taken as for
        // beta == 0 or 1
        int mode, tail_setting;
        { std::lock_guard<std::mutex> lock(runtime().mu); mode = runtime().f64_launch; tail_setting = runtime().f64_tail_slices; }
        const int64_t n_items = int64_t(plan.items.size());
        const bool per_item = mode == SYRK_F64_LAUNCH_PER_ITEM ||
                              (mode == SYRK_F64_LAUNCH_AUTO && !f64_persistent_pays(n_items, 0.0, 148));
        if (tail_setting == 0 && plan_tail_split_f64(plan.items, (M + ks.bk - 1) / ks.bk, 148).slices > 1)
            out->launches = 2;
        f64_persistent = !per_item;
    }
    out->n_tiles = plan.p.n_tiles;
    out->items = int64_t(plan.items.size());
    out->tri_items = plan.n_tri;
    out->rect_items = plan.n_rect;
    out->diag_items = plan.n_diag;
    out->tri_tiles = plan.tri_tiles;
    out->all_tiles = plan.p.n_tiles * (plan.p.n_tiles + 1) / 2;
    out->a_loads = sim.a_loads;
    out->c_elems = N * (N + 1) / 2;
    out->s_acc = ks.s_acc;
    out->s_total = ks.s_acc + int64_t(kMaxSeg) * ks.tile * ks.bk * ks.stages;
    if (is_tcgen05_dtype(dtype)) out->s_total = ks.s_acc + int64_t(bf16_seg_slots()) * ks.tile * ks.bk * ks.stages;
    // the persistent FP64 form: the accumulators, their shared-memory image, and its shorter ring of stages
    if (f64_persistent) out->s_total = 2 * ks.s_acc + int64_t(kMaxSeg) * ks.tile * ks.bk * f64_persistent_stages();
    return SYRK_OK;
}

void* tbs_plan_build(int64_t n_tiles, int k, int rect_rows, int rect_cols, int diag_side, int schedule) {
    PlanParams p;
    p.n_tiles = n_tiles; p.k = k; p.rect_rows = rect_rows; p.rect_cols = rect_cols;
    p.diag_side = diag_side; p.schedule = schedule;
    Plan* plan = new (std::nothrow) Plan();
    if (!plan) return nullptr;
    if (!build_plan(p, plan)) { delete plan; return nullptr; }
    return plan;
}

int tbs_plan_balance(void* plan, int slots) {
    if (!plan) return SYRK_ERR_NULL;
    if (slots < 1) return SYRK_ERR_SIZE;
    balance_for_slots(static_cast<Plan*>(plan), slots);
    return SYRK_OK;
}

int64_t tbs_plan_num_items(const void* plan) {
    return plan ? int64_t(static_cast<const Plan*>(plan)->items.size()) : SYRK_ERR_NULL;
}

int tbs_plan_item(const void* plan, int64_t index, int32_t* kind, int32_t* n_seg, int32_t seg[TBS_MAX_SEG],
                  int32_t* n_tile, int32_t tile_x[TBS_MAX_TILE], int32_t tile_y[TBS_MAX_TILE]) {
    if (!plan || !kind || !n_seg || !seg || !n_tile || !tile_x || !tile_y) return SYRK_ERR_NULL;
    const Plan* p = static_cast<const Plan*>(plan);
    if (index < 0 || index >= int64_t(p->items.size())) return SYRK_ERR_SIZE;
    const WorkItem& it = p->items[size_t(index)];
    *kind = it.kind; *n_seg = it.n_seg; *n_tile = it.n_tile;
    for (int s = 0; s < TBS_MAX_SEG; ++s) seg[s] = s < it.n_seg ? it.seg[s] : -1;
    for (int t = 0; t < TBS_MAX_TILE; ++t) {
        tile_x[t] = t < it.n_tile ? it.tile_x[t] : -1;
        tile_y[t] = t < it.n_tile ? it.tile_y[t] : -1;
    }
    return SYRK_OK;
}

void tbs_plan_free(void* plan) { delete static_cast<Plan*>(plan); }

int tbs_plan_simulate(const void* plan, int64_t N, int64_t M, int b, int64_t* a_loads, int64_t* c_loads,
                      int32_t* min_cover, int32_t* max_cover, int32_t* upper_cover) {
    if (!plan) return SYRK_ERR_NULL;
    const Plan* p = static_cast<const Plan*>(plan);
    if (N < 0 || M < 0 || b < 1 || (N + b - 1) / b != p->p.n_tiles) return SYRK_ERR_SIZE;
    const SimResult r = simulate_plan(*p, N, M, b);
    if (a_loads) *a_loads = r.a_loads;
    if (c_loads) *c_loads = r.c_loads;
    if (min_cover) *min_cover = r.min_cover;
    if (max_cover) *max_cover = r.max_cover;
    if (upper_cover) *upper_cover = r.upper_cover;
    return SYRK_OK;
}

}  // extern "C"
