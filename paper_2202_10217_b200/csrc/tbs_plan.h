// Work items of the tiled triangle-block schedule: the host generator's output
// and the kernels' input.  Host/device shared POD, no CUDA types.
#pragma once
#include <cstdint>
#include <vector>

namespace tbsyrk {

constexpr int kMaxSeg = 8;    // row segments an item may hold in shared memory
constexpr int kMaxTile = 16;  // output tiles an item may own

enum ItemKind : int32_t { kTri = 0, kRect = 1, kDiag = 2 };

// One unit of work: a set of tile rows ("segments") streamed along M, and the
// output tiles C[seg[tile_x[t]], seg[tile_y[t]]] accumulated from them.
// For a triangle block (Section 3.2 of the paper) the tiles are all pairs x > y.
struct alignas(16) WorkItem {
    int32_t seg[kMaxSeg];
    uint8_t tile_x[kMaxTile];
    uint8_t tile_y[kMaxTile];
    int32_t n_seg;
    int32_t n_tile;
    int32_t kind;
    int32_t pad;
};
static_assert(sizeof(WorkItem) == 80, "WorkItem layout is part of the kernel ABI");

struct PlanParams {
    int64_t n_tiles = 0;  // tile rows of C
    int k = 3;            // segments per triangle block
    int rect_rows = 2;    // square-block fallback: rows x cols tiles per item
    int rect_cols = 2;
    int diag_side = 2;    // adjacent tile rows per diagonal item and per band (>= rect_rows)
    int schedule = 0;     // 0: triangle blocks + leftovers, 1: squares only
};

struct Plan {
    PlanParams p;
    int64_t c_top = 0;  // zone side used at the top level (0: no triangle blocks)
    std::vector<WorkItem> items;
    int64_t n_tri = 0, n_rect = 0, n_diag = 0, tri_tiles = 0;
};

// Product of the primes <= k-2, and the largest c <= floor(n/k) coprime with it.
int64_t primes_product_upto(int k_minus_2);
int64_t pick_zone_side(int64_t n, int k);

// Builds the item list; returns false on invalid parameters.
bool build_plan(const PlanParams& p, Plan* out);

// Ordering for a machine that runs `slots` items at a time, each item costing about its tile
// count (ours; the paper's block loop is order-free): heaviest first, and enough full
// rect_rows x rect_cols rectangles at the end cut into quarters to leave about half a wave of
// small items that fill the last wave evenly.  Coverage is unchanged.
void balance_for_slots(Plan* plan, int slots);

// Two-level-model replay (Section 3): elements of A and C moved, tile coverage.
struct SimResult {
    int64_t a_loads = 0, c_loads = 0;
    int32_t min_cover = 0, max_cover = 0, upper_cover = 0;
};
SimResult simulate_plan(const Plan& plan, int64_t N, int64_t M, int b);

}  // namespace tbsyrk
