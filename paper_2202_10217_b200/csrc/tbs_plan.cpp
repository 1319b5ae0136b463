// Host-side block-set generator for the tiled triangle-block schedule.
//
// Follows Algorithm 4 (TBS) of the paper in its tiled form (Section 5.1.4), with
// tile rows in the place of matrix rows:
//   q  = product of the primes <= k-2,   c = largest integer <= n/k coprime with q,
//   l  = n - c*k.
//   c < k-1  : the whole triangle is done with square and diagonal blocks;
//   otherwise: square blocks for the last l tile rows, a recursive call for each
//              of the k diagonal zones [u*c, (u+1)*c), and c*c triangle blocks with
//              rows  r_u = u*c + f(u),  f(0) = j,  f(u) = (i + j*(u-1)) mod c
//              (cyclic indexing family, Section 5.1.2).
// Integer arithmetic only.  The square-block fallback is only cited by the paper;
// here it is a band decomposition: bands of `diag_side` tile rows, each cut into
// rect_rows x rect_cols rectangles left of the diagonal plus one diagonal block.
#include "tbs_plan.h"

#include <algorithm>
#include <numeric>

namespace tbsyrk {

int64_t primes_product_upto(int m) {
    int64_t q = 1;
    for (int p = 2; p <= m; ++p) {
        bool prime = true;
        for (int d = 2; d * d <= p; ++d)
            if (p % d == 0) { prime = false; break; }
        if (prime) q *= p;
    }
    return q;
}

int64_t pick_zone_side(int64_t n, int k) {
    const int64_t q = primes_product_upto(k - 2);
    for (int64_t c = n / k; c >= 1; --c)
        if (std::gcd(c, q) == 1) return c;
    return 0;
}

namespace {

struct Builder {
    const PlanParams& p;
    Plan* plan;

    void push(WorkItem& it) {
        it.pad = 0;
        plan->items.push_back(it);
        if (it.kind == kTri) { plan->n_tri++; plan->tri_tiles += it.n_tile; }
        else if (it.kind == kRect) plan->n_rect++;
        else plan->n_diag++;
    }

    // rows [r0, r1) x cols [c0, c1), entirely below the diagonal (c1 <= r0)
    void rect_item(int64_t r0, int64_t r1, int64_t c0, int64_t c1) {
        WorkItem it{};
        it.kind = kRect;
        const int nc = int(c1 - c0), nr = int(r1 - r0);
        for (int y = 0; y < nc; ++y) it.seg[y] = int32_t(c0 + y);
        for (int x = 0; x < nr; ++x) it.seg[nc + x] = int32_t(r0 + x);
        it.n_seg = nc + nr;
        int t = 0;
        for (int x = 0; x < nr; ++x)
            for (int y = 0; y < nc; ++y) {
                it.tile_x[t] = uint8_t(nc + x);
                it.tile_y[t] = uint8_t(y);
                ++t;
            }
        it.n_tile = t;
        push(it);
    }

    // lower triangle, diagonal tiles included, of tile rows [r0, r1)
    void diag_item(int64_t r0, int64_t r1) {
        WorkItem it{};
        it.kind = kDiag;
        const int n = int(r1 - r0);
        for (int x = 0; x < n; ++x) it.seg[x] = int32_t(r0 + x);
        it.n_seg = n;
        int t = 0;
        for (int x = 0; x < n; ++x)
            for (int y = 0; y <= x; ++y) {
                it.tile_x[t] = uint8_t(x);
                it.tile_y[t] = uint8_t(y);
                ++t;
            }
        it.n_tile = t;
        push(it);
    }

    // {(r, t) : row_lo <= r < row_hi, col_lo <= t <= r}, col_lo <= row_lo
    void square_blocks(int64_t row_lo, int64_t row_hi, int64_t col_lo) {
        for (int64_t r0 = row_lo; r0 < row_hi; r0 += p.diag_side) {
            const int64_t r1 = std::min<int64_t>(r0 + p.diag_side, row_hi);
            for (int64_t q0 = r0; q0 < r1; q0 += p.rect_rows)
                for (int64_t c0 = col_lo; c0 < r0; c0 += p.rect_cols)
                    rect_item(q0, std::min<int64_t>(q0 + p.rect_rows, r1), c0,
                              std::min<int64_t>(c0 + p.rect_cols, r0));
            diag_item(r0, r1);
        }
    }

    void triangle_blocks(int64_t base, int64_t c) {
        const int k = p.k;
        // Blocks are emitted in square patches of the (i, j) index space: blocks of a
        // patch share many rows (zone 0 depends on j only, zone 1 on i only), which
        // keeps the rows that co-running thread blocks stream close together in L2.
        const int64_t patch = 12;
        for (int64_t i0 = 0; i0 < c; i0 += patch)
            for (int64_t j0 = 0; j0 < c; j0 += patch)
                for (int64_t i = i0; i < std::min(i0 + patch, c); ++i)
                    for (int64_t j = j0; j < std::min(j0 + patch, c); ++j) {
                        WorkItem it{};
                        it.kind = kTri;
                        it.n_seg = k;
                        for (int u = 0; u < k; ++u) {
                            const int64_t f = (u == 0) ? j : (i + j * int64_t(u - 1)) % c;
                            it.seg[u] = int32_t(base + u * c + f);
                        }
                        int t = 0;
                        for (int x = 1; x < k; ++x)
                            for (int y = 0; y < x; ++y) {
                                it.tile_x[t] = uint8_t(x);
                                it.tile_y[t] = uint8_t(y);
                                ++t;
                            }
                        it.n_tile = t;
                        push(it);
                    }
    }

    void tbs(int64_t base, int64_t n, bool top) {
        const int64_t c = (p.schedule == 0) ? pick_zone_side(n, p.k) : 0;
        if (c < p.k - 1) {  // c is too small: squares only
            square_blocks(base, base + n, base);
            return;
        }
        if (top) plan->c_top = c;
        triangle_blocks(base, c);
        for (int u = 0; u < p.k; ++u) tbs(base + u * c, c, false);
        square_blocks(base + c * p.k, base + n, base);  // the last l tile rows
    }
};

}  // namespace

bool build_plan(const PlanParams& p, Plan* out) {
    if (p.n_tiles < 0 || p.n_tiles > (int64_t(1) << 30)) return false;
    if (p.k < 2 || p.k > kMaxSeg || p.k * (p.k - 1) / 2 > kMaxTile) return false;
    if (p.rect_rows < 1 || p.rect_cols < 1 || p.rect_rows + p.rect_cols > kMaxSeg ||
        p.rect_rows * p.rect_cols > kMaxTile)
        return false;
    if (p.diag_side < p.rect_rows || p.diag_side > kMaxSeg || p.diag_side * (p.diag_side + 1) / 2 > kMaxTile) return false;
    if (p.schedule != 0 && p.schedule != 1) return false;
    out->p = p;
    out->c_top = 0;
    out->items.clear();
    out->n_tri = out->n_rect = out->n_diag = out->tri_tiles = 0;
    Builder b{p, out};
    if (p.n_tiles > 0) b.tbs(0, p.n_tiles, true);
    return true;
}

void balance_for_slots(Plan* plan, int slots) {
    auto by_cost = [](const WorkItem& a, const WorkItem& b) { return a.n_tile > b.n_tile; };
    std::stable_sort(plan->items.begin(), plan->items.end(), by_cost);
    const PlanParams& p = plan->p;
    const int full = p.rect_rows * p.rect_cols;
    if (slots <= 0 || p.rect_rows % 2 != 0 || p.rect_cols % 2 != 0 || full < 4) return;
    int64_t total = 0;
    for (const WorkItem& it : plan->items) total += it.n_tile;
    if (total < int64_t(slots) * full) return;            // less than one wave: nothing to even out
    const int64_t want = int64_t(slots) * full / 2;        // tiles to turn into small items
    std::vector<WorkItem> out, small;
    int64_t cut = 0;
    for (auto it = plan->items.rbegin(); it != plan->items.rend(); ++it) {
        if (cut < want && it->kind == kRect && it->n_tile == full) {
            const int nc = p.rect_cols, nr = p.rect_rows;  // seg = [cols..., rows...]
            for (int qr = 0; qr < 2; ++qr)
                for (int qc = 0; qc < 2; ++qc) {
                    WorkItem q{};
                    q.kind = kRect;
                    const int hc = nc / 2, hr = nr / 2;
                    for (int y = 0; y < hc; ++y) q.seg[y] = it->seg[qc * hc + y];
                    for (int x = 0; x < hr; ++x) q.seg[hc + x] = it->seg[nc + qr * hr + x];
                    q.n_seg = hc + hr;
                    int t = 0;
                    for (int x = 0; x < hr; ++x)
                        for (int y = 0; y < hc; ++y) { q.tile_x[t] = uint8_t(hc + x); q.tile_y[t] = uint8_t(y); ++t; }
                    q.n_tile = t;
                    small.push_back(q);
                }
            cut += full;
            plan->n_rect += 3;
        } else {
            out.push_back(*it);
        }
    }
    std::reverse(out.begin(), out.end());
    out.insert(out.end(), small.begin(), small.end());
    std::stable_sort(out.begin(), out.end(), by_cost);
    plan->items.swap(out);
}

SimResult simulate_plan(const Plan& plan, int64_t N, int64_t M, int b) {
    SimResult r;
    const int64_t nt = plan.p.n_tiles;
    auto height = [&](int64_t t) -> int64_t {
        const int64_t h = N - t * int64_t(b);
        return h <= 0 ? 0 : std::min<int64_t>(h, b);
    };
    std::vector<int32_t> cover(size_t(nt) * size_t(nt), 0);
    for (const WorkItem& it : plan.items) {
        for (int s = 0; s < it.n_seg; ++s) r.a_loads += height(it.seg[s]) * M;
        for (int t = 0; t < it.n_tile; ++t) {
            const int64_t x = it.seg[it.tile_x[t]], y = it.seg[it.tile_y[t]];
            cover[size_t(x) * nt + y] += 1;
            r.c_loads += (x == y) ? height(x) * (height(x) + 1) / 2 : height(x) * height(y);
        }
    }
    r.min_cover = nt > 0 ? INT32_MAX : 0;
    for (int64_t x = 0; x < nt; ++x)
        for (int64_t y = 0; y < nt; ++y) {
            const int32_t v = cover[size_t(x) * nt + y];
            if (y <= x) { r.min_cover = std::min(r.min_cover, v); r.max_cover = std::max(r.max_cover, v); }
            else r.upper_cover = std::max(r.upper_cover, v);
        }
    return r;
}

}  // namespace tbsyrk
