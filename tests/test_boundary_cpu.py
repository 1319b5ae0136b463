"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol,
and its host-side work lists agree with the integer reference of the schedule."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import tbs as T
from paper_2202_10217_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    from paper_2202_10217_b200 import build
    build.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "tbsyrk.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b((?:syrk|syr2k|herk|tbs|cholesky)_[a-z_0-9]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    L = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(L, name), name


def test_strerror_and_argument_validation_need_no_device():
    assert B.strerror(0) == "success"
    L = B.lib()
    one = ctypes.c_double(0.0)
    p = ctypes.addressof(one)
    assert L.syrk_lower(-1, 4, p, 4, p, 4, 1.0, 0.0, 0, None) == -2          # negative N
    assert L.syrk_lower(4, 4, p, 3, p, 4, 1.0, 0.0, 0, None) == -3           # lda < M
    assert L.syrk_lower(4, 4, p, 4, p, 3, 1.0, 0.0, 0, None) == -3           # ldc < N
    assert L.syrk_lower(4, 4, None, 4, p, 4, 1.0, 0.0, 0, None) == -1        # null A
    assert L.syrk_lower(4, 4, p, 4, None, 4, 1.0, 0.0, 0, None) == -1        # null C
    assert L.syrk_lower(4, 4, p, 4, p, 4, 1.0, 0.0, 7, None) == -4           # dtype
    assert L.syrk_lower(0, 4, None, 4, None, 1, 1.0, 0.0, 0, None) == 0      # N == 0
    assert L.syrk_ex(2, 0, 4, 4, p, 4, p, 4, 1.0, 0.0, 0, None) == -2           # unknown uplo
    assert L.syrk_ex(1, 3, 4, 4, p, 4, p, 4, 1.0, 0.0, 0, None) == -2           # unknown trans
    assert L.syrk_ex(1, 1, 4, 8, p, 3, p, 4, 1.0, 0.0, 0, None) == -3           # M x N operand: lda < N
    assert L.syrk_ex(1, 0, 0, 8, None, 8, None, 1, 1.0, 0.0, 0, None) == 0      # N == 0
    assert L.syrk_lower_batched(-1, 4, 4, p, 4, 16, p, 4, 16, 1.0, 0.0, 0, None) == -2      # negative batch
    assert L.syrk_lower_batched(3, 4, 4, p, 4, 15, p, 4, 16, 1.0, 0.0, 0, None) == -3       # matrices of A overlap
    assert L.syrk_lower_batched(3, 4, 4, p, 4, 16, p, 4, 15, 1.0, 0.0, 0, None) == -3       # matrices of C overlap
    assert L.syrk_lower_batched(0, 4, 4, None, 4, 16, None, 4, 16, 1.0, 0.0, 0, None) == -1  # arguments are still checked
    assert L.syrk_lower_batched(0, 4, 4, p, 4, 16, p, 4, 16, 1.0, 0.0, 0, None) == 0        # empty batch
    assert L.syrk_set_schedule(5) == -7
    assert B.Plan.__init__ is not None
    with pytest.raises(B.SyrkError):
        B.Plan(10, 9, 2, 2, 2)                                                # k(k-1)/2 tiles > 16


def test_balancing_keeps_exact_once_coverage_and_puts_small_items_last():
    for n_t, k, rr, rc in [(128, 6, 4, 4), (40, 6, 4, 4), (257, 6, 4, 4), (64, 3, 2, 2), (31, 4, 2, 4)]:
        plan = B.Plan(n_t, k, rr, rc, rr)
        before = len(plan)
        plan.balance(148)
        cover = np.zeros((n_t, n_t), dtype=np.int64)
        sizes = []
        for kind, seg, pairs in plan_ops(plan):
            sizes.append(len(pairs))
            assert len(set(seg)) == len(seg)
            for (r, t) in pairs:
                cover[r, t] += 1
        assert np.array_equal(cover, np.tril(np.ones((n_t, n_t), dtype=np.int64)))
        assert sizes == sorted(sizes, reverse=True) and len(plan) >= before
        plan.close()


def plan_ops(plan):
    """Library work list -> operations of the reference simulator."""
    ops = []
    for idx in range(len(plan)):
        kind, seg, tiles = plan.item(idx)
        pairs = [(seg[x], seg[y]) for x, y in tiles]
        ops.append((kind, seg, pairs))
    return ops


@pytest.mark.parametrize("k,rr,rc,dg", [(3, 2, 2, 2), (6, 4, 4, 4), (4, 3, 3, 3), (5, 4, 4, 4), (3, 1, 2, 2), (4, 2, 3, 5)])
@pytest.mark.parametrize("schedule", [B.SCHEDULE_TBS, B.SCHEDULE_SQUARE])
def test_work_list_covers_every_tile_exactly_once(k, rr, rc, dg, schedule):
    for n_t in list(range(0, 41)) + [64, 128, 131, 256]:
        plan = B.Plan(n_t, k, rr, rc, dg, schedule)
        cover = np.zeros((n_t, n_t), dtype=np.int64)
        for kind, seg, pairs in plan_ops(plan):
            assert len(set(seg)) == len(seg) and all(0 <= s < n_t for s in seg)
            for (r, t) in pairs:
                assert r >= t
                cover[r, t] += 1
            if kind == B.ITEM_TRI:      # a triangle block: all pairs of its k segments, no diagonal
                assert len(seg) == k and sorted(pairs) == sorted(T.triangle_block(seg))
        assert np.array_equal(cover, np.tril(np.ones((n_t, n_t), dtype=np.int64))), (n_t, k)
        b = 8
        N = max(n_t * b - 3, 0) if n_t else 0
        sim = plan.simulate(N, 5, b)
        if n_t:
            assert (sim["min_cover"], sim["max_cover"], sim["upper_cover"]) == (1, 1, 0)
            assert sim["c_loads"] == N * (N + 1) // 2
        plan.close()


@pytest.mark.parametrize("k", [3, 4, 6])
def test_triangle_blocks_are_those_of_the_reference_schedule(k):
    """Same block sets as Algorithm 4 with the cyclic family (order aside), and the
    library's own load count equals the reference simulator's on the library's list."""
    b, M = 8, 7
    for n_t in [k * (k - 1), 32, 57, 128]:
        N = n_t * b - 1
        plan = B.Plan(n_t, k, 2, 2, 2)
        ops = plan_ops(plan)
        mine = sorted(tuple(seg) for kind, seg, _ in ops if kind == B.ITEM_TRI)
        ref_ops, w, _ = T.tiled_schedule(N, b, k)
        theirs = sorted(tuple(op[1]) for op in ref_ops if op[0] == "tb")
        assert mine == theirs and len(mine) > 0
        a_ref = sum(sum(w[s] for s in seg) for _, seg, _ in ops) * M
        sim = plan.simulate(N, M, b)
        assert sim["a_loads"] == a_ref
        # replay through the reference simulator as generic operations
        generic = []
        for kind, seg, pairs in ops:
            if kind == B.ITEM_TRI:
                generic.append(("tb", seg))
            elif kind == B.ITEM_DIAG:
                generic.append(("diag", seg))
            else:
                generic.append(("rect", sorted({r for r, _ in pairs}), sorted({t for _, t in pairs})))
        cover, a_loads, c_loads = T.simulate(generic, n_t, M, w)
        assert a_loads == sim["a_loads"] and c_loads == sim["c_loads"] == N * (N + 1) // 2
        plan.close()


def test_schedule_stats_for_the_benchmark_shapes():
    st = B.syrk_get_schedule_stats(4096, 4096, B.DTYPE_F64)
    assert st["tile"] == 32 and st["k"] == 6 and st["n_tiles"] == 128 and st["c"] == 19
    assert st["tri_items"] == 361 and st["tri_tiles"] == 361 * 15
    assert st["all_tiles"] == 128 * 129 // 2 and st["c_elems"] == 4096 * 4097 // 2
    st = B.syrk_get_schedule_stats(16384, 4096, B.DTYPE_BF16_F32)
    assert st["tile"] == 128 and st["k"] == 3 and st["n_tiles"] == 128 and st["c"] == 42
    # triangle blocks stream fewer rows of A than squares of the same accumulator budget
    B.syrk_set_schedule(B.SCHEDULE_SQUARE)
    sq = B.syrk_get_schedule_stats(4096, 4096, B.DTYPE_F64)
    B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
    tb = B.syrk_get_schedule_stats(4096, 4096, B.DTYPE_F64)
    assert sq["tri_items"] == 0 and tb["a_loads"] < sq["a_loads"]


def test_effective_schedule_follows_the_size_rule():
    """Default setting: triangle blocks once the list is long (N large against the block side, as the
    paper's tiled scheme asks), square blocks on CTA pairs below, binary64 always on triangle blocks; an
    explicit setting is reported as set, with the single-CTA square list where the pair form has too
    few blocks."""
    assert B.syrk_effective_schedule(16384, 4096, B.DTYPE_BF16_F32) == B.SCHEDULE_TBS          # 2848 items
    assert B.syrk_effective_schedule(2048, 262144, B.DTYPE_BF16_F32) == B.SCHEDULE_PAIR_SQUARE  # 55 items
    assert B.syrk_effective_schedule(7168, 4096, B.DTYPE_E4M3_F32) == B.SCHEDULE_PAIR_SQUARE
    assert B.syrk_effective_schedule(8192, 4096, B.DTYPE_F16_F32) == B.SCHEDULE_TBS
    assert B.syrk_effective_schedule(300, 64, B.DTYPE_BF16_F32) == B.SCHEDULE_TBS               # too few blocks for the pairs
    assert B.syrk_effective_schedule(4096, 4096, B.DTYPE_F64) == B.SCHEDULE_TBS
    assert B.syrk_effective_schedule(512, 0, B.DTYPE_BF16_F32) == B.SCHEDULE_TBS
    try:
        B.syrk_set_schedule(B.SCHEDULE_TBS)
        assert B.syrk_effective_schedule(2048, 262144, B.DTYPE_BF16_F32) == B.SCHEDULE_TBS
        B.syrk_set_schedule(B.SCHEDULE_PAIR_SQUARE)
        assert B.syrk_effective_schedule(16384, 4096, B.DTYPE_BF16_F32) == B.SCHEDULE_PAIR_SQUARE
        assert B.syrk_effective_schedule(300, 64, B.DTYPE_BF16_F32) == B.SCHEDULE_SQUARE
        assert B.syrk_effective_schedule(4096, 4096, B.DTYPE_F64) == B.SCHEDULE_SQUARE
        B.syrk_set_schedule(B.SCHEDULE_SQUARE)
        assert B.syrk_effective_schedule(16384, 4096, B.DTYPE_BF16_F32) == B.SCHEDULE_SQUARE
    finally:
        B.syrk_set_schedule(B.SCHEDULE_DEFAULT)
    with pytest.raises(B.SyrkError):
        B.syrk_effective_schedule(-1, 4, B.DTYPE_F64)
    with pytest.raises(B.SyrkError):
        B.syrk_effective_schedule(4, 4, 9)
