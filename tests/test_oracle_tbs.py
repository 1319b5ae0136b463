"""Pins for the integer schedule reference (oracle/tbs.py), CPU only.

Brute force on small sizes, the paper's definitions checked exhaustively, and the
load count compared with a closed-form recurrence evaluated without simulation.
"""
import math
import os

import numpy as np
import pytest

from oracle import tbs as T

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def exact_lower_once(cover):
    n = cover.shape[0]
    return np.array_equal(cover, np.tril(np.ones((n, n), dtype=cover.dtype)))


# ---- Section 3.2 -----------------------------------------------------------------

def test_sigma_closed_form_against_brute_force():
    for m in range(0, 10001):
        s = 0
        while s * (s - 1) // 2 < m:
            s += 1
        assert T.sigma(m) == s
        if m > 0:
            assert T.sigma(m) == math.ceil(math.sqrt(0.25 + 2 * m) + 0.5)


def test_triangle_block_size_and_footprint():
    R = [3, 11, 4, 20, 7]
    tb = T.triangle_block(R)
    assert len(tb) == len(R) * (len(R) - 1) // 2 == len(set(tb))
    assert all(r > rp for r, rp in tb)
    assert {x for pair in tb for x in pair} == set(R)


# ---- Section 5.1.2 ----------------------------------------------------------------

def test_cyclic_family_hand_values():
    for line in open(os.path.join(GOLDEN, "cyclic_family_c5_k4.txt")):
        if line.startswith("#"):
            continue
        i, j, *f = map(int, line.split())
        assert [T.cyclic_f(i, j, u, 5) for u in range(4)] == f


def test_q_is_product_of_primes_up_to_k_minus_2():
    assert [T.q_of(k) for k in range(2, 12)] == [1, 1, 2, 6, 6, 30, 30, 210, 210, 210]


def family_is_valid(c, k):
    """Validity definition: two distinct (i, j) never agree at two positions u != v."""
    seen = set()
    for i in range(c):
        for j in range(c):
            f = [T.cyclic_f(i, j, u, c) for u in range(k)]
            assert f[0] == j and f[1] == i and all(0 <= x < c for x in f)   # indexing family
            for u in range(k):
                for v in range(u + 1, k):
                    key = (u, v, f[u], f[v])
                    if key in seen:
                        return False
                    seen.add(key)
    return True


def test_cyclic_family_valid_when_c_coprime_with_q():
    for k in range(3, 10):
        q = T.q_of(k)
        for c in range(k - 1, 41):
            if math.gcd(c, q) == 1:
                assert family_is_valid(c, k), (c, k)


def test_cyclic_family_invalid_when_c_shares_a_factor():
    assert not family_is_valid(4, 4)      # 2 | 4 and 2 in [2, k-2]
    assert not family_is_valid(9, 5)      # 3 | 9 and 3 in [2, k-2]
    assert not family_is_valid(10, 7)     # 5 | 10


def test_choose_c():
    assert T.choose_c(128, 6) == 19       # floor(128/6) = 21; 21, 20 share factors with 6
    assert T.choose_c(32, 3) == 10
    assert T.choose_c(5, 6) == 0
    for k in range(3, 9):
        for N in range(1, 200):
            c = T.choose_c(N, k)
            assert c * k <= N and (c == 0 or math.gcd(c, T.q_of(k)) == 1)
            assert all(math.gcd(d, T.q_of(k)) != 1 for d in range(c + 1, N // k + 1))


# ---- Section 5.1.1: zones and blocks ------------------------------------------------

@pytest.mark.parametrize("k,c", [(3, 2), (3, 7), (4, 5), (5, 7), (6, 11), (8, 7)])
def test_blocks_tile_the_square_zones_exactly(k, c):
    n = c * k
    cover = np.zeros((n, n), dtype=np.int64)
    per_row = np.zeros(n, dtype=np.int64)
    for i in range(c):
        for j in range(c):
            R = T.block_rows(i, j, c, k)
            assert [r // c for r in R] == list(range(k))            # one row per zone row
            assert (R[1], R[0]) == (i + c, j)                        # contains (i + c, j)
            for r in R:
                per_row[r] += 1
            for (r, rp) in T.triangle_block(R):
                cover[r, rp] += 1
    assert np.all(per_row == c)                                      # each row is in c blocks
    want = np.zeros_like(cover)
    for r in range(n):
        for t in range(n):
            if r // c > t // c:                                      # the k(k-1)/2 square zones
                want[r, t] = 1
    assert np.array_equal(cover, want)
    assert cover.sum() == c * c * k * (k - 1) // 2


# ---- Algorithm 4: exact-once coverage ------------------------------------------------

@pytest.mark.parametrize("k", [3, 4, 5, 6, 7, 8])
def test_element_level_covers_lower_triangle_exactly_once(k):
    for N in list(range(1, 60)) + [97, 128, 200, 301]:
        ops, S = T.element_schedule(N, k)
        cover, a_loads, c_loads = T.simulate(ops, N, 1)
        assert exact_lower_once(cover), (N, k)
        assert c_loads == N * (N + 1) // 2                           # every entry loaded once
        for op in ops:                                               # fast memory is respected
            held = len(T.op_entries(op)) + len(T.op_rows(op))
            assert held <= S, (op[0], held, S)
        # diagonal entries are produced by the square-block fallback only
        assert all(r != t for op in ops if op[0] == "tb" for r, t in T.op_entries(op))


@pytest.mark.parametrize("k", [3, 4, 5, 6, 8])
def test_tile_level_covers_exactly_once_with_ragged_edge(k):
    b = 8
    for n_t in list(range(1, 70)) + [128, 256]:
        N = n_t * b - 3                                              # last tile has 5 rows
        ops, w, S = T.tiled_schedule(N, b, k)
        assert len(w) == n_t and sum(w) == N
        cover, a_loads, c_loads = T.simulate(ops, n_t, 1, w)
        assert exact_lower_once(cover), (n_t, k)
        assert c_loads == N * (N + 1) // 2
        for op in ops:
            tiles = len(T.op_entries(op))
            assert tiles * b * b <= S


# ---- Section 5.1.3 / 5.1.4: load counts ------------------------------------------------

def strip_loads_closed_form(row_lo, row_hi, col_lo, s):
    """Loads per column of the square-block cover, by counting squares (no simulation)."""
    l = row_hi - row_lo
    if l <= 0:
        return 0
    width = row_lo - col_lo
    n_r = -(-l // s)
    n_c = -(-width // s)
    total = n_c * l + n_r * width                  # rectangle: every square loads rows + cols
    for m in range(n_r):
        h = min(s, l - m * s)
        total += m * (h + s) + h                    # m squares left of the diagonal one
    return total


def tbs_loads_closed_form(N, k, s):
    """Q(N) = c^2 k + k Q(c) + Q_squares(last l rows), per column of A."""
    c = T.choose_c(N, k)
    if c < k - 1:
        return strip_loads_closed_form(0, N, 0, s)
    return c * c * k + k * tbs_loads_closed_form(c, k, s) + strip_loads_closed_form(c * k, N, 0, s)


@pytest.mark.parametrize("k", [3, 4, 5, 6, 7])
def test_loads_equal_closed_form_recurrence_and_are_linear_in_M(k):
    S = k * (k + 1) // 2
    s = max(1, math.isqrt(S + 1) - 1)
    for N in [k, k * k, 37, 100, 257, 400]:
        ops, _ = T.element_schedule(N, k)
        per_col = tbs_loads_closed_form(N, k, s)
        for M in (1, 2, 3):
            _, a_loads, _ = T.simulate(ops, N, M)
            assert a_loads == per_col * M


def test_triangle_block_term_is_c2kM_and_bounded_by_N2M_over_k():
    for k in (4, 6):
        for N in (100, 333):
            c = T.choose_c(N, k)
            ops, _ = T.element_schedule(N, k)
            top = [op for op in ops if op[0] == "tb" and min(op[1]) < c <= (k - 1) * c <= max(op[1])]
            assert len(top) == c * c
            q1 = sum(len(T.op_rows(op)) for op in top)
            assert q1 == c * c * k <= N * N // k


@pytest.mark.parametrize("k", [4, 6, 9])
def test_total_volume_bound_and_convergence_to_lower_bound(k):
    """Q_A <= N^2 M/(k-1) + K0 N M log_k N with one frozen constant, and the
    ratio to the lower bound N^2 M / sqrt(2S) falls towards 1 as N grows."""
    S = k * (k + 1) // 2
    s = max(1, math.isqrt(S + 1) - 1)
    K0 = 4.0
    ratios = []
    for e in (2, 3, 4, 5):
        N = k ** e
        if N > 70000:
            break
        q = tbs_loads_closed_form(N, k, s)
        assert q <= N * N / (k - 1) + K0 * N * max(1.0, math.log(N, k))
        ratios.append(q / T.lower_bound(N, 1, S))
    assert all(a > b for a, b in zip(ratios, ratios[1:]))
    limit = math.sqrt(2 * S) / (k - 1)               # N^2/(k-1) over N^2/sqrt(2S)
    assert limit <= ratios[-1] < limit * 1.25


def test_square_only_schedule_matches_N2M_over_sqrtS():
    S = 120
    s = math.isqrt(S + 1) - 1
    N = 4000
    q = strip_loads_closed_form(0, N, 0, s)
    assert abs(q / (N * N / s) - 1.0) < 0.01          # leading term N^2 M / side
    ops = T.square_block_ops(0, 200, 0, s)
    cover, a_loads, _ = T.simulate(ops, 200, 1)
    assert exact_lower_once(cover) and a_loads == strip_loads_closed_form(0, 200, 0, s)


def test_tiled_leading_term():
    """Tiled variant: the c^2 blocks load k b M each; the whole schedule stays within
    N^2 M / ((k-1) b) plus a lower-order term, and beats squares at equal footprint."""
    b, k = 4, 6
    for n_t in (36, 216):
        N = n_t * b
        ops, w, S = T.tiled_schedule(N, b, k)
        _, a_loads, _ = T.simulate(ops, n_t, 1, w)
        c = T.choose_c(n_t, k)
        top = [op for op in ops if op[0] == "tb" and min(op[1]) < c <= (k - 1) * c <= max(op[1])]
        assert sum(len(T.op_rows(op)) * b for op in top) == c * c * k * b
        assert a_loads <= N * N / ((k - 1) * b) + 2.0 * N * math.log(N, k)
    sq = strip_loads_closed_form(0, N, 0, math.isqrt(S))
    assert a_loads < sq
