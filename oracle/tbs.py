"""Integer reference of the triangle-block schedule (TBS) and its I/O count.

TEST INFRASTRUCTURE ONLY: used by the tests (and nothing in the GPU library).
Pure Python / numpy, integer arithmetic only, written to be compared with the
paper by eye.  It shares no code with the library's own block-set generator.

What it follows
---------------
* Triangle block ``TB(R)`` - all sub-diagonal pairs of a row set R
  (Definition "Triangle block", Section 3.2).
* Zones and block rows ``R^{i,j} = {u*c + f^{i,j}(u)}`` (Eq. "def.blocks",
  Section 5.1.1) with the cyclic indexing family
  ``f(0) = j, f(u) = (i + j*(u-1)) mod c`` (Definition "cyclic", Section 5.1.2).
* ``q`` = product of the primes <= k-2 and ``c`` = the largest integer coprime
  with q that is <= N/k (Section 5.1.2, text after Algorithm 4).
* Algorithm 4 (TBS): square-block fallback when c < k-1; square blocks for the
  last l = N - c*k rows; recursion on the k diagonal zones; then the c*c
  triangle blocks, each streaming the M columns of its k rows.
* Tiled variant (Section 5.1.4): the same schedule over b x b tiles; a block
  still loads its k*b rows of A one column at a time.
* Two-level I/O accounting (Section 3): an operation that holds a set of C
  entries in fast memory and streams the columns of A loads, per column, one
  element for every row in the symmetric footprint of its entries.

Readings taken where the paper is silent (each also listed in the design notes):
* ``c`` is the largest c' in [1, floor(N/k)] with gcd(c', q) = 1; floor(N/k) = 0
  gives c = 0, i.e. the fallback.
* The zone range is half open, [u*c, (u+1)*c).
* "The last l rows of C" are rows c*k .. N-1 with columns 0 .. row.
* The square-block fallback (only cited in the paper) tiles its region with
  squares of side s, anchored at the region's first row/column; a square off the
  diagonal loads (rows + cols) elements of A per column, a diagonal square
  loads its rows once and updates its lower half including the diagonal.
  s is a parameter: s = floor(sqrt(S + 1)) - 1 (so that s*s + 2*s <= S) at
  element level.  Only the leading term N^2 M / sqrt(S) is fixed by the paper,
  so this detail is "parity unpinned" beyond exact-once coverage.
* Diagonal entries (i, i) are never in a triangle block; they are produced only
  by the square-block fallback.

Parity status: pinned by the CPU tests (exhaustive validity of the cyclic
family, exact-once coverage by brute force, block counts, the closed-form load
recurrence evaluated independently, linearity in M, convergence of the ratio to
the lower bound N^2 M / sqrt(2 S)).
"""
from __future__ import annotations

import math
from typing import Iterable, List, Sequence, Tuple

import numpy as np

Op = Tuple  # ("tb", rows) | ("rect", rows, cols) | ("diag", rows)


def sigma(m: int) -> int:
    """Smallest side of a triangle block with at least m entries (Lemma, Section 3.2)."""
    if m == 0:
        return 0
    # ceil(sqrt(1/4 + 2m) + 1/2), done in integers: smallest s with s(s-1)/2 >= m.
    s = (1 + math.isqrt(1 + 8 * m)) // 2
    while s * (s - 1) // 2 < m:
        s += 1
    while s > 0 and (s - 1) * (s - 2) // 2 >= m:
        s -= 1
    return s


def triangle_block(R: Sequence[int]) -> List[Tuple[int, int]]:
    """TB(R): every pair (r, r') of R with r > r'."""
    return [(r, rp) for r in R for rp in R if r > rp]


def q_of(k: int) -> int:
    """Product of all primes <= k-2 (1 when there is none)."""
    q = 1
    for p in range(2, k - 1):
        if all(p % d for d in range(2, int(math.isqrt(p)) + 1)):
            q *= p
    return q


def choose_c(N: int, k: int) -> int:
    """Largest c in [1, floor(N/k)] coprime with q(k); 0 when floor(N/k) == 0."""
    q = q_of(k)
    c = N // k
    while c >= 1 and math.gcd(c, q) != 1:
        c -= 1
    return max(c, 0)


def cyclic_f(i: int, j: int, u: int, c: int) -> int:
    """Cyclic (c, k)-indexing family."""
    return j if u == 0 else (i + j * (u - 1)) % c


def block_rows(i: int, j: int, c: int, k: int) -> List[int]:
    """Row indices R^{i,j} of block B^{i,j}: one row in each of the k zone rows."""
    return [u * c + cyclic_f(i, j, u, c) for u in range(k)]


def square_block_ops(row_lo: int, row_hi: int, col_lo: int, s: int) -> List[Op]:
    """Square-block cover of {(r, t): row_lo <= r < row_hi, col_lo <= t <= r}.

    Requires col_lo <= row_lo.  The part left of column row_lo is a rectangle cut
    into s x s squares; the part from column row_lo on is a lower triangle cut into
    diagonal squares and squares below them.
    """
    ops: List[Op] = []
    assert col_lo <= row_lo and s >= 1
    for r0 in range(row_lo, row_hi, s):
        rows = list(range(r0, min(r0 + s, row_hi)))
        for c0 in range(col_lo, row_lo, s):
            ops.append(("rect", rows, list(range(c0, min(c0 + s, row_lo)))))
        for c0 in range(row_lo, r0, s):
            ops.append(("rect", rows, list(range(c0, min(c0 + s, r0)))))
        ops.append(("diag", rows))
    return ops


def tbs_ops(N: int, k: int, s: int, base: int = 0) -> List[Op]:
    """Algorithm 4 on the N x N lower triangle that starts at global index ``base``.

    ``k`` is the side of a triangle block and ``s`` the side of the fallback's
    squares, both in index units (elements, or tiles for the tiled variant).
    """
    c = choose_c(N, k)
    if c < k - 1:                                   # c is too small
        return square_block_ops(base, base + N, base, s)
    ops: List[Op] = []
    ops += square_block_ops(base + c * k, base + N, base, s)   # the last l rows
    for u in range(k):                              # recursive calls, triangular zones
        ops += tbs_ops(c, k, s, base + u * c)
    for i in range(c):                              # loop over all blocks
        for j in range(c):
            ops.append(("tb", [base + r for r in block_rows(i, j, c, k)]))
    return ops


def op_entries(op: Op) -> List[Tuple[int, int]]:
    """C entries (index units) an operation holds in fast memory."""
    if op[0] == "tb":
        return triangle_block(op[1])
    if op[0] == "rect":
        return [(r, t) for r in op[1] for t in op[2]]
    if op[0] == "diag":
        return [(r, t) for r in op[1] for t in op[1] if r >= t]
    raise ValueError(op[0])


def op_rows(op: Op) -> List[int]:
    """Rows of A an operation loads for each column: the symmetric footprint."""
    if op[0] == "rect":
        return sorted(set(op[1]) | set(op[2]))
    return sorted(set(op[1]))


def simulate(ops: Iterable[Op], n: int, M: int, weights: Sequence[int] | None = None):
    """Replay a schedule in the two-level model.

    ``n`` is the number of index units (rows, or tile rows); ``weights[r]`` is the
    number of matrix rows unit r stands for (1 at element level, the tile height
    at tile level; the last tile may be ragged).  Returns ``(cover, a_loads,
    c_loads)``: an n x n int array counting how many operations hold each entry,
    the elements of A loaded, and the elements of C loaded.
    """
    w = np.ones(n, dtype=np.int64) if weights is None else np.asarray(weights, dtype=np.int64)
    cover = np.zeros((n, n), dtype=np.int64)
    a_loads = 0
    c_loads = 0
    for op in ops:
        for (r, t) in op_entries(op):
            cover[r, t] += 1
            c_loads += int(w[r] * (w[r] + 1) // 2) if r == t else int(w[r] * w[t])
        a_loads += int(sum(int(w[r]) for r in op_rows(op))) * M
    return cover, a_loads, c_loads


def element_schedule(N: int, k: int) -> Tuple[List[Op], int]:
    """Element-level TBS for memory S = k(k+1)/2; returns (ops, S)."""
    S = k * (k + 1) // 2
    s = max(1, math.isqrt(S + 1) - 1)
    return tbs_ops(N, k, s), S


def tiled_schedule(N: int, b: int, k: int) -> Tuple[List[Op], List[int], int]:
    """Tiled TBS (Section 5.1.4): returns (ops over tile rows, tile heights, S).

    S = b^2 k(k-1)/2; the fallback uses squares of g x g tiles with
    g = floor(sqrt(k(k-1)/2)), the largest that fits S.
    """
    n_t = -(-N // b)
    weights = [min(b, N - t * b) for t in range(n_t)]
    S = b * b * k * (k - 1) // 2
    g = max(1, math.isqrt(k * (k - 1) // 2))
    return tbs_ops(n_t, k, g), weights, S


def lower_bound(N: int, M: int, S: int) -> float:
    """SYRK I/O lower bound N^2 M / (sqrt(2) sqrt(S)) (Corollary, Section 4.1)."""
    return N * N * M / math.sqrt(2.0 * S)
