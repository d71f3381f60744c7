"""CPU oracle of the feed-back search for index arrays (Section 3.2).  TEST INFRASTRUCTURE ONLY:
it shares no code with the library and nothing in the product path imports it.

Section 3.2 describes the search only in words: take the absolute values of a trained layer matrix and
pick the row and column permutations that maximise the sum of the entries landing in the upper-left and
the lower-right sub-block, by a greedy optimisation started from randomly chosen permutations; the
entries of the two off-diagonal sub-blocks are deleted (half of the block); repeat on every remaining
block, so that every level has twice as many blocks as the one before (Section 3.2).  The reading implemented here, step by step:

  one bisection of a block (rows R, columns C of the current pivoted order, |R| = m, |C| = n):
    side 0 holds the first ceil(m/2) rows / ceil(n/2) columns, side 1 the rest (the starting
    permutation decides who starts where);
    repeat up to max_sweeps times, stop when a whole sweep changes nothing:
      rows:    with the columns fixed, gain_i = sum_{j on side 0} a_ij - sum_{j on side 1} a_ij;
               the ceil(m/2) rows of largest gain (ties: the row that comes first in the current
               order) go to side 0 -- the best balanced choice for these columns;
      columns: the same with the rows fixed;
    inside a side the current relative order is kept (a stable partition).
  levels bisections, every block of level l split again at level l + 1.

Every step can only raise the kept sum, so the sweeps end.  Parity unpinned by the paper (it prints
neither the algorithm nor a worked example); pinned by planted structures that must be recovered
exactly, by the monotone objective and by brute force over all balanced splits on tiny matrices.
"""
from __future__ import annotations

import numpy as np


def _half(n: int) -> int:
    return (n + 1) // 2


def kept_mass(absW, row_perm, col_perm, blocks) -> float:
    A = np.asarray(absW, dtype=np.float64)[np.ix_(row_perm, col_perm)]
    return float(sum(A[r0:r0 + h, c0:c0 + w].sum() for r0, c0, h, w in blocks))


def bisect(A, rows, cols, max_sweeps):
    """One bisection.  rows / cols: original indices in current pivoted order.  Returns the new orders
    and the kept sum after every half-sweep (for the monotonicity pin)."""
    rows, cols = list(rows), list(cols)
    m, n = len(rows), len(cols)
    hm, hn = _half(m), _half(n)
    history = []
    for _ in range(max_sweeps):
        changed = False
        sub = A[np.ix_(rows, cols)]
        gain = sub[:, :hn].sum(axis=1) - sub[:, hn:].sum(axis=1)
        order = sorted(range(m), key=lambda i: (-gain[i], i))
        top = set(order[:hm])
        new_rows = [rows[i] for i in range(m) if i in top] + [rows[i] for i in range(m) if i not in top]
        changed |= new_rows != rows
        rows = new_rows
        sub = A[np.ix_(rows, cols)]
        history.append(float(sub[:hm, :hn].sum() + sub[hm:, hn:].sum()))
        gain = sub[:hm, :].sum(axis=0) - sub[hm:, :].sum(axis=0)
        order = sorted(range(n), key=lambda j: (-gain[j], j))
        top = set(order[:hn])
        new_cols = [cols[j] for j in range(n) if j in top] + [cols[j] for j in range(n) if j not in top]
        changed |= new_cols != cols
        cols = new_cols
        sub = A[np.ix_(rows, cols)]
        history.append(float(sub[:hm, :hn].sum() + sub[hm:, hn:].sum()))
        if not changed:
            break
    return rows, cols, history


def pivot_find(absW, levels, max_sweeps=32, row_init=None, col_init=None):
    """(row_perm, col_perm, blocks [2^levels][4], kept sum).  Index arrays map pivoted -> original."""
    A = np.asarray(absW, dtype=np.float64)
    M, N = A.shape
    rows = list(range(M)) if row_init is None else [int(v) for v in row_init]
    cols = list(range(N)) if col_init is None else [int(v) for v in col_init]
    blocks = [(0, 0, M, N)]
    for _ in range(levels):
        nxt = []
        for r0, c0, h, w in blocks:
            nr, nc, _ = bisect(A, rows[r0:r0 + h], cols[c0:c0 + w], max_sweeps)
            rows[r0:r0 + h] = nr
            cols[c0:c0 + w] = nc
            hm, hn = _half(h), _half(w)
            nxt += [(r0, c0, hm, hn), (r0 + hm, c0 + hn, h - hm, w - hn)]
        blocks = nxt
    rp, cp = np.array(rows, dtype=np.int32), np.array(cols, dtype=np.int32)
    bl = np.array(blocks, dtype=np.int32).reshape(-1, 4)
    return rp, cp, bl, kept_mass(A, rp, cp, bl)
