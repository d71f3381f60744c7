"""Feed-back search for index arrays (Section 3.2): pins of the oracle, then the library's host routine
against the oracle (integer work: bit for bit on matrices whose sums are exact)."""
import itertools

import numpy as np
import pytest

from oracle import pp_pivot_oracle as pv


def _planted(seed, M, N, levels, noise=0.0, integer=True):
    """|W| with a planted PBP structure: 2^levels diagonal blocks of large entries hidden by random permutations."""
    rng = np.random.default_rng(seed)
    nb = 2 ** levels
    A = rng.integers(0, 2, size=(M, N)).astype(np.float64) * noise if noise else np.zeros((M, N))
    def pieces(n):                               # the ceil/floor halves the search itself makes
        sizes = [n]
        for _ in range(levels):
            sizes = [v for s_ in sizes for v in ((s_ + 1) // 2, s_ // 2)]
        return np.split(np.arange(n), np.cumsum(sizes)[:-1])
    rb, cb = pieces(M), pieces(N)
    for r, c in zip(rb, cb):
        A[np.ix_(r, c)] = rng.integers(8, 16, size=(len(r), len(c))) if integer else rng.uniform(8, 16, (len(r), len(c)))
    pr, pc = rng.permutation(M), rng.permutation(N)
    planted = sum(A[np.ix_(r, c)].sum() for r, c in zip(rb, cb))
    return A[np.ix_(pr, pc)], float(planted)


@pytest.mark.parametrize("M,N,levels", [(32, 32, 1), (64, 48, 2), (96, 128, 3), (30, 50, 2)])
def test_oracle_recovers_planted_structure(M, N, levels):
    A, planted = _planted(M + levels, M, N, levels)
    rng = np.random.default_rng(1)
    rp, cp, bl, kept = pv.pivot_find(A, levels, row_init=rng.permutation(M), col_init=rng.permutation(N))
    assert sorted(rp) == list(range(M)) and sorted(cp) == list(range(N))
    assert len(bl) == 2 ** levels
    assert kept == planted == A.sum()          # every planted entry kept, nothing else exists


def test_oracle_objective_never_decreases():
    rng = np.random.default_rng(3)
    A = rng.uniform(0, 1, (40, 56))
    rows, cols, hist = pv.bisect(A, rng.permutation(40), rng.permutation(56), 32)
    assert all(b >= a - 1e-12 for a, b in zip(hist, hist[1:]))
    assert hist[-1] > 0.5 * A.sum()          # and ends above what a random balanced split keeps (half, on average)


def test_oracle_row_step_is_the_best_balanced_choice():
    """With the columns fixed, no balanced choice of rows keeps more than the greedy one (brute force, 8 rows)."""
    rng = np.random.default_rng(5)
    A = rng.integers(0, 9, (8, 10)).astype(np.float64)
    cols = list(rng.permutation(10))
    rows, _, hist = pv.bisect(A, range(8), cols, 1)
    sub = A[:, cols]
    best = max(sub[list(s), :5].sum() + sub[[i for i in range(8) if i not in s], 5:].sum()
               for s in itertools.combinations(range(8), 4))
    assert hist[0] == best


def test_oracle_blocks_feed_the_block_layer_form():
    """The blocks tile the diagonal of the pivoted matrix; the kept sum is the sum over reconstruct_blocks' W."""
    from oracle import pp_oracle as po
    A, _ = _planted(9, 64, 64, 2, noise=1.0)
    rp, cp, bl, kept = pv.pivot_find(A, 2)
    vals = np.concatenate([A[np.ix_(rp[r0:r0 + h], cp[c0:c0 + w])].ravel() for r0, c0, h, w in bl])
    W = po.reconstruct_blocks(64, 64, rp, cp, bl, vals)
    assert W.sum() == kept
    assert np.array_equal(W != 0, (W == A) & (A != 0) & (W != 0))


# ---------------------------------------------------------------- the library's routine against the oracle
@pytest.mark.parametrize("M,N,levels,noise", [(64, 64, 2, 0.0), (96, 80, 3, 1.0), (50, 70, 2, 1.0), (128, 128, 4, 1.0)])
def test_library_matches_oracle_bit_for_bit(M, N, levels, noise):
    from paper_1712_01084_b200 import binding as pb
    A, _ = _planted(100 + M, M, N, levels, noise=noise)          # small integers: every sum is exact
    rng = np.random.default_rng(M)
    r0, c0 = rng.permutation(M).astype(np.int32), rng.permutation(N).astype(np.int32)
    rp, cp, bl, kept = pb.pp_pivot_find(A.astype(np.float32), levels, 32, r0, c0)
    rp_o, cp_o, bl_o, kept_o = pv.pivot_find(A, levels, 32, r0, c0)
    assert np.array_equal(rp, rp_o) and np.array_equal(cp, cp_o) and np.array_equal(bl, bl_o)
    assert kept == kept_o


def test_library_real_valued_input_is_valid_and_no_worse_than_start():
    from paper_1712_01084_b200 import binding as pb
    rng = np.random.default_rng(11)
    A = np.abs(rng.standard_normal((120, 90))).astype(np.float32)
    rp, cp, bl, kept = pb.pp_pivot_find(A, 2, 32, None, None)
    assert sorted(rp) == list(range(120)) and sorted(cp) == list(range(90))
    assert abs(kept - pv.kept_mass(A, rp, cp, bl)) <= 1e-9 * A.sum()
    ident = pv.kept_mass(A, np.arange(120), np.arange(90), bl)
    assert kept >= ident
    assert kept > 0.25 * A.sum() * 1.15          # two bisections keep a quarter of the entries, but the heavier quarter


def test_library_error_codes():
    from paper_1712_01084_b200 import binding as pb
    A = np.ones((8, 8), dtype=np.float32)
    with pytest.raises(pb.PPError) as e:
        pb.pp_pivot_find(A, 5, 4, None, None)            # more levels than the matrix can be halved
    assert e.value.status == 1
    with pytest.raises(pb.PPError) as e:
        pb.pp_pivot_find(A, 1, 4, np.zeros(8, dtype=np.int32), None)
    assert e.value.status == 2
