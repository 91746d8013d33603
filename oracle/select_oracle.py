"""Oracle of the fused full-vocabulary draft selection.

TEST INFRASTRUCTURE ONLY (see oracle/gdn_oracle.cpp): plain NumPy and plain Python, shares nothing
with the CUDA library.

What it computes (Sec. "Fuse draft selection without changing proposals"): for each row of logits
the spine token and three ordered sibling candidates.  The paper fixes that the spine token is the
reference argmax, the lowest index among equal maxima, that the candidate list comes from a top-k
whose order of tied entries differs from argmax's, and that duplicates are kept.  It does not say
how top-k orders ties; the reading taken here is the mirror convention:

    spine[r]      = min { i : x[r, i] = max_j x[r, j] }
    cand[r, 0..2] = the first three entries of the row sorted by (value descending, index descending)

so on a tie for the maximum spine and cand[0] differ, and with a unique maximum cand[0] repeats the
spine token.  Values compare as IEEE numbers (-0.0 == +0.0, -inf is an ordinary value); NaN is not
allowed.  bf16 inputs are widened exactly before comparing.

`select` is the definition written with sorting; `select_by_rank` restates it by counting, for
tiny inputs: entry i has candidate rank #{ j : x_j > x_i or (x_j == x_i and j > i) }.
Pins (tests/test_oracle_select.py): hand-worked rows with ties; all-equal rows; agreement of the
two formulations on exhaustive small inputs; invariants (candidate values non-increasing, spine
value equals cand[0] value, spine <= cand[0] with equality iff the maximum is unique).
"""
import numpy as np


def select(x):
    """x [R, V] float array (V >= 3) -> spine int32 [R], cand int32 [R, 3]."""
    x = np.asarray(x, dtype=np.float64)
    if x.ndim != 2 or x.shape[1] < 3:
        raise ValueError("x must be [R, V] with V >= 3")
    if np.isnan(x).any():
        raise ValueError("NaN logits are not allowed")
    R, V = x.shape
    spine = np.empty(R, np.int32)
    cand = np.empty((R, 3), np.int32)
    idx = np.arange(V)
    for r in range(R):
        row = x[r] + 0.0                       # -0.0 -> +0.0 so that sorting sees them as equal
        m = row.max()
        spine[r] = idx[row == m][0]
        # lexsort: last key is the primary one; ascending sort of (-value, -index)
        order = np.lexsort((-idx, -row))
        cand[r] = order[:3]
    return spine, cand


def select_by_rank(x):
    """Counting restatement, O(V^2): for tiny inputs."""
    x = [[float(v) for v in row] for row in x]
    spine, cand = [], []
    for row in x:
        V = len(row)
        m = max(row)
        spine.append(min(i for i in range(V) if row[i] == m))
        c = [None, None, None]
        for i in range(V):
            rank = sum(1 for j in range(V) if row[j] > row[i] or (row[j] == row[i] and j > i))
            if rank < 3:
                c[rank] = i
        cand.append(c)
    return np.asarray(spine, np.int32), np.asarray(cand, np.int32)
