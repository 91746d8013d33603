"""Pins of the draft-selection oracle: hand-worked rows, closed forms, a counting restatement on
exhaustive small inputs, invariants."""
import itertools

import numpy as np
import pytest

from oracle import select_oracle as S


def test_hand_worked_rows():
    # unique maximum: candidate 0 repeats the spine token
    sp, c = S.select([[0.1, 2.0, -1.0, 1.5, 0.3]])
    assert sp.tolist() == [1] and c.tolist() == [[1, 3, 4]]
    # tie for the maximum: argmax takes the lowest index, the candidate list the highest first
    sp, c = S.select([[5.0, 1.0, 5.0, 5.0, 0.0]])
    assert sp.tolist() == [0] and c.tolist() == [[3, 2, 0]]
    # tie below the maximum
    sp, c = S.select([[1.0, 7.0, 3.0, 3.0, 3.0, 2.0]])
    assert sp.tolist() == [1] and c.tolist() == [[1, 4, 3]]
    # -inf entries (masked tokens) are ordinary values; signed zeros are equal
    sp, c = S.select([[-np.inf, -np.inf, -np.inf, -np.inf]])
    assert sp.tolist() == [0] and c.tolist() == [[3, 2, 1]]
    sp, c = S.select([[-0.0, 0.0, -1.0, 0.0]])
    assert sp.tolist() == [0] and c.tolist() == [[3, 1, 0]]


@pytest.mark.parametrize("V", [3, 4, 17, 1000])
def test_all_equal_row_closed_form(V):
    sp, c = S.select(np.full((2, V), 0.25))
    assert sp.tolist() == [0, 0]
    assert c.tolist() == [[V - 1, V - 2, V - 3]] * 2


def test_strictly_increasing_and_decreasing_rows():
    V = 50
    sp, c = S.select([np.arange(V), -np.arange(V)])
    assert sp.tolist() == [V - 1, 0]
    assert c.tolist() == [[V - 1, V - 2, V - 3], [0, 1, 2]]


def test_counting_restatement_exhaustive_small():
    # every row of length 3..5 over three distinct values: all tie patterns
    for V in (3, 4, 5):
        rows = list(itertools.product([0.0, 1.0, 2.0], repeat=V))
        a = S.select(rows)
        b = S.select_by_rank(rows)
        assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_counting_restatement_random_with_ties():
    rs = np.random.default_rng(5)
    x = rs.integers(0, 6, size=(40, 23)).astype(np.float64)     # few distinct values: many ties
    a, b = S.select(x), S.select_by_rank(x)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_invariants():
    rs = np.random.default_rng(6)
    x = np.round(rs.standard_normal((64, 301)) * 2) / 2                 # quantised: ties occur
    sp, c = S.select(x)
    rows = np.arange(64)
    v = x[rows[:, None], c]
    assert np.all(v[:, 0] >= v[:, 1]) and np.all(v[:, 1] >= v[:, 2])
    assert np.all(x[rows, sp] == v[:, 0]) and np.all(x[rows, sp] == x.max(1))
    assert np.all(sp <= c[:, 0])
    unique_max = (x == x.max(1, keepdims=True)).sum(1) == 1
    assert np.array_equal(sp == c[:, 0], unique_max)
    assert all(len(set(r)) == 3 for r in c.tolist())
    # nothing outside the list beats its last entry
    for r in range(64):
        rest = np.setdiff1d(np.arange(301), c[r])
        assert np.all((x[r, rest] < v[r, 2]) | ((x[r, rest] == v[r, 2]) & (rest < c[r, 2])))


def test_matches_library_routines_without_ties():
    rs = np.random.default_rng(7)
    x = rs.standard_normal((16, 5000))                                   # distinct with probability 1
    sp, c = S.select(x)
    assert np.array_equal(sp, np.argmax(x, axis=1))
    assert np.array_equal(c, np.argsort(-x, axis=1, kind="stable")[:, :3])


def test_rejects_bad_input():
    with pytest.raises(ValueError):
        S.select([[1.0, 2.0]])
    with pytest.raises(ValueError):
        S.select([[1.0, np.nan, 0.0]])
