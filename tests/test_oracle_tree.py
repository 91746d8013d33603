"""Pins for the oracle's integer products (oracle/tree_tables.py).

Expected values here are written by hand from the definitions (the 7-node tree of the
smallest configuration, chains, stars) or come from an independent formulation
(child-to-root counting with no shared helper), never from the oracle itself.
"""
import random

import pytest

from oracle import tree_tables as T

TINY = [-1, -1, 0, 0, 1, 1, 2]


def test_tiny_tree_tables_by_hand():
    # R -> {0, 1}; 0 -> {2, 3}; 1 -> {4, 5}; 2 -> {6}
    assert T.depth(TINY) == [1, 1, 2, 2, 2, 2, 3]
    root, ch = T.children(TINY)
    assert root == [0, 1]
    assert ch == [[2, 3], [4, 5], [6], [], [], [], []]
    assert T.leaves(TINY) == [3, 4, 5, 6]
    off, nodes = T.paths(TINY)
    assert off == [0, 2, 4, 6, 9]
    assert nodes == [0, 3, 1, 4, 1, 5, 0, 2, 6]
    assert T.anc_win(TINY) == [
        [-3, -2, -1, 0], [-3, -2, -1, 1],
        [-2, -1, 0, 2], [-2, -1, 0, 3], [-2, -1, 1, 4], [-2, -1, 1, 5],
        [-1, 0, 2, 6]]


def test_tiny_accepted_path_is_0_2_6():
    # the smallest configuration fixes the accepted path 0 -> 2 -> 6
    assert T.path_from_node(TINY, 6, 3) == ([0, 2, 6], 3, T.PATH_OK)
    assert T.path_from_node(TINY, 6, 5) == ([0, 2, 6, -1, -1], 3, T.PATH_OK)
    assert T.path_from_node(TINY, -1, 3) == ([-1, -1, -1], 0, T.PATH_OK)
    assert T.path_from_node(TINY, 6, 2) == ([-1, -1], 0, T.PATH_BAD_LEN)
    assert T.path_from_node(TINY, 7, 3) == ([-1, -1, -1], 0, T.PATH_BAD_NODE)
    assert T.validate_accepted(TINY, [0, 2, 6], 3, 3) == T.PATH_OK


def test_tiny_chain_decomposition_by_hand():
    # principal child = lowest index: chains 0-2-6, 1-4, 3, 5; 3 hangs off chain 0, 5 off chain 1
    cd = T.chains(TINY)
    assert cd["chain_head"] == [0, 1, 3, 5]
    assert cd["chain_off"] == [0, 3, 5, 6, 7]
    assert cd["chain_nodes"] == [0, 2, 6, 1, 4, 3, 5]
    assert cd["chain_level"] == [0, 0, 1, 1]
    assert cd["cut_nodes"] == [0, 1]


def test_accepted_path_validation_codes():
    assert T.validate_accepted(TINY, [0, 2, 6], 0, 3) == T.PATH_OK          # empty prefix
    assert T.validate_accepted(TINY, [0, 2, 99], 2, 3) == T.PATH_OK         # beyond len ignored
    assert T.validate_accepted(TINY, [0, 2, 6], 4, 3) == T.PATH_BAD_LEN
    assert T.validate_accepted(TINY, [0, 2, 6], -1, 3) == T.PATH_BAD_LEN
    assert T.validate_accepted(TINY, [0, 7, 6], 3, 3) == T.PATH_BAD_NODE
    assert T.validate_accepted(TINY, [-1, 2, 6], 3, 3) == T.PATH_BAD_NODE
    assert T.validate_accepted(TINY, [2, 6, -1], 2, 3) == T.PATH_BAD_ROOT   # 2 is not a child of R
    assert T.validate_accepted(TINY, [0, 4, -1], 2, 3) == T.PATH_BAD_LINK   # sibling substitution
    assert T.validate_accepted(TINY, [0, 6, -1], 2, 3) == T.PATH_BAD_LINK   # skipped a node


def test_chain_closed_forms():
    n = 9
    p = [i - 1 for i in range(n)]
    assert T.depth(p) == list(range(1, n + 1))
    assert T.leaves(p) == [n - 1]
    assert T.paths(p) == ([0, n], list(range(n)))
    w = T.anc_win(p)
    assert w[0] == [-3, -2, -1, 0] and w[1] == [-2, -1, 0, 1] and w[2] == [-1, 0, 1, 2]
    assert all(w[i] == [i - 3, i - 2, i - 1, i] for i in range(3, n))
    cd = T.chains(p)
    assert cd["chain_head"] == [0] and cd["chain_level"] == [0] and cd["cut_nodes"] == []


def test_star_closed_forms():
    n = 12
    p = [-1] + [0] * (n - 1)
    assert T.depth(p) == [1] + [2] * (n - 1)
    assert T.leaves(p) == list(range(1, n))
    off, nodes = T.paths(p)
    assert off == list(range(0, 2 * n - 1, 2))
    assert nodes == [e for i in range(1, n) for e in (0, i)]
    assert all(T.anc_win(p)[i] == [-2, -1, 0, i] for i in range(1, n))
    cd = T.chains(p)
    assert cd["chain_head"] == [0] + list(range(2, n))     # child 1 continues chain 0
    assert cd["chain_level"] == [0] + [1] * (n - 2)
    assert cd["cut_nodes"] == [0]


def test_slot_inverse():
    assert T.slot_inv([2, 0, 3], 5) == [1, -1, 0, 2, -1]
    assert T.slot_inv([2, 2, 3], 5) is None      # not injective
    assert T.slot_inv([2, 5, 3], 5) is None      # out of range


def _random_parent(rng, n):
    return [rng.randint(-1, i - 1) for i in range(n)]


@pytest.mark.parametrize("seed", range(20))
def test_brute_force_independent_formulation(seed):
    """Child-to-root counting that shares nothing with the oracle's helpers."""
    rng = random.Random(seed)
    n = rng.randint(1, 40)
    p = _random_parent(rng, n)
    assert T.validate_parent(p)
    # depth by fixed-point relaxation instead of walking
    d = [0] * n
    for _ in range(n):
        for i in range(n):
            d[i] = 1 if p[i] == -1 else d[p[i]] + 1
    assert T.depth(p) == d
    # leaves: nodes never named as a parent
    lv = sorted(set(range(n)) - set(p))
    assert T.leaves(p) == lv
    off, nodes = T.paths(p)
    assert len(off) == len(lv) + 1 and off[-1] == sum(d[l] for l in lv)
    for j, l in enumerate(lv):
        seg = nodes[off[j]:off[j + 1]]
        assert seg[-1] == l and p[seg[0]] == -1
        assert all(p[seg[t]] == seg[t - 1] for t in range(1, len(seg)))
    # windows: entry 3-j is the j-th ancestor, then history -1, -2, -3
    win = T.anc_win(p)
    for i in range(n):
        cur, hist = i, 0
        for j in range(4):
            if cur >= 0:
                assert win[i][3 - j] == cur
                cur = p[cur]
            else:
                hist += 1
                assert win[i][3 - j] == -hist
    # chains partition the nodes, one per leaf, each following lowest-index children
    cd = T.chains(p)
    assert sorted(cd["chain_nodes"]) == list(range(n))
    assert len(cd["chain_head"]) == len(lv)
    for c in range(len(cd["chain_head"])):
        seg = cd["chain_nodes"][cd["chain_off"][c]:cd["chain_off"][c + 1]]
        assert seg[0] == cd["chain_head"][c] and seg[-1] in lv
        for a, b in zip(seg, seg[1:]):
            assert p[b] == a and min(j for j in range(n) if p[j] == a) == b
        h = seg[0]
        if p[h] == -1:
            assert cd["chain_level"][c] == 0
        else:
            assert cd["chain_level"][c] == cd["chain_level"][cd["chain_of"][p[h]]] + 1
            assert p[h] in cd["cut_nodes"]
    # every accepted path built from a node validates; corrupting a link does not
    for i in range(n):
        acc, ln, st = T.path_from_node(p, i, n)
        assert st == T.PATH_OK and ln == d[i] and acc[ln - 1] == i
        assert T.validate_accepted(p, acc, ln, n) == T.PATH_OK
