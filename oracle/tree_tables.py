"""Integer products of a candidate tree, written out from their definitions.

TEST INFRASTRUCTURE ONLY: this is part of the CPU oracle.  Nothing in the product
path may import it; only tests, the smoke check and the benchmark's CPU-baseline
leg do.  It shares no code with the CUDA library.

Every function takes one tree as ``parent`` (parent[i] in {-1} U [0, i); -1 is the
pre-tree state R, Sec. "The recurrence and path locality": a node consumes the state
of its root-to-parent path, and the previous packed row need not be its parent) and
answers by walking parent pointers, node by node, with no shortcuts.  All answers are
unique, so the CUDA library's tables must match them bit for bit.

Pins (tests/test_oracle_tree.py): hand-written tables for the 7-node tree of the
smallest configuration, including its accepted path 0 -> 2 -> 6; chains and stars
whose tables are known in closed form; randomised brute force against an
independent child-to-root formulation.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

# status words for an accepted path (Sec. "One device-selected path drives native
# continuation": padded path entries must not advance state; an invalid path leaves
# the sequence untouched).  First failing check wins, in the order below.
PATH_OK = 0
PATH_BAD_LEN = 1    # len < 0 or len > lmax
PATH_BAD_NODE = 2   # an entry t < len is outside [0, N)
PATH_BAD_ROOT = 3   # first entry is not a child of R
PATH_BAD_LINK = 4   # entry t is not a child of entry t-1


def validate_parent(parent: Sequence[int]) -> bool:
    return all(-1 <= p < i for i, p in enumerate(parent))


def ancestry(parent: Sequence[int], i: int) -> List[int]:
    """Root-first list of the nodes on the path from R to node i (inclusive)."""
    out = []
    while i >= 0:
        out.append(i)
        i = parent[i]
    return out[::-1]


def depth(parent: Sequence[int]) -> List[int]:
    """depth[i] = number of updates from the pre-tree state = 1 + depth[parent]; depth[R] = 0."""
    return [len(ancestry(parent, i)) for i in range(len(parent))]


def children(parent: Sequence[int]) -> Tuple[List[int], List[List[int]]]:
    """(children of R, children of each node), each in ascending logical index."""
    n = len(parent)
    root = [i for i in range(n) if parent[i] == -1]
    ch = [[j for j in range(n) if parent[j] == i] for i in range(n)]
    return root, ch


def leaves(parent: Sequence[int]) -> List[int]:
    n = len(parent)
    return [i for i in range(n) if not any(parent[j] == i for j in range(n))]


def paths(parent: Sequence[int]) -> Tuple[List[int], List[int]]:
    """CSR (path_off, path_nodes): path p is the root-first ancestry of leaf p
    (leaves in ascending logical index)."""
    off = [0]
    nodes: List[int] = []
    for lf in leaves(parent):
        nodes += ancestry(parent, lf)
        off.append(len(nodes))
    return off, nodes


def anc_win(parent: Sequence[int]) -> List[List[int]]:
    """Four-wide causal window of every node for the ancestry-gathered convolution
    (Sec. "Precompute branch histories while preserving arithmetic"): entry 3 is the
    node, 2 its parent, 1 its grandparent, 0 its great-grandparent.  Once the walk
    passes R the entries are -1, -2, -3: the most recent, second and third most recent
    rows of the committed convolution history."""
    out = []
    for i in range(len(parent)):
        win = [0, 0, 0, 0]
        cur = i
        below = 0  # how many history rows consumed so far
        for j in (3, 2, 1, 0):
            if cur >= 0:
                win[j] = cur
                cur = parent[cur]
            else:
                below += 1
                win[j] = -below
        out.append(win)
    return out


def slot_inv(slot: Sequence[int], n_slots: int) -> Optional[List[int]]:
    """Logical node held by each physical row, -1 for a padding row; None if the
    logical->physical map is not injective into [0, n_slots)."""
    inv = [-1] * n_slots
    for i, s in enumerate(slot):
        if not (0 <= s < n_slots) or inv[s] != -1:
            return None
        inv[s] = i
    return inv


def chains(parent: Sequence[int]) -> Dict[str, List[int]]:
    """Canonical chain decomposition (Sec. "Path-parallel verification and state
    lifetime": dependent path groups; a first path exports the cut states downstream
    paths start from).  The paper stops at two levels and takes the MTP spine as the
    principal path; the reading here: the principal child of a node is its
    lowest-index child, a chain starts at every child of R and at every non-principal
    child and follows principal children to a leaf, a chain's level is 0 when its head
    is a child of R and otherwise one more than the level of the chain holding the
    head's parent, and a cut node is the parent (other than R) of a chain head.

    Returns chain_head, chain_off (CSR), chain_nodes, chain_level, chain_of (per node)
    and cut_nodes (ascending, unique).  Chains are ordered by head index."""
    n = len(parent)
    _, ch = children(parent)
    heads = []
    for i in range(n):
        p = parent[i]
        if p == -1 or ch[p][0] != i:
            heads.append(i)
    chain_off = [0]
    chain_nodes: List[int] = []
    chain_of = [-1] * n
    for c, h in enumerate(heads):
        cur = h
        while True:
            chain_nodes.append(cur)
            chain_of[cur] = c
            if not ch[cur]:
                break
            cur = ch[cur][0]
        chain_off.append(len(chain_nodes))
    level = []
    for c, h in enumerate(heads):
        lv = 0
        cur = h
        while parent[cur] != -1:
            # climb to the head of the chain that holds the parent
            cur = heads[chain_of[parent[cur]]]
            lv += 1
        level.append(lv)
    cut = sorted({parent[h] for h in heads if parent[h] != -1})
    return dict(chain_head=heads, chain_off=chain_off, chain_nodes=chain_nodes,
                chain_level=level, chain_of=chain_of, cut_nodes=cut)


def path_from_node(parent: Sequence[int], node: int, lmax: int) -> Tuple[List[int], int, int]:
    """(accepted, length, status): the root-first list ending at ``node`` padded with -1
    to ``lmax``.  node = -1 gives the empty path (status OK).  A node outside [0, N)
    gives the empty path with PATH_BAD_NODE; a path longer than lmax gives the empty
    path with PATH_BAD_LEN."""
    if node == -1:
        return [-1] * lmax, 0, PATH_OK
    if not (0 <= node < len(parent)):
        return [-1] * lmax, 0, PATH_BAD_NODE
    a = ancestry(parent, node)
    if len(a) > lmax:
        return [-1] * lmax, 0, PATH_BAD_LEN
    return a + [-1] * (lmax - len(a)), len(a), PATH_OK


def validate_accepted(parent: Sequence[int], accepted: Sequence[int], length: int, lmax: int) -> int:
    """Status word of a supplied accepted path; entries at or beyond ``length`` are ignored."""
    n = len(parent)
    if length < 0 or length > lmax:
        return PATH_BAD_LEN
    for t in range(length):
        a = accepted[t]
        if not (0 <= a < n):
            return PATH_BAD_NODE
        if t == 0:
            if parent[a] != -1:
                return PATH_BAD_ROOT
        elif parent[a] != accepted[t - 1]:
            return PATH_BAD_LINK
    return PATH_OK


def all_tables(parent: Sequence[int], slot: Sequence[int], n_slots: int) -> Dict[str, List[int]]:
    """Every table the CUDA library exposes through lumo_tree_desc_get, flattened the same way."""
    root, ch = children(parent)
    child_off = [0]
    child_list: List[int] = []
    for c in [root] + ch:  # entry 0 = R, entry i+1 = node i
        child_list += c
        child_off.append(len(child_list))
    off, nodes = paths(parent)
    win = anc_win(parent)
    cd = chains(parent)
    return dict(
        depth=depth(parent),
        n_child=[len(c) for c in ch],
        child_off=child_off,
        child_list=child_list,
        is_leaf=[int(not c) for c in ch],
        leaves=leaves(parent),
        path_off=off,
        path_nodes=nodes,
        anc_win=[e for w in win for e in w],
        slot_inv=slot_inv(slot, n_slots),
        chain_head=cd["chain_head"],
        chain_off=cd["chain_off"],
        chain_nodes=cd["chain_nodes"],
        chain_level=cd["chain_level"],
        cut_nodes=cd["cut_nodes"],
    )
