"""Seeded synthetic inputs for the GDN tree verify + commit path.

This module only draws numbers and tree shapes.  It contains none of the
method's arithmetic (no convolution, no recurrence, no path tables): both the
CPU oracle's tests and the CUDA parity tests call it so that the two sides read
the very same rounded arrays.

Random numbers come from a counter-based splitmix64 generator: the value at
index ``i`` of a stream depends only on the stream key and ``i``, so any slice
of any tensor can be regenerated independently.  Uniforms use the top 53 bits;
normals use Box-Muller in float64.  Every array is then rounded to the dtype
the kernels read (bf16 or fp32) and returned as float32, which holds both
exactly.

Workload shapes follow the evaluated hybrid model of the paper (Sec. "Evaluation
Setup": 48 GDN layers, candidate trees of a principal MTP spine plus branches,
rows padded to a fixed count) and the five benchmark configurations.  The
paper's own workload is a coding-agent run on a public benchmark; these
synthetic tensors stand in for it and take only its shapes.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Sequence

import numpy as np

_MASK = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
BASE_SEED = 0x4C554D4F  # "LUMO"

# tensor ids used to derive stream keys
_T = {name: i for i, name in enumerate(
    ["tree", "slot", "state", "x", "hist", "conv_w", "conv_b", "q", "k", "v",
     "alpha", "beta", "accept", "rows", "misc"], start=1)}


# ---------------------------------------------------------------------------
# counter-based generator
# ---------------------------------------------------------------------------
def _mix_int(z: int) -> int:
    z = (z + _GOLDEN) & _MASK
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK
    return z ^ (z >> 31)


def stream_key(*parts: int) -> int:
    """Hash a tuple of integers (seed, tensor id, layer, ...) into a 64-bit key."""
    k = 0x243F6A8885A308D3
    for p in parts:
        k = _mix_int(k ^ (int(p) & _MASK))
    return k


def _mix_vec(z: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        z = z + np.uint64(_GOLDEN)
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        return z ^ (z >> np.uint64(31))


def raw_u64(key: int, n: int, start: int = 0) -> np.ndarray:
    with np.errstate(over="ignore"):
        ctr = (np.arange(start, start + n, dtype=np.uint64) + np.uint64(1)) * np.uint64(_GOLDEN)
        return _mix_vec(np.uint64(key) + ctr)


def uniforms(key: int, n: int, start: int = 0) -> np.ndarray:
    """float64 uniforms in [0, 1)."""
    return (raw_u64(key, n, start) >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))


def normals(key: int, n: int) -> np.ndarray:
    """float64 standard normals (Box-Muller; element i uses counters 2i, 2i+1)."""
    u = uniforms(key, 2 * n)
    u1 = 1.0 - u[0::2]  # (0, 1]
    u2 = u[1::2]
    return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * math.pi * u2)


class IntStream:
    """Sequential integer draws for tree construction (pure Python, exact)."""

    def __init__(self, key: int):
        self.key = key
        self.ctr = 0

    def next_u64(self) -> int:
        self.ctr += 1
        return _mix_int((self.key + self.ctr * _GOLDEN) & _MASK)

    def randint(self, lo: int, hi: int) -> int:
        """uniform integer in [lo, hi] (modulo bias < 2^-60 at these ranges)."""
        return lo + self.next_u64() % (hi - lo + 1)

    def uniform(self) -> float:
        return (self.next_u64() >> 11) * (1.0 / (1 << 53))


# ---------------------------------------------------------------------------
# rounding to the kernels' input dtypes (storage only, not method arithmetic)
# ---------------------------------------------------------------------------
def round_to(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float64 to ``dtype`` ("f32" or "bf16"), returned as float32."""
    x32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    if dtype == "f32":
        return x32
    if dtype != "bf16":
        raise ValueError(dtype)
    bits = x32.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return bits.astype(np.uint32).view(np.float32).reshape(x32.shape)


# ---------------------------------------------------------------------------
# tree shapes.  parent[i] in {-1} U [0, i); -1 is the pre-tree state R.
# ---------------------------------------------------------------------------
def tree_tiny() -> List[int]:
    """The 7-node tree of the smallest configuration."""
    return [-1, -1, 0, 0, 1, 1, 2]


def tree_chain(n: int) -> List[int]:
    return [i - 1 for i in range(n)]


def tree_chains(n_chains: int, length: int) -> List[int]:
    """``n_chains`` disjoint chains of ``length`` nodes hanging off R."""
    parent = []
    for c in range(n_chains):
        for j in range(length):
            parent.append(-1 if j == 0 else len(parent) - 1)
    return parent


def tree_star(n: int) -> List[int]:
    """Node 0 under R, nodes 1..n-1 children of node 0."""
    return [-1] + [0] * (n - 1)


def tree_mtp_spine(rs: IntStream, n: int = 16, spine: int = 4) -> List[int]:
    """MTP spine of ``spine`` nodes plus 2-3 single-node siblings per level;
    left-over nodes extend the earliest sibling branches by one node each."""
    parent = [i - 1 for i in range(spine)]
    sib_heads: List[int] = []
    for lvl in range(spine):
        for _ in range(rs.randint(2, 3)):
            if len(parent) >= n:
                break
            parent.append(lvl - 1)  # sibling of spine node lvl: child of spine lvl-1 (or R)
            sib_heads.append(len(parent) - 1)
    tails = list(sib_heads)
    j = 0
    while len(parent) < n:
        parent.append(tails[j % len(tails)])
        tails[j % len(tails)] = len(parent) - 1
        j += 1
    return parent


def tree_random(rs: IntStream, n: int, max_depth: int, max_children: int = 4) -> List[int]:
    """Frontier expansion: pop a uniformly random frontier node; if it is above
    ``max_depth`` give it U{1..max_children} children; stop at ``n`` nodes.
    Restarts (continuing the same stream) if the frontier empties first; gives up with ValueError
    when the shape cannot hold ``n`` nodes or after 1000 restarts."""
    if sum(max_children ** k for k in range(1, max_depth + 1)) < n:
        raise ValueError(f"a tree of depth <= {max_depth} with fan-out <= {max_children} cannot hold {n} nodes")
    for _ in range(1000):
        parent: List[int] = []
        depth: List[int] = []
        frontier = [-1]
        while len(parent) < n and frontier:
            p = frontier.pop(rs.randint(0, len(frontier) - 1))
            d = 0 if p < 0 else depth[p]
            if d >= max_depth:
                continue
            c = rs.randint(1, max_children)
            for _ in range(c):
                if len(parent) >= n:
                    break
                parent.append(p)
                depth.append(d + 1)
                frontier.append(len(parent) - 1)
        if len(parent) == n:
            return parent
    raise ValueError("tree_random: the frontier kept emptying before the tree was full")


def tree_paper_geometry() -> List[int]:
    """28 active nodes in the shape the paper evaluates (Sec. "Evaluation Setup"):
    node 0 is the root token; a five-depth MTP head of 15 candidates (three per
    depth, the first of each depth on the spine); a six-node principal tail; rescue
    branches of four and two nodes.  Where the rescue branches attach is not stated
    in the paper; here they hang off the depth-1 and depth-2 runner-up candidates."""
    parent = [-1]
    spine_prev = 0
    runner = []
    for _ in range(5):
        first = len(parent)
        parent += [spine_prev, spine_prev, spine_prev]
        runner.append(first + 1)
        spine_prev = first
    for _ in range(6):  # principal tail
        parent.append(spine_prev)
        spine_prev = len(parent) - 1
    for head, ln in ((runner[0], 4), (runner[1], 2)):
        prev = head
        for _ in range(ln):
            parent.append(prev)
            prev = len(parent) - 1
    assert len(parent) == 28
    return parent


def _children(parent: Sequence[int]) -> Dict[int, List[int]]:
    ch: Dict[int, List[int]] = {-1: []}
    for i, p in enumerate(parent):
        ch.setdefault(i, [])
        ch[p].append(i)
    return ch


def draw_accepted(rs: IntStream, parent: Sequence[int], p_stop: float = 0.35,
                  lmax: Optional[int] = None) -> List[int]:
    """Accepted path: length L with P(L=l) = p (1-p)^(l-1), l >= 1; walk from R taking a
    uniformly random child each step until L nodes or a leaf (or ``lmax``)."""
    ch = _children(parent)
    L = 1
    while rs.uniform() >= p_stop:
        L += 1
    if lmax is not None:
        L = min(L, lmax)
    path: List[int] = []
    cur = -1
    while len(path) < L and ch[cur]:
        kids = ch[cur]
        cur = kids[rs.randint(0, len(kids) - 1)]
        path.append(cur)
    return path


def tree_depths(parent: Sequence[int]) -> List[int]:
    d: List[int] = []
    for p in parent:
        d.append(1 if p < 0 else d[p] + 1)
    return d


# ---------------------------------------------------------------------------
# cases
# ---------------------------------------------------------------------------
@dataclasses.dataclass
class LayerTensors:
    """One GDN layer's tensors.  All float arrays are float32 holding values exactly
    representable in ``in_dtype``; per-node arrays are indexed by PHYSICAL row."""
    x: np.ndarray        # [B, Ns, C]   pre-conv projections, channels [q | k | v]
    conv_w: np.ndarray   # [C, 4]       tap 3 multiplies the current row
    conv_b: Optional[np.ndarray]  # [C] or None
    hist: np.ndarray     # [rows, 3, C] committed raw inputs, oldest first
    q: np.ndarray        # [B, Ns, Hk, d]  scan-only operands (L2-normalised)
    k: np.ndarray        # [B, Ns, Hk, d]
    v: np.ndarray        # [B, Ns, Hv, d]
    alpha: np.ndarray    # [B, Ns, Hv]
    beta: np.ndarray     # [B, Ns, Hv]
    state: np.ndarray    # [rows, Hv, d, d] fp32 pre-tree states


@dataclasses.dataclass
class Case:
    name: str
    seed: int
    B: int
    N: int
    Ns: int
    Hk: int
    Hv: int
    d: int
    in_dtype: str            # "f32" | "bf16"
    rows: int                # state / history pool rows
    parent: np.ndarray       # int32 [B, N]
    slot: np.ndarray         # int32 [B, N] logical -> physical row
    state_row: np.ndarray    # int32 [B]
    accepted: np.ndarray     # int32 [B, Lmax], -1 padded
    accepted_len: np.ndarray  # int32 [B]
    lmax: int
    layers: List[LayerTensors]

    @property
    def C(self) -> int:
        return 2 * self.Hk * self.d + self.Hv * self.d


def _l2_normalise(a: np.ndarray) -> np.ndarray:
    # input recipe: q, k are unit vectors per head before rounding
    return a / np.sqrt(np.sum(a * a, axis=-1, keepdims=True))


def make_layer(seed: int, layer: int, B: int, Ns: int, Hk: int, Hv: int, d: int, rows: int,
               in_dtype: str, alpha_lo: float = 0.9, beta_uniform: bool = False,
               with_bias: bool = False) -> LayerTensors:
    C = 2 * Hk * d + Hv * d
    key = lambda t: stream_key(seed, _T[t], layer)
    r = lambda a: round_to(a, in_dtype)
    x = r(normals(key("x"), B * Ns * C).reshape(B, Ns, C))
    hist = r(normals(key("hist"), rows * 3 * C).reshape(rows, 3, C))
    conv_w = r(0.5 * normals(key("conv_w"), C * 4).reshape(C, 4))
    conv_b = r(0.1 * normals(key("conv_b"), C)) if with_bias else None
    q = r(_l2_normalise(normals(key("q"), B * Ns * Hk * d).reshape(B, Ns, Hk, d)))
    k = r(_l2_normalise(normals(key("k"), B * Ns * Hk * d).reshape(B, Ns, Hk, d)))
    v = r(normals(key("v"), B * Ns * Hv * d).reshape(B, Ns, Hv, d))
    alpha = r(alpha_lo + (1.0 - alpha_lo) * uniforms(key("alpha"), B * Ns * Hv).reshape(B, Ns, Hv))
    if beta_uniform:
        beta = r(uniforms(key("beta"), B * Ns * Hv).reshape(B, Ns, Hv))
    else:
        beta = r(1.0 / (1.0 + np.exp(-normals(key("beta"), B * Ns * Hv).reshape(B, Ns, Hv))))
    state = (0.02 * normals(key("state"), rows * Hv * d * d)).astype(np.float32).reshape(rows, Hv, d, d)
    return LayerTensors(x, conv_w, conv_b, hist, q, k, v, alpha, beta, state)


def make_case(name: str, parents: Sequence[Sequence[int]], *, seed: int, Hk: int, Hv: int, d: int,
              in_dtype: str, n_layers: int = 1, Ns: Optional[int] = None, permute_slots: bool = False,
              extra_rows: int = 1, alpha_lo: float = 0.9, beta_uniform: bool = False,
              with_bias: bool = False, accepted: Optional[Sequence[Sequence[int]]] = None,
              lmax: Optional[int] = None, shuffle_rows: bool = True) -> Case:
    """Assemble a case from per-sequence parent arrays (all of one length N)."""
    B = len(parents)
    N = len(parents[0])
    assert all(len(p) == N for p in parents)
    Ns = N if Ns is None else Ns
    rows = B + extra_rows
    parent = np.asarray(parents, dtype=np.int32).reshape(B, N)
    slot = np.tile(np.arange(N, dtype=np.int32), (B, 1))
    if permute_slots:
        for b in range(B):
            rs = IntStream(stream_key(seed, _T["slot"], b))
            perm = list(range(Ns))
            for i in range(Ns - 1, 0, -1):  # Fisher-Yates
                j = rs.randint(0, i)
                perm[i], perm[j] = perm[j], perm[i]
            slot[b] = np.asarray(perm[:N], dtype=np.int32)
    # state rows: a seeded permutation of the pool so that row != b in general
    rows_perm = list(range(rows))
    if shuffle_rows:
        rs = IntStream(stream_key(seed, _T["rows"]))
        for i in range(rows - 1, 0, -1):
            j = rs.randint(0, i)
            rows_perm[i], rows_perm[j] = rows_perm[j], rows_perm[i]
    state_row = np.asarray(rows_perm[:B], dtype=np.int32)
    if accepted is None:
        accepted = []
        for b in range(B):
            rs = IntStream(stream_key(seed, _T["accept"], b))
            accepted.append(draw_accepted(rs, parents[b]))
    max_depth = max(max(tree_depths(p)) for p in parents)
    lmax = max_depth if lmax is None else lmax
    acc = np.full((B, lmax), -1, dtype=np.int32)
    acc_len = np.zeros(B, dtype=np.int32)
    for b, a in enumerate(accepted):
        acc[b, :len(a)] = a
        acc_len[b] = len(a)
    layers = [make_layer(seed, l, B, Ns, Hk, Hv, d, rows, in_dtype, alpha_lo, beta_uniform, with_bias)
              for l in range(n_layers)]
    return Case(name, seed, B, N, Ns, Hk, Hv, d, in_dtype, rows, parent, slot, state_row, acc,
                acc_len, lmax, layers)


# The five benchmark configurations (plus the paper's evaluated geometry).
def config0(seed: int = BASE_SEED + 0) -> Case:
    """Tiny: batch 1, 2 heads, d=64, fp32; 7-node tree; accepted path 0 -> 2 -> 6."""
    return make_case("cfg0_tiny", [tree_tiny()], seed=seed, Hk=2, Hv=2, d=64, in_dtype="f32",
                     accepted=[[0, 2, 6]], extra_rows=0)


def config1(seed: int = BASE_SEED + 1) -> Case:
    """Single layer, batch 1, 16/32 heads, d=128, bf16; 16-node MTP spine + branches."""
    p = tree_mtp_spine(IntStream(stream_key(seed, _T["tree"], 0)))
    return make_case("cfg1_b1_n16", [p], seed=seed, Hk=16, Hv=32, d=128, in_dtype="bf16")


def config2(seed: int = BASE_SEED + 2, B: int = 8, n_layers: int = 1) -> Case:
    """Serving batch 8: per-sequence random 64-node trees, depth <= 8, fan-out U{1..4}."""
    ps = [tree_random(IntStream(stream_key(seed, _T["tree"], b)), 64, 8) for b in range(B)]
    return make_case("cfg2_b8_n64", ps, seed=seed, Hk=16, Hv=32, d=128, in_dtype="bf16",
                     n_layers=n_layers)


def config3(seed: int = BASE_SEED + 3, B: int = 4, n_layers: int = 48) -> Case:
    """Hybrid-stack sweep: 48 layers, batch 4, 32-node trees of depth <= 6."""
    ps = [tree_random(IntStream(stream_key(seed, _T["tree"], b)), 32, 6) for b in range(B)]
    return make_case("cfg3_48L_b4_n32", ps, seed=seed, Hk=16, Hv=32, d=128, in_dtype="bf16",
                     n_layers=n_layers)


def config4(shape: str, seed: int = BASE_SEED + 4, B: int = 32, N: int = 256) -> Case:
    """Topology stress on 256-node trees: 16 chains x 16, a 255-child star, or a random
    tree of depth <= 12; alpha ~ U(0.5, 1), beta ~ U(0, 1)."""
    if shape == "chains":
        ps = [tree_chains(N // 16, 16) for _ in range(B)]
    elif shape == "star":
        ps = [tree_star(N) for _ in range(B)]
    elif shape == "random":
        ps = [tree_random(IntStream(stream_key(seed, _T["tree"], b)), N, 12) for b in range(B)]
    else:
        raise ValueError(shape)
    return make_case(f"cfg4_{shape}", ps, seed=seed, Hk=16, Hv=32, d=128, in_dtype="bf16",
                     alpha_lo=0.5, beta_uniform=True)


def config_paper(seed: int = BASE_SEED + 5, B: int = 1, n_layers: int = 1) -> Case:
    """The paper's evaluated geometry: 28 active rows padded to 32, slots permuted."""
    return make_case("cfgP_28of32", [tree_paper_geometry() for _ in range(B)], seed=seed, Hk=16,
                     Hv=32, d=128, in_dtype="bf16", n_layers=n_layers, Ns=32, permute_slots=True)


# ---------------------------------------------------------------------------
# attention half: KV cache, tree queries and entries
# ---------------------------------------------------------------------------
def spine_first_slots(parent: Sequence[int]) -> List[int]:
    """Slot map that places the principal spine (from the first child of the pre-tree state, always the
    lowest-index child) in slots 0, 1, ... and the remaining nodes after it in logical order (the layout
    of Sec. "One slot map governs attention and publication")."""
    ch = _children(parent)
    spine, cur = [], -1
    while ch[cur]:
        cur = ch[cur][0]
        spine.append(cur)
    on = set(spine)
    order = spine + [i for i in range(len(parent)) if i not in on]
    slot = [0] * len(parent)
    for s, i in enumerate(order):
        slot[i] = s
    return slot


@dataclasses.dataclass
class AttnCase:
    """Inputs of one full-attention layer; float arrays are float32 holding bf16 values exactly."""
    name: str
    B: int
    N: int
    Ns: int
    Hq: int
    Hkv: int
    dh: int
    scale: float
    parent: np.ndarray      # int32 [B, N]
    slot: np.ndarray        # int32 [B, N]
    ctx_len: np.ndarray     # int32 [B]
    cache_row: np.ndarray   # int32 [B]
    q: np.ndarray           # [B, N, Hq, dh]
    k_new: np.ndarray       # [B, N, Hkv, dh]
    v_new: np.ndarray
    k_cache: np.ndarray     # [rows, S, Hkv, dh]; the suffix holds unrelated values until the tree is written
    v_cache: np.ndarray
    accepted: np.ndarray    # int32 [B, lmax], -1 padded
    accepted_len: np.ndarray
    lmax: int


def make_attn_case(name: str, parents: Sequence[Sequence[int]], ctx_len: Sequence[int], *, seed: int, Hq: int, Hkv: int,
                   dh: int = 128, Ns: Optional[int] = None, layout: str = "identity", max_positions: Optional[int] = None,
                   extra_rows: int = 1, layer: int = 0) -> AttnCase:
    """layout: "identity", "spine" (spine_first_slots) or "permuted" (seeded injective map into Ns slots).
    q, k, v ~ N(0, 1); scale = dh^-1/2, so logits are ~N(0, 1) like trained attention at moderate temperature."""
    B, N = len(parents), len(parents[0])
    Ns = N if Ns is None else Ns
    parent = np.asarray(parents, dtype=np.int32).reshape(B, N)
    slot = np.tile(np.arange(N, dtype=np.int32), (B, 1))
    for b in range(B):
        if layout == "spine":
            slot[b] = np.asarray(spine_first_slots(parents[b]), dtype=np.int32)
        elif layout == "permuted":
            rs = IntStream(stream_key(seed, _T["slot"], b, 77))
            perm = list(range(Ns))
            for i in range(Ns - 1, 0, -1):
                j = rs.randint(0, i)
                perm[i], perm[j] = perm[j], perm[i]
            slot[b] = np.asarray(perm[:N], dtype=np.int32)
        elif layout != "identity":
            raise ValueError(layout)
    ctx = np.asarray(ctx_len, dtype=np.int32).reshape(B)
    S = int(ctx.max()) + Ns if max_positions is None else int(max_positions)
    rows = B + extra_rows
    rows_perm = list(range(rows))
    rs = IntStream(stream_key(seed, _T["rows"], 77))
    for i in range(rows - 1, 0, -1):
        j = rs.randint(0, i)
        rows_perm[i], rows_perm[j] = rows_perm[j], rows_perm[i]
    cache_row = np.asarray(rows_perm[:B], dtype=np.int32)

    def draw(tid: int, shape) -> np.ndarray:
        n = int(np.prod(shape))
        return round_to(normals(stream_key(seed, tid, layer, 77), n).reshape(shape), "bf16")

    q = draw(_T["q"], (B, N, Hq, dh))
    k_new = draw(_T["k"], (B, N, Hkv, dh))
    v_new = draw(_T["v"], (B, N, Hkv, dh))
    k_cache = draw(_T["state"], (rows, S, Hkv, dh))
    v_cache = draw(_T["hist"], (rows, S, Hkv, dh))
    acc_lists = [draw_accepted(IntStream(stream_key(seed, _T["accept"], b, 77)), parents[b]) for b in range(B)]
    lmax = max(max(tree_depths(p)) for p in parents)
    acc = np.full((B, lmax), -1, dtype=np.int32)
    ln = np.zeros(B, dtype=np.int32)
    for b, a in enumerate(acc_lists):
        acc[b, :len(a)] = a
        ln[b] = len(a)
    return AttnCase(name, B, N, Ns, Hq, Hkv, dh, float(dh) ** -0.5, parent, slot, ctx, cache_row, q, k_new, v_new,
                    k_cache, v_cache, acc, ln, lmax)
