"""fp64 oracle of the attention half of the tree verifier: ancestry-masked decode attention over
[committed context ; candidate tree] under a slot map, and the re-linearisation of the accepted
path's KV entries at publication.

TEST INFRASTRUCTURE ONLY: imported by tests; never by the product path.  Plain NumPy, float64, one
(sequence, query head, node) at a time; no blocking, no split, no fused rescaling.

What it computes (paper Sec. "One slot map governs attention and publication"; Sec. "State and the
execution boundary": the attention visibility relation selects the same logical prefix and ancestry as
the recurrent path; Algorithm 1, "remap KV"):

  * The KV cache of sequence b is row cache_row[b] of k_cache / v_cache [rows, S, Hkv, dh].  Positions
    [0, ctx_len[b]) hold the committed context; the entry of tree node i sits at position
    ctx_len[b] + slot[b][i] (the slot map places the candidates in the physical suffix; logical query
    order is kept: q and out are indexed by logical node).
  * Node i sees every context position and the entries of its ancestors and of itself, nothing else
    (padding slots and other branches are invisible).  Query head h reads KV head h // (Hq / Hkv).
  * The tree's own entries reach the cache through the same map: kv_write puts the key / value of node i
    at position ctx_len[b] + slot[b][i] before attention runs.
  * logits = scale * q . k;  lse = log sum exp(logits);  out = sum softmax(logits) v.
    Keys are taken in logical order (context ascending, then the ancestry root first, the node last), so
    the result does not depend on the slot map bit for bit.
  * Publication: the accepted path a_0 .. a_{L-1} moves entry ctx + slot[a_t] to position ctx + t (all
    reads before any write), the new context length is ctx + L.  An invalid path (same four rules as the
    recurrent commit) changes nothing and sets a status code.

Readings where the paper is silent: the softmax scale is a parameter; the grouping of query heads and
the number of split-K partitions are kernel schedule, not semantics (the oracle has neither);
`merge_partials` states the log-sum-exp combination rule any split must satisfy.

Pins (tests/test_oracle_attn.py): a chain tree equals causal attention by
torch.nn.functional.scaled_dot_product_attention; visibility by poisoning invisible entries; slot
permutation invariance bit for bit; single-key and uniform-logit closed forms; the split merge identity;
the grouped-head map; the write by a hand-worked table and by "write, attend, publish" against plain
causal attention over the appended path; publication by hand-worked tables and by "attention over the published cache equals
tree attention at the accepted node".
"""
from __future__ import annotations

import numpy as np

SEQ_OK, SEQ_BAD_LEN, SEQ_BAD_NODE, SEQ_BAD_ROOT, SEQ_BAD_LINK = 0, 1, 2, 3, 4


def ancestry(parent, i):
    """Root-first list of the ancestors of node i followed by i itself."""
    path = []
    while i >= 0:
        path.append(int(i))
        i = int(parent[i])
    return path[::-1]


def visible_positions(parent, slot, ctx, i):
    """Cache positions node i attends to, in logical order."""
    return list(range(int(ctx))) + [int(ctx) + int(slot[a]) for a in ancestry(parent, i)]


def attend(q, K, V, scale):
    """One query vector over explicit key / value rows: (out, lse) in float64."""
    logits = scale * (K @ q)
    m = logits.max()
    w = np.exp(logits - m)
    l = w.sum()
    return (w @ V) / l, m + np.log(l)


def tree_attention(parent, slot, q, k_cache, v_cache, ctx_len, cache_row, scale):
    """out [B, N, Hq, dh], lse [B, N, Hq]."""
    parent, slot = np.asarray(parent), np.asarray(slot)
    q = np.asarray(q, np.float64)
    k_cache, v_cache = np.asarray(k_cache, np.float64), np.asarray(v_cache, np.float64)
    B, N, Hq, dh = q.shape
    Hkv = k_cache.shape[2]
    assert Hq % Hkv == 0
    out = np.zeros((B, N, Hq, dh))
    lse = np.zeros((B, N, Hq))
    for b in range(B):
        row = int(cache_row[b])
        for i in range(N):
            pos = visible_positions(parent[b], slot[b], ctx_len[b], i)
            for h in range(Hq):
                g = h // (Hq // Hkv)
                out[b, i, h], lse[b, i, h] = attend(q[b, i, h], k_cache[row, pos, g], v_cache[row, pos, g], scale)
    return out, lse


def kv_write(slot, k_new, v_new, k_cache, v_cache, ctx_len, cache_row):
    """Places the tree's entries: k_new / v_new [B, N, Hkv, dh] (logical node order) go to position
    ctx_len[b] + slot[b][i] of row cache_row[b].  Returns new caches; inputs untouched."""
    k2, v2 = np.array(k_cache, copy=True), np.array(v_cache, copy=True)
    B, N = np.asarray(slot).shape
    for b in range(B):
        for i in range(N):
            p = int(ctx_len[b]) + int(slot[b][i])
            k2[int(cache_row[b]), p] = k_new[b][i]
            v2[int(cache_row[b]), p] = v_new[b][i]
    return k2, v2


def merge_partials(outs, lses):
    """Combination of attention results over disjoint key sets: the rule a split-K schedule must obey.
    outs [P, dh], lses [P] -> (out, lse)."""
    outs, lses = np.asarray(outs, np.float64), np.asarray(lses, np.float64)
    m = lses.max()
    w = np.exp(lses - m)
    return (w[:, None] * outs).sum(0) / w.sum(), m + np.log(w.sum())


def check_path(parent, acc, length, lmax):
    N = len(parent)
    if length < 0 or length > lmax:
        return SEQ_BAD_LEN
    prev = -1
    for t in range(length):
        a = int(acc[t])
        if a < 0 or a >= N:
            return SEQ_BAD_NODE
        if t == 0:
            if parent[a] != -1:
                return SEQ_BAD_ROOT
        elif parent[a] != prev:
            return SEQ_BAD_LINK
        prev = a
    return SEQ_OK


def kv_publish(parent, slot, k_cache, v_cache, ctx_len, cache_row, accepted, length):
    """(k_cache', v_cache', ctx_len', status [B]); inputs untouched."""
    k2, v2 = np.array(k_cache, copy=True), np.array(v_cache, copy=True)
    ctx2 = np.array(ctx_len, dtype=np.int32, copy=True)
    B = len(ctx_len)
    lmax = np.asarray(accepted).shape[1]
    status = np.zeros(B, dtype=np.int32)
    for b in range(B):
        L = int(length[b])
        st = check_path(np.asarray(parent[b]), accepted[b], L, lmax)
        status[b] = st
        if st != SEQ_OK or L == 0:
            continue
        row, ctx = int(cache_row[b]), int(ctx_len[b])
        src = [ctx + int(slot[b][int(accepted[b][t])]) for t in range(L)]
        kk, vv = k_cache[row, src].copy(), v_cache[row, src].copy()      # all reads before any write
        k2[row, ctx:ctx + L] = kk
        v2[row, ctx:ctx + L] = vv
        ctx2[b] = ctx + L
    return k2, v2, ctx2, status
