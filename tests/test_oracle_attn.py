"""Pins for the attention oracle (oracle/attn_oracle.py): every check compares it with something fixed by
the mathematics or computed by another route (a library attention routine, closed forms, hand tables),
never with a re-typed copy of its own loop."""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as A
from synthetic import workload as W


def make(parents, *, seed=0, Hq=4, Hkv=2, dh=16, ctx=(5, 9), Ns=None, permute=False, S=None):
    rs = np.random.default_rng(seed)
    B, N = len(parents), len(parents[0])
    Ns = N if Ns is None else Ns
    parent = np.asarray(parents, dtype=np.int32)
    slot = np.tile(np.arange(N, dtype=np.int32), (B, 1))
    if permute:
        for b in range(B):
            slot[b] = rs.permutation(Ns)[:N]
    ctx_len = np.asarray([ctx[b % len(ctx)] for b in range(B)], dtype=np.int32)
    S = int(ctx_len.max()) + Ns + 3 if S is None else S
    rows = B + 1
    cache_row = rs.permutation(rows)[:B].astype(np.int32)
    q = rs.standard_normal((B, N, Hq, dh))
    k_cache = rs.standard_normal((rows, S, Hkv, dh))
    v_cache = rs.standard_normal((rows, S, Hkv, dh))
    return dict(parent=parent, slot=slot, q=q, k_cache=k_cache, v_cache=v_cache, ctx_len=ctx_len,
                cache_row=cache_row, scale=dh ** -0.5, N=N, Ns=Ns, B=B)


def run(c):
    return A.tree_attention(c["parent"], c["slot"], c["q"], c["k_cache"], c["v_cache"], c["ctx_len"], c["cache_row"], c["scale"])


def test_chain_tree_equals_causal_attention_by_the_library_routine():
    """A chain with identity slots is a token sequence appended to the context: node i sees positions
    0 .. ctx + i.  torch's scaled_dot_product_attention with that mask and repeated KV heads is the pin
    (also pins the map of query heads onto KV heads)."""
    n = 7
    c = make([W.tree_chain(n)] * 2, seed=1, Hq=6, Hkv=2, dh=8, ctx=(4, 11))
    out, lse = run(c)
    for b in range(c["B"]):
        ctx, row = int(c["ctx_len"][b]), int(c["cache_row"][b])
        T = ctx + n
        q = torch.from_numpy(c["q"][b]).permute(1, 0, 2)                      # [Hq, n, dh]
        k = torch.from_numpy(c["k_cache"][row, :T]).permute(1, 0, 2).repeat_interleave(3, dim=0)
        v = torch.from_numpy(c["v_cache"][row, :T]).permute(1, 0, 2).repeat_interleave(3, dim=0)
        mask = torch.arange(T)[None, :] <= (ctx + torch.arange(n))[:, None]
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask, scale=c["scale"])
        np.testing.assert_allclose(out[b], ref.permute(1, 0, 2).numpy(), rtol=1e-12, atol=1e-14)
        logits = c["scale"] * torch.einsum("hnd,htd->hnt", q, k).masked_fill(~mask, float("-inf"))
        np.testing.assert_allclose(lse[b], torch.logsumexp(logits, -1).T.numpy(), rtol=1e-12, atol=1e-13)


def test_visibility_is_context_plus_ancestors_and_self():
    """Entries of other branches, of padding slots and beyond the suffix are never read (poison them with
    NaN: bitwise unchanged); an ancestor's entry is read (poison it: the result changes)."""
    parents = [[-1, -1, 0, 0, 1, 1, 2]]
    c = make(parents, seed=2, Ns=10, permute=True)
    out, lse = run(c)
    ctx, row = int(c["ctx_len"][0]), int(c["cache_row"][0])
    node = 6                                                            # path 0 -> 2 -> 6
    vis = set(A.visible_positions(c["parent"][0], c["slot"][0], ctx, node))
    assert vis == set(range(ctx)) | {ctx + int(c["slot"][0][a]) for a in (0, 2, 6)}
    k2, v2 = c["k_cache"].copy(), c["v_cache"].copy()
    for p in range(k2.shape[1]):
        if p not in vis:
            k2[row, p] = np.nan
            v2[row, p] = np.nan
    o2, l2 = A.tree_attention(c["parent"], c["slot"], c["q"], k2, v2, c["ctx_len"], c["cache_row"], c["scale"])
    assert np.array_equal(o2[0, node], out[0, node]) and np.array_equal(l2[0, node], lse[0, node])
    k3 = c["k_cache"].copy()
    k3[row, ctx + int(c["slot"][0][2])] += 1.0
    o3, _ = A.tree_attention(c["parent"], c["slot"], c["q"], k3, c["v_cache"], c["ctx_len"], c["cache_row"], c["scale"])
    assert not np.array_equal(o3[0, node], out[0, node])
    assert np.array_equal(o3[0, 4], out[0, 4])                         # node 4 (path 1 -> 4) does not see node 2


def test_slot_permutation_leaves_logical_results_bitwise_unchanged():
    parents = [W.tree_random(W.IntStream(5 + b), 12, 5) for b in range(2)]
    c = make(parents, seed=3, Ns=12)
    out, lse = run(c)
    rs = np.random.default_rng(9)
    c2 = dict(c)
    c2["slot"] = c["slot"].copy()
    c2["k_cache"], c2["v_cache"] = c["k_cache"].copy(), c["v_cache"].copy()
    Ns = 15
    for b in range(c["B"]):
        perm = rs.permutation(Ns)[:c["N"]].astype(np.int32)
        ctx, row = int(c["ctx_len"][b]), int(c["cache_row"][b])
        c2["k_cache"][row, ctx:] = rs.standard_normal(c2["k_cache"][row, ctx:].shape)     # fresh garbage in the suffix
        c2["v_cache"][row, ctx:] = rs.standard_normal(c2["v_cache"][row, ctx:].shape)
        for i in range(c["N"]):
            c2["k_cache"][row, ctx + perm[i]] = c["k_cache"][row, ctx + c["slot"][b, i]]
            c2["v_cache"][row, ctx + perm[i]] = c["v_cache"][row, ctx + c["slot"][b, i]]
        c2["slot"][b] = perm
    # the cache must be long enough for the wider suffix
    assert c2["k_cache"].shape[1] >= int(c["ctx_len"].max()) + Ns
    o2, l2 = run(c2)
    assert np.array_equal(o2, out) and np.array_equal(l2, lse)


def test_closed_forms_single_key_and_uniform_logits():
    c = make([[-1, 0, 0]], seed=4, ctx=(0,), Hq=2, Hkv=1, dh=8)
    out, lse = run(c)
    row = int(c["cache_row"][0])
    # node 0 with an empty context sees its own entry only: out = v, lse = scale q.k
    np.testing.assert_allclose(out[0, 0, 1], c["v_cache"][row, 0, 0], rtol=0, atol=1e-15)
    np.testing.assert_allclose(lse[0, 0, 1], c["scale"] * c["q"][0, 0, 1] @ c["k_cache"][row, 0, 0], rtol=1e-14)
    # zero query: uniform weights over the visible entries
    c["q"][:] = 0.0
    out, lse = run(c)
    np.testing.assert_allclose(out[0, 2, 0], c["v_cache"][row, [0, 2], 0].mean(0), rtol=1e-14)
    np.testing.assert_allclose(lse[0, 2, 0], np.log(2.0), rtol=1e-14)


@pytest.mark.parametrize("cuts", [(3,), (1, 2, 9), (5, 6, 7, 8)])
def test_partial_results_over_disjoint_key_sets_merge_to_the_whole(cuts):
    """The log-sum-exp combination rule of split-K schedules, on arbitrary partitions of the visible keys."""
    rs = np.random.default_rng(6)
    K, V, q = rs.standard_normal((11, 8)) * 3, rs.standard_normal((11, 8)), rs.standard_normal(8)
    whole_o, whole_l = A.attend(q, K, V, 0.7)
    edges = (0,) + cuts + (11,)
    parts = [A.attend(q, K[a:b], V[a:b], 0.7) for a, b in zip(edges[:-1], edges[1:])]
    o, l = A.merge_partials([p[0] for p in parts], [p[1] for p in parts])
    np.testing.assert_allclose(o, whole_o, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(l, whole_l, rtol=1e-14)


def test_publication_hand_worked_with_overlapping_moves():
    """ctx = 2; tree 0 -> 1 -> 2 stored at slots [2, 0, 1]: the accepted path (0, 1, 2) moves
    positions (4, 2, 3) to (2, 3, 4).  Position 2 is both a destination (of node 0) and a source (of node 1):
    reads must come before writes."""
    parent = np.array([[-1, 0, 1]], dtype=np.int32)
    slot = np.array([[2, 0, 1]], dtype=np.int32)
    k = np.arange(8, dtype=np.float64).reshape(1, 8, 1, 1) * 10          # entry value = 10 x position
    v = -k
    acc = np.array([[0, 1, 2]], dtype=np.int32)
    k2, v2, ctx2, st = A.kv_publish(parent, slot, k, v, np.array([2]), np.array([0]), acc, np.array([3]))
    assert st.tolist() == [0] and ctx2.tolist() == [5]
    assert k2[0, :, 0, 0].tolist() == [0, 10, 40, 20, 30, 50, 60, 70]
    assert np.array_equal(v2, -k2)
    # spine-first layout (slot[a_t] = t): publication is the identity on the cache
    k3, _, ctx3, _ = A.kv_publish(parent, np.array([[0, 1, 2]], dtype=np.int32), k, v, np.array([2]), np.array([0]), acc, np.array([2]))
    assert np.array_equal(k3, k) and ctx3.tolist() == [4]
    # nothing accepted, and invalid paths: unchanged, with the code of the first failing rule
    for a, ln, code in (([0, 1, 2], 0, 0), ([1, 2, 0], 2, A.SEQ_BAD_ROOT), ([0, 2, 1], 2, A.SEQ_BAD_LINK),
                        ([0, 7, 1], 2, A.SEQ_BAD_NODE), ([0, 1, 2], 4, A.SEQ_BAD_LEN)):
        k4, v4, ctx4, st4 = A.kv_publish(parent, slot, k, v, np.array([2]), np.array([0]), np.array([a], dtype=np.int32), np.array([ln]))
        assert st4.tolist() == [code] and np.array_equal(k4, k) and np.array_equal(v4, v) and ctx4.tolist() == [2]


def test_attention_over_the_published_cache_equals_tree_attention_at_the_accepted_node():
    """After publication the accepted path is ordinary context: plain attention of the last accepted
    node's query over positions [0, ctx + L) of the new cache equals what the tree attention gave that
    node, bit for bit (same keys in the same order)."""
    parents = [W.tree_random(W.IntStream(40 + b), 14, 6) for b in range(3)]
    c = make(parents, seed=7, Ns=17, permute=True, Hq=4, Hkv=2)
    out, lse = run(c)
    depth = [W.tree_depths(p) for p in parents]
    acc = np.full((3, 6), -1, dtype=np.int32)
    ln = np.zeros(3, dtype=np.int32)
    for b in range(3):
        leaf = int(np.argmax(depth[b]))
        path = A.ancestry(c["parent"][b], leaf)
        acc[b, :len(path)] = path
        ln[b] = len(path)
    k2, v2, ctx2, st = A.kv_publish(c["parent"], c["slot"], c["k_cache"], c["v_cache"], c["ctx_len"], c["cache_row"], acc, ln)
    assert st.tolist() == [0, 0, 0]
    for b in range(3):
        row, T, last = int(c["cache_row"][b]), int(ctx2[b]), int(acc[b, ln[b] - 1])
        assert T == c["ctx_len"][b] + ln[b]
        for h in range(4):
            o, l = A.attend(c["q"][b, last, h], k2[row, :T, h // 2], v2[row, :T, h // 2], c["scale"])
            assert np.array_equal(o, out[b, last, h]) and l == lse[b, last, h]


def test_write_attend_publish_equals_plain_causal_attention_over_the_appended_path():
    """The three steps under one slot map: the tree's entries are written through the map, attention reads
    them through it, publication moves the accepted ones; the result is what a sequential decoder that
    appended the accepted tokens one by one would hold and compute (library attention, explicit lists)."""
    rs = np.random.default_rng(11)
    parent = np.array([[-1, 0, 0, 1, 1, 2, 4]], dtype=np.int32)
    slot = np.array([[0, 4, 1, 6, 2, 5, 3]], dtype=np.int32)            # spine 0 -> 1 -> 4 -> 6 is NOT contiguous here
    ctx, Hkv, Hq, dh, N = 6, 2, 4, 8, 7
    k_cache, v_cache = rs.standard_normal((2, 16, Hkv, dh)), rs.standard_normal((2, 16, Hkv, dh))
    k_new, v_new, q = rs.standard_normal((1, N, Hkv, dh)), rs.standard_normal((1, N, Hkv, dh)), rs.standard_normal((1, N, Hq, dh))
    ctx_len, row = np.array([ctx]), np.array([1])
    k1, v1 = A.kv_write(slot, k_new, v_new, k_cache, v_cache, ctx_len, row)
    # hand table: position ctx + s holds node slot^-1(s)
    inv = {int(s): i for i, s in enumerate(slot[0])}
    for s_, i in inv.items():
        assert np.array_equal(k1[1, ctx + s_], k_new[0, i]) and np.array_equal(v1[1, ctx + s_], v_new[0, i])
    assert np.array_equal(k1[0], k_cache[0]) and np.array_equal(k1[1, :ctx], k_cache[1, :ctx]) and np.array_equal(k1[1, ctx + N:], k_cache[1, ctx + N:])
    out, _ = A.tree_attention(parent, slot, q, k1, v1, ctx_len, row, 0.5)
    path = [0, 1, 4, 6]
    acc = np.array([path], dtype=np.int32)
    k2, v2, ctx2, st = A.kv_publish(parent, slot, k1, v1, ctx_len, row, acc, np.array([4]))
    assert st.tolist() == [0] and ctx2.tolist() == [ctx + 4]
    # the sequential decoder's cache: old context followed by the accepted tokens' entries
    Kseq = np.concatenate([k_cache[1, :ctx], k_new[0, path]], 0)
    Vseq = np.concatenate([v_cache[1, :ctx], v_new[0, path]], 0)
    assert np.array_equal(k2[1, :ctx + 4], Kseq) and np.array_equal(v2[1, :ctx + 4], Vseq)
    for t, node in enumerate(path):
        T = ctx + t + 1
        qq = torch.from_numpy(q[0, node])[:, None, :]                                    # [Hq, 1, dh]
        kk = torch.from_numpy(Kseq[:T]).permute(1, 0, 2).repeat_interleave(2, dim=0)
        vv = torch.from_numpy(Vseq[:T]).permute(1, 0, 2).repeat_interleave(2, dim=0)
        ref = torch.nn.functional.scaled_dot_product_attention(qq, kk, vv, scale=0.5)[:, 0]
        np.testing.assert_allclose(out[0, node], ref.numpy(), rtol=1e-12, atol=1e-14)
