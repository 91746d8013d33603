"""Parity of the attention half (tree KV write, ancestry-masked decode attention, KV publication) with
the fp64 oracle, through the C ABI.

Tolerance of the attention outputs.  Inputs are bf16 on both sides; logits are exact products summed in
fp32; the only rounding that matters is that of the probabilities to bf16 (unit roundoff of bf16: relative 2^-8 each) before the
second product, whose sums are fp32 again.  So per output element

    |out - ref| <= 2^-8 * sum_p softmax_p |v_p|  (+ fp32 noise),

and the oracle evaluates that bound itself (the same attention over |v|).  The test allows 1.05 x the bound
plus 2e-5 (1 + |ref|) for the fp32 sums and the exp2 approximation; lse within 2e-5 (1 + |ref|)."""
import numpy as np
import pytest
import torch

from oracle import attn_oracle as A
from paper_2609_23900_b200 import binding
from synthetic import workload as W
from synthetic.device_case import DeviceAttnCase
from tests.harness import ctx

pytestmark = pytest.mark.gpu


def oracle_caches(c):
    return A.kv_write(c.slot, c.k_new, c.v_new, c.k_cache, c.v_cache, c.ctx_len, c.cache_row)


def check_attention(dc, c, k1, v1, what, layer=0):
    ref, lse = A.tree_attention(c.parent, c.slot, c.q, k1, v1, c.ctx_len, c.cache_row, c.scale)
    bound, _ = A.tree_attention(c.parent, c.slot, c.q, k1, np.abs(v1), c.ctx_len, c.cache_row, c.scale)
    got, got_lse = dc.np("out", layer), dc.np("lse", layer)
    assert np.all(np.isfinite(got)) and np.all(np.isfinite(got_lse)), f"{what}: non-finite values"
    err = np.abs(got - ref)
    tol = 1.05 * 2.0 ** -8 * bound + 2e-5 * (1.0 + np.abs(ref))
    assert (err <= tol).all(), f"{what}: {(err > tol).sum()} outputs outside tolerance, worst ratio {(err / tol).max():.2f}"
    el = np.abs(got_lse - lse)
    assert (el <= 2e-5 * (1.0 + np.abs(lse))).all(), f"{what}: lse worst {el.max():.3e}"
    assert dc.t("status", layer).tolist() == [0] * c.B
    return float((err / tol).max())


def trees(kind, B, N, seed):
    if kind == "paper":
        return [W.tree_paper_geometry() for _ in range(B)]
    if kind == "chain":
        return [W.tree_chain(N) for _ in range(B)]
    if kind == "star":
        return [W.tree_star(N) for _ in range(B)]
    return [W.tree_random(W.IntStream(W.stream_key(seed, b)), N, 8) for b in range(B)]


CASES = [
    # name, tree kind, B, N, Ns, Hq, Hkv, ctx lengths, layout, n_splits
    ("tiny_ctx0", "random", 2, 7, 7, 2, 1, [0, 3], "identity", 1),
    ("paper_b1_split4", "paper", 1, 28, 32, 8, 2, [1000], "spine", 4),            # the paper's geometry, 4 partitions
    ("paper_b3_auto", "paper", 3, 28, 32, 8, 2, [517, 64, 1999], "permuted", 0),
    ("ragged_tiles", "random", 4, 16, 24, 4, 4, [63, 64, 65, 127], "permuted", 3),   # context ends at / around tile edges
    ("group_of_one", "random", 2, 32, 32, 4, 4, [300, 90], "spine", 2),           # G = 1: 32 of 128 rows in use
    ("two_row_tiles", "random", 2, 40, 48, 8, 1, [200, 333], "permuted", 2),      # G N = 320 rows: three row tiles
    ("wide_suffix", "star", 1, 200, 256, 2, 2, [130], "permuted", 2),             # suffix of four key tiles
    ("deep_chain", "chain", 2, 64, 64, 4, 2, [0, 1], "permuted", 1),
    ("more_splits_than_tiles", "random", 2, 8, 8, 4, 2, [10, 100], "identity", 8),
    # a unit spread over many CTAs: the merge takes more slots than one flight of its wide variant holds
    ("long_b1_auto", "paper", 1, 28, 32, 8, 2, [16384], "spine", 0),
    ("split32", "paper", 1, 28, 32, 4, 1, [5000], "spine", 32),
]


@pytest.mark.parametrize("kv_layout", [0, 1], ids=["pos_major", "head_major"])
@pytest.mark.parametrize("name,kind,B,N,Ns,Hq,Hkv,ctxs,layout,splits", CASES, ids=[c[0] for c in CASES])
def test_write_attend_publish_match_the_oracle(name, kind, B, N, Ns, Hq, Hkv, ctxs, layout, splits, kv_layout):
    c = W.make_attn_case(name, trees(kind, B, N, 900), ctxs, seed=W.BASE_SEED + 40, Hq=Hq, Hkv=Hkv, Ns=Ns, layout=layout)
    dc = DeviceAttnCase(ctx(), c, n_splits=splits, kv_layout=kv_layout)
    dc.write()
    k1, v1 = oracle_caches(c)
    torch.cuda.synchronize()
    assert np.array_equal(dc.np("k_cache"), k1) and np.array_equal(dc.np("v_cache"), v1), "tree KV write"
    dc.attend()
    check_attention(dc, c, k1, v1, name)
    dc.publish()
    k2, v2, ctx2, st = A.kv_publish(c.parent, c.slot, k1, v1, c.ctx_len, c.cache_row, c.accepted, c.accepted_len)
    assert dc.t("status").tolist() == st.tolist() == [0] * B
    assert dc.ctx_len_out.tolist() == ctx2.tolist()
    assert np.array_equal(dc.np("k_cache"), k2) and np.array_equal(dc.np("v_cache"), v2), "publication"


def test_bytes_outside_the_visible_set_never_reach_an_output():
    """Poison (NaN patterns) in padding slots, beyond the suffix, in the unused cache row and, for one node,
    in every other branch: outputs stay bitwise what they were."""
    c = W.make_attn_case("poison", trees("random", 2, 20, 31), [150, 70], seed=W.BASE_SEED + 41, Hq=4, Hkv=2, Ns=40,
                         layout="permuted", max_positions=300)
    dc = DeviceAttnCase(ctx(), c, n_splits=2)
    dc.write()
    dc.attend()
    torch.cuda.synchronize()
    out0, lse0 = dc.t("out").clone(), dc.t("lse").clone()
    kc, vc = dc.t("k_cache"), dc.t("v_cache")
    nan = float("nan")
    used_rows = set(c.cache_row.tolist())
    for r in range(kc.shape[0]):
        if r not in used_rows:
            kc[r] = nan
            vc[r] = nan
    for b in range(c.B):
        row, cx = int(c.cache_row[b]), int(c.ctx_len[b])
        owned = set(c.slot[b].tolist())
        for s in range(c.Ns):
            if s not in owned:
                kc[row, cx + s] = nan
                vc[row, cx + s] = nan
        kc[row, cx + c.Ns:] = nan
        vc[row, cx + c.Ns:] = nan
    dc.attend()
    torch.cuda.synchronize()
    assert torch.equal(dc.t("out"), out0) and torch.equal(dc.t("lse"), lse0)
    # other branches: node i's row must not change when a non-ancestor's entry is poisoned
    b, i = 0, c.N - 1
    anc = set(A.ancestry(c.parent[b], i))
    row, cx = int(c.cache_row[b]), int(c.ctx_len[b])
    for j in range(c.N):
        if j not in anc:
            kc[row, cx + int(c.slot[b, j])] = 1e30      # finite: those rows are legitimately read by other nodes
            vc[row, cx + int(c.slot[b, j])] = -1e30
    dc.attend()
    torch.cuda.synchronize()
    assert torch.equal(dc.t("out")[b, i], out0[b, i]) and torch.equal(dc.t("lse")[b, i], lse0[b, i])


def test_slot_layout_does_not_change_the_logical_result_beyond_rounding_and_repeats_bitwise():
    parents = trees("paper", 2, 28, 0)
    outs = {}
    for layout in ("identity", "spine", "permuted"):
        c = W.make_attn_case("layout", parents, [700, 45], seed=W.BASE_SEED + 42, Hq=8, Hkv=2, Ns=32, layout=layout)
        dc = DeviceAttnCase(ctx(), c, n_splits=4)
        dc.write()
        dc.attend()
        torch.cuda.synchronize()
        outs[layout] = (dc.t("out").clone(), dc.t("lse").clone())
        dc.attend()                                  # same inputs again: bit for bit
        torch.cuda.synchronize()
        assert torch.equal(dc.t("out"), outs[layout][0]) and torch.equal(dc.t("lse"), outs[layout][1])
        k1, v1 = oracle_caches(c)
        check_attention(dc, c, k1, v1, layout)
    # the three layouts order the suffix keys differently inside a tile: equal up to fp32 summation order
    for layout in ("spine", "permuted"):
        assert torch.allclose(outs[layout][0], outs["identity"][0], rtol=0, atol=2 ** -7)


def test_bad_rows_and_contexts_are_reported_and_skipped():
    c = W.make_attn_case("bad", trees("random", 3, 10, 5), [20, 30, 40], seed=W.BASE_SEED + 43, Hq=4, Hkv=2, Ns=12,
                         layout="identity", max_positions=60)
    dc = DeviceAttnCase(ctx(), c, n_splits=2)
    dc.cache_row[0] = 99                     # no such row
    dc.ctx_len[2] = 49                       # 49 + 12 > 60
    k0, v0 = dc.t("k_cache").clone(), dc.t("v_cache").clone()
    dc.write()
    torch.cuda.synchronize()
    assert dc.t("status").tolist() == [binding.SEQ_BAD_ROW, 0, binding.SEQ_BAD_CTX]
    row1 = int(c.cache_row[1])
    others = [r for r in range(k0.shape[0]) if r != row1]
    assert torch.equal(dc.t("k_cache")[others], k0[others]) and torch.equal(dc.t("v_cache")[others], v0[others])
    dc.attend()
    torch.cuda.synchronize()
    assert dc.t("status").tolist() == [binding.SEQ_BAD_ROW, 0, binding.SEQ_BAD_CTX]
    out = dc.t("out")
    assert (out[0] == 0).all() and (out[2] == 0).all() and (dc.t("lse")[0] == 0).all()
    k1, v1 = oracle_caches(c)
    ref, _ = A.tree_attention(c.parent[1:2], c.slot[1:2], c.q[1:2], k1, v1, c.ctx_len[1:2], c.cache_row[1:2], c.scale)
    assert np.abs(dc.np("out")[1] - ref[0]).max() < 2e-2
    k_before = dc.t("k_cache").clone()
    dc.publish()
    torch.cuda.synchronize()
    assert dc.t("status").tolist() == [binding.SEQ_BAD_ROW, 0, binding.SEQ_BAD_CTX]
    assert dc.ctx_len_out.tolist() == [20, 30 + int(c.accepted_len[1]), 49]
    assert torch.equal(dc.t("k_cache")[others], k_before[others])


def test_publication_rules_invalid_paths_length_zero_and_spine_first_identity():
    parents = trees("paper", 4, 28, 0)
    c = W.make_attn_case("pub", parents, [10, 20, 30, 40], seed=W.BASE_SEED + 44, Hq=8, Hkv=2, Ns=32, layout="spine")
    # sequence 0: the whole principal spine (already in place); 1: nothing; 2: broken link; 3: a rescue branch
    spine = [0, 1, 4, 7, 10, 13, 16, 17, 18, 19, 20, 21]
    acc = np.full((4, 12), -1, dtype=np.int32)
    acc[0, :12] = spine
    acc[2, :3] = [0, 1, 7]
    branch = A.ancestry(parents[3], 25)
    acc[3, :len(branch)] = branch
    c.accepted, c.accepted_len, c.lmax = acc, np.array([12, 0, 3, len(branch)], dtype=np.int32), 12
    dc = DeviceAttnCase(ctx(), c)
    dc.write()
    torch.cuda.synchronize()
    before_k = dc.t("k_cache").clone()
    dc.publish()
    torch.cuda.synchronize()
    k1, v1 = oracle_caches(c)
    k2, v2, ctx2, st = A.kv_publish(c.parent, c.slot, k1, v1, c.ctx_len, c.cache_row, c.accepted, c.accepted_len)
    assert st.tolist() == [0, 0, binding.SEQ_BAD_LINK, 0] == dc.t("status").tolist()
    assert dc.ctx_len_out.tolist() == ctx2.tolist() == [22, 20, 30, 40 + len(branch)]
    assert np.array_equal(dc.np("k_cache"), k2) and np.array_equal(dc.np("v_cache"), v2)
    for b in (0, 1, 2):                         # spine in place, nothing accepted, refused: rows bitwise untouched
        r = int(c.cache_row[b])
        assert torch.equal(dc.t("k_cache")[r], before_k[r])


def test_attention_after_publication_continues_the_accepted_path():
    """Two cycles: write, attend, publish; then a new tree on the advanced context.  The second cycle's
    attention must equal the oracle run on the oracle's own published cache."""
    parents = trees("random", 2, 12, 77)
    c = W.make_attn_case("cycle1", parents, [100, 37], seed=W.BASE_SEED + 45, Hq=4, Hkv=2, Ns=16, layout="permuted",
                         max_positions=200)
    dc = DeviceAttnCase(ctx(), c, n_splits=2)
    dc.write(); dc.attend(); dc.publish()
    torch.cuda.synchronize()
    k1, v1 = oracle_caches(c)
    k2, v2, ctx2, _ = A.kv_publish(c.parent, c.slot, k1, v1, c.ctx_len, c.cache_row, c.accepted, c.accepted_len)
    c2 = W.make_attn_case("cycle2", trees("random", 2, 12, 78), ctx2.tolist(), seed=W.BASE_SEED + 46, Hq=4, Hkv=2, Ns=16,
                          layout="spine", max_positions=200)
    c2.cache_row = c.cache_row
    c2.k_cache, c2.v_cache = k2.astype(np.float32), v2.astype(np.float32)
    dc2 = DeviceAttnCase(ctx(), c2, n_splits=2)
    # the device continues on ITS cache and ITS advanced context lengths
    dc2.layers[0].tensors["k_cache"].copy_(dc.t("k_cache"))
    dc2.layers[0].tensors["v_cache"].copy_(dc.t("v_cache"))
    dc2.ctx_len.copy_(dc.ctx_len_out)
    dc2.write(); dc2.attend()
    torch.cuda.synchronize()
    k3, v3 = oracle_caches(c2)
    check_attention(dc2, c2, k3, v3, "second cycle")


def test_several_layers_in_one_call_and_optional_outputs():
    """Two layers with different inputs through one call each of write, attend and publish; the second
    layer without lse and without status words."""
    parents = trees("random", 2, 14, 5)
    cs = [W.make_attn_case("multi", parents, [90, 310], seed=W.BASE_SEED + 47, Hq=4, Hkv=2, Ns=16, layout="spine", layer=l,
                           max_positions=340) for l in range(2)]
    dc = DeviceAttnCase(ctx(), cs[0], cases=cs, n_splits=0)
    L1 = dc.layers[1]
    L1.tensors["lse"], L1.tensors["status"] = None, None
    L1.args.lse, L1.args.status = None, None
    dc.packed = ctx().pack_attn(dc.layers)
    dc.write(); dc.attend()
    torch.cuda.synchronize()
    for l, c in enumerate(cs):
        k1, v1 = oracle_caches(c)
        ref, _ = A.tree_attention(c.parent, c.slot, c.q, k1, v1, c.ctx_len, c.cache_row, c.scale)
        bound, _ = A.tree_attention(c.parent, c.slot, c.q, k1, np.abs(v1), c.ctx_len, c.cache_row, c.scale)
        err = np.abs(dc.np("out", l) - ref)
        assert (err <= 1.05 * 2.0 ** -8 * bound + 2e-5 * (1.0 + np.abs(ref))).all(), f"layer {l}"
    dc.publish()
    torch.cuda.synchronize()
    for l, c in enumerate(cs):
        k1, v1 = oracle_caches(c)
        k2, v2, ctx2, _ = A.kv_publish(c.parent, c.slot, k1, v1, c.ctx_len, c.cache_row, c.accepted, c.accepted_len)
        assert np.array_equal(dc.np("k_cache", l), k2) and np.array_equal(dc.np("v_cache", l), v2), f"layer {l} publication"
    assert dc.ctx_len_out.tolist() == ctx2.tolist()


def test_host_side_refusals_enqueue_nothing():
    c = W.make_attn_case("refuse", trees("random", 1, 6, 1), [10], seed=1, Hq=4, Hkv=2, Ns=8, layout="identity")
    cx = ctx()
    dc = DeviceAttnCase(cx, c)
    out0 = dc.t("out").clone()

    def refused(mutate, call=None, code=None):
        L = dc.layers[0]
        saved = {f[0]: getattr(L.args, f[0]) for f in L.args._fields_}
        mutate(L.args)
        try:
            with pytest.raises(binding.LumoError) as e:
                (call or (lambda: cx.tree_attention(dc.desc, cx.pack_attn([L]))))()
            if code is not None:
                assert e.value.code == code
        finally:
            for k, v in saved.items():
                setattr(L.args, k, v)

    refused(lambda a: setattr(a, "dh", 64), code=4)
    refused(lambda a: setattr(a, "Hq", 5), code=4)
    refused(lambda a: setattr(a, "scale", 0.0), code=1)
    refused(lambda a: setattr(a, "n_splits", 33), code=1)
    refused(lambda a: setattr(a, "kv_layout", 2), code=1)
    refused(lambda a: setattr(a, "max_positions", 4), code=1)          # fewer positions than slots
    refused(lambda a: setattr(a, "q", None), code=1)
    refused(lambda a: setattr(a, "k_new", None), call=lambda: cx.kv_write_tree(dc.desc, cx.pack_attn([dc.layers[0]])), code=1)
    refused(lambda a: None, call=lambda: cx.kv_publish(dc.desc, dc.packed, dc.accepted, dc.accepted_len, dc.ctx_len), code=1)  # alias
    wide = cx.tree_desc(np.array([[-1, 0]], dtype=np.int32), n_slots=300)
    with pytest.raises(binding.LumoError) as e:
        cx.tree_attention(wide, dc.packed)
    assert e.value.code == 4
    torch.cuda.synchronize()
    assert torch.equal(dc.t("out"), out0) or (torch.isnan(dc.t("out")) & torch.isnan(out0)).all()
    dc.write(); dc.attend()                                             # the context is still usable
    torch.cuda.synchronize()
    assert dc.t("status").tolist() == [0]


def test_write_attend_publish_replayed_from_one_cuda_graph():
    """The three calls captured once (after a warm-up that sizes the library's scratch) and replayed on new
    contents of the same buffers: new tree entries and queries, advanced context lengths, another accepted
    path.  Every replay must match the oracle run on the same contents (Sec. "Device-resident commitment":
    fixed-shape device products feed captured publication)."""
    parents = trees("paper", 2, 28, 0)
    c = W.make_attn_case("graph0", parents, [300, 77], seed=W.BASE_SEED + 60, Hq=8, Hkv=2, Ns=32, layout="spine",
                         max_positions=500)
    cx = ctx()
    dc = DeviceAttnCase(cx, c, n_splits=0)
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        dc.write(st); dc.attend(st); dc.publish(st)                 # warm-up outside capture (scratch, kernel attributes)
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            dc.write(st); dc.attend(st); dc.publish(st)
        k_host, v_host = c.k_cache.copy(), c.v_cache.copy()
        ctx_host = c.ctx_len.copy()
        for rep in range(3):
            cn = W.make_attn_case(f"graph{rep + 1}", parents, ctx_host.tolist(), seed=W.BASE_SEED + 61 + rep, Hq=8, Hkv=2,
                                  Ns=32, layout="spine", max_positions=500)
            cn.cache_row = c.cache_row
            cn.k_cache, cn.v_cache = k_host, v_host
            up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(torch.bfloat16).to(dc.dev)
            for name, arr in (("q", cn.q), ("k_new", cn.k_new), ("v_new", cn.v_new), ("k_cache", k_host), ("v_cache", v_host)):
                dc.t(name).copy_(up(arr))
            dc.ctx_len.copy_(torch.from_numpy(ctx_host).to(dc.dev))
            dc.accepted.fill_(-1)
            dc.accepted[:, :cn.accepted.shape[1]].copy_(torch.from_numpy(cn.accepted).to(dc.dev))
            dc.accepted_len.copy_(torch.from_numpy(cn.accepted_len).to(dc.dev))
            dc.t("out").fill_(float("nan")); dc.t("status").fill_(-1)
            g.replay()
            st.synchronize()
            k1, v1 = A.kv_write(cn.slot, cn.k_new, cn.v_new, k_host, v_host, ctx_host, cn.cache_row)
            ref, _ = A.tree_attention(cn.parent, cn.slot, cn.q, k1, v1, ctx_host, cn.cache_row, cn.scale)
            bound, _ = A.tree_attention(cn.parent, cn.slot, cn.q, k1, np.abs(v1), ctx_host, cn.cache_row, cn.scale)
            err = np.abs(dc.np("out") - ref)
            assert (err <= 1.05 * 2.0 ** -8 * bound + 2e-5 * (1.0 + np.abs(ref))).all(), f"replay {rep}"
            acc = np.full((2, c.lmax), -1, dtype=np.int32)
            acc[:, :cn.accepted.shape[1]] = cn.accepted
            k2, v2, ctx2, stt = A.kv_publish(cn.parent, cn.slot, k1, v1, ctx_host, cn.cache_row, acc, cn.accepted_len)
            assert dc.t("status").tolist() == stt.tolist() == [0, 0]
            assert np.array_equal(dc.np("k_cache"), k2) and np.array_equal(dc.np("v_cache"), v2), f"replay {rep} publication"
            assert dc.ctx_len_out.tolist() == ctx2.tolist()
            k_host, v_host, ctx_host = k2.astype(np.float32), v2.astype(np.float32), ctx2.astype(np.int32)
