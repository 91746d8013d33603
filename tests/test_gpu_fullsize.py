"""Parity at the full benchmark sizes, in the launch configuration bench.py times (conv + scan with
in-kernel q/k normalisation, bf16 outputs, then commit): the oracle is run on sampled (sequence,
value head) pairs and sampled layers, one by one, on the operands the GPU recorded."""
import numpy as np
import pytest
import torch

from oracle import gdn_oracle as O
from synthetic import workload as W
from synthetic.device_case import DeviceCase
from tests.harness import assert_close, ctx

pytestmark = pytest.mark.gpu


def check_conv_samples(dc, case, layer, seqs):
    """The operands the convolution recorded for the sampled sequences, element by element against the
    conv oracle (all channels, every row): the scan checks below read these same buffers on both sides,
    so they alone would not notice a wrong convolution."""
    L = case.layers[layer]
    hk = case.Hk * case.d
    for b in seqs:
        sl = slice(b, b + 1)
        y = O.conv(case.parent[sl], case.slot[sl], case.state_row[sl], L.x[sl], L.conv_w, L.conv_b, L.hist, case.Ns,
                   out_dtype="none")
        f = lambda name: dc.t(name, layer)[b].to(torch.float64).cpu().numpy()
        got = np.concatenate([f("q").reshape(case.Ns, hk), f("k").reshape(case.Ns, hk),
                              f("v").reshape(case.Ns, case.Hv * case.d)], axis=-1)
        assert_close(got, y[0], bf16=True, what=f"{case.name} layer {layer} b={b} recorded operands")


def check_samples(dc, case, layer, pairs):
    L = case.layers[layer]
    rep = case.Hv // case.Hk
    f = lambda name: dc.t(name, layer)
    out = f("out")
    state = f("state")
    for b, h in pairs:
        g = h // rep
        sl = lambda t, hh: t[b:b + 1, :, hh:hh + 1].to(torch.float64).cpu().numpy()
        q, k, v = sl(f("q"), g), sl(f("k"), g), sl(f("v"), h)
        al, be = sl(f("alpha"), h), sl(f("beta"), h)
        row = case.state_row[b:b + 1]
        S0 = L.state[:, h:h + 1]
        o_ref, _, _ = O.scan(case.parent[b:b + 1], case.slot[b:b + 1], row, q, k, v, al, be, S0, l2norm=True, threads=4)
        assert_close(out[b, :, h].to(torch.float64).cpu().numpy(), o_ref[0, :, 0], bf16=True,
                     what=f"{case.name} layer {layer} b={b} h={h} outputs")
        st_ref, _, status, _ = O.commit(case.parent[b:b + 1], case.slot[b:b + 1], row, q, k, v, al, be, S0,
                                        case.accepted[b:b + 1], case.accepted_len[b:b + 1], l2norm=True, threads=4)
        assert status[0] == 0
        assert_close(state[row[0], h].to(torch.float64).cpu().numpy(), st_ref[row[0], 0],
                     what=f"{case.name} layer {layer} b={b} h={h} committed state")


@pytest.mark.parametrize("shape", ["chains", "star", "random"])
def test_config4_full_size_sampled(shape):
    case = W.config4(shape)                       # batch 32, 256 nodes, 16/32 heads
    dc = DeviceCase(ctx("auto"), case, out_dtype="bf16")
    dc.verify()
    dc.commit()
    torch.cuda.synchronize()
    assert dc.np("status").tolist() == [0] * case.B
    rs = np.random.default_rng(4)
    pairs = [(int(rs.integers(case.B)), int(rs.integers(case.Hv))) for _ in range(5)] + [(0, 0), (case.B - 1, case.Hv - 1)]
    check_samples(dc, case, 0, pairs)
    check_conv_samples(dc, case, 0, sorted({b for b, _ in pairs})[:4])
    # properties that hold at any size: finite everywhere, rows of the pool that belong to nobody untouched
    assert torch.isfinite(dc.t("out").float()).all()
    other = sorted(set(range(case.rows)) - set(case.state_row.tolist()))
    assert torch.equal(dc.t("state")[other].cpu(), torch.from_numpy(case.layers[0].state[other]))


def test_config3_full_stack_sampled():
    case = W.config3()                            # 48 layers, batch 4, 32 nodes
    dc = DeviceCase(ctx("auto"), case, out_dtype="bf16")
    dc.verify()
    dc.commit()
    torch.cuda.synchronize()
    rs = np.random.default_rng(3)
    for layer in (0, 23, 47):
        assert dc.np("status", layer).tolist() == [0] * case.B
        pairs = [(int(rs.integers(case.B)), int(rs.integers(case.Hv))) for _ in range(4)]
        check_samples(dc, case, layer, pairs)
        check_conv_samples(dc, case, layer, sorted({b for b, _ in pairs})[:2])
    for layer in range(48):
        assert torch.isfinite(dc.t("out", layer).float()).all()


def test_config3_fused_commit_verify_matches_the_separate_calls():
    """48 layers in the launch configuration bench.py times: lumo_gdn_commit_verify against
    lumo_gdn_commit followed by lumo_gdn_tree_verify, every layer, state and outputs."""
    from paper_2609_23900_b200 import binding
    from tests.test_gpu_fused import _share_state
    P, C = W.config3(seed=W.BASE_SEED + 303), W.config3()
    C.state_row = P.state_row.copy()
    for LP, LC in zip(P.layers, C.layers):
        LC.state = LP.state.copy()
        LC.hist = LP.hist.copy()
    c = ctx()
    results = []
    for fused in (True, False):
        dcP, dcC = DeviceCase(c, P, out_dtype="bf16"), DeviceCase(c, C, out_dtype="bf16")
        dcP.verify()
        layersC = _share_state(dcP, dcC)
        if fused:
            c.commit_verify(dcP.desc, dcP.layers, dcP.accepted, dcP.accepted_len, dcC.desc, layersC)
        else:
            dcP.commit()
            c.verify(dcC.desc, layersC)
        torch.cuda.synchronize()
        results.append((dcP, layersC))
    (pf, lf), (pu, lu) = results
    for l in range(len(C.layers)):
        sf, su = pf.t("state", l), pu.t("state", l)
        assert torch.isfinite(sf).all()
        assert (sf - su).abs().max().item() <= 1e-5 * max(1.0, su.abs().max().item())
        assert torch.equal(pf.t("conv_hist", l), pu.t("conv_hist", l))
        assert torch.equal(pf.t("status", l), pu.t("status", l))
        of, ou = lf[l].tensors["out"].float(), lu[l].tensors["out"].float()
        assert bool(((of - ou).abs() <= 2.0 ** -7 * ou.abs() + 1e-3).all())   # bf16 outputs: one ulp apart at most
        assert torch.equal(lf[l].tensors["k"], lu[l].tensors["k"]) and torch.equal(lf[l].tensors["v"], lu[l].tensors["v"])


def test_attention_at_the_bench_shape_sampled():
    """The attention launch bench.py times (batch 8, 32/8 heads, 16k-token contexts, paper tree, spine-first
    slots, automatic decomposition over all SMs): inputs drawn on the device by a seeded generator, the
    oracle run on sampled (sequence, query head) pairs from copies of those inputs, every node of the pair."""
    from oracle import attn_oracle as A
    from paper_2609_23900_b200 import binding
    c = ctx()
    dev = torch.device("cuda", c.device)
    B, context, Hq, Hkv, dh = 8, 16384, 32, 8, 128
    tree = W.tree_paper_geometry()
    N, Ns = len(tree), 32
    parent = np.asarray([tree] * B, dtype=np.int32)
    slot = np.asarray([W.spine_first_slots(tree)] * B, dtype=np.int32)
    desc = c.tree_desc(parent, slot=slot, n_slots=Ns)
    S = context + Ns
    ctx_host = np.asarray([context - 37 * b for b in range(B)], dtype=np.int32)        # ragged tile edges
    ctx_len = torch.from_numpy(ctx_host).to(dev)
    rows = torch.arange(B - 1, -1, -1, dtype=torch.int32, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(99)
    rnd = lambda *shape: torch.randn(*shape, device=dev, dtype=torch.float32, generator=gen).to(torch.bfloat16)
    L = binding.AttnLayer(Hq=Hq, Hkv=Hkv, k_cache=rnd(B, S, Hkv, dh), v_cache=rnd(B, S, Hkv, dh), ctx_len=ctx_len, cache_row=rows,
                          scale=dh ** -0.5, q=rnd(B, N, Hq, dh), k_new=rnd(B, N, Hkv, dh), v_new=rnd(B, N, Hkv, dh),
                          out=torch.empty(B, N, Hq, dh, device=dev), lse=torch.empty(B, N, Hq, device=dev),
                          status=torch.full((B,), -1, dtype=torch.int32, device=dev))
    pk = c.pack_attn([L])
    k0 = {b: L.tensors["k_cache"][int(rows[b])].to(torch.float64).cpu().numpy() for b in (0, 3, 7)}     # before the write
    v0 = {b: L.tensors["v_cache"][int(rows[b])].to(torch.float64).cpu().numpy() for b in (0, 3, 7)}
    c.kv_write_tree(desc, pk)
    c.tree_attention(desc, pk)
    torch.cuda.synchronize()
    assert L.tensors["status"].tolist() == [0] * B
    out, lse = L.tensors["out"].to(torch.float64).cpu().numpy(), L.tensors["lse"].to(torch.float64).cpu().numpy()
    q = L.tensors["q"].to(torch.float64).cpu().numpy()
    kn, vn = L.tensors["k_new"].to(torch.float64).cpu().numpy(), L.tensors["v_new"].to(torch.float64).cpu().numpy()
    worst = 0.0
    for b in (0, 3, 7):
        one = lambda a: a[b:b + 1]
        k1, v1 = A.kv_write(one(slot), one(kn), one(vn), k0[b][None], v0[b][None], ctx_host[b:b + 1], np.zeros(1, np.int32))
        for h in (0, 13, 31):
            g = h // (Hq // Hkv)
            qq = q[b:b + 1, :, h:h + 1]
            kk, vv = k1[:, :, g:g + 1], v1[:, :, g:g + 1]
            ref, rl = A.tree_attention(one(parent), one(slot), qq, kk, vv, ctx_host[b:b + 1], np.zeros(1, np.int32), dh ** -0.5)
            bound, _ = A.tree_attention(one(parent), one(slot), qq, kk, np.abs(vv), ctx_host[b:b + 1], np.zeros(1, np.int32), dh ** -0.5)
            err = np.abs(out[b, :, h] - ref[0, :, 0])
            tol = 1.05 * 2.0 ** -8 * bound[0, :, 0] + 2e-5 * (1.0 + np.abs(ref[0, :, 0]))
            assert (err <= tol).all(), f"b={b} h={h}: worst ratio {(err / tol).max():.2f}"
            assert (np.abs(lse[b, :, h] - rl[0, :, 0]) <= 2e-5 * (1.0 + np.abs(rl[0, :, 0]))).all(), f"b={b} h={h}: lse"
            worst = max(worst, float((err / tol).max()))
    assert worst > 0.0
