"""lumo_gdn_commit_verify: the previous cycle's commit folded into this cycle's verify must equal the
two separate steps: committed state, history, statuses and the new tree's outputs against the oracle
(commit oracle, then conv and scan oracles from the committed state), and against the unfused calls."""
import numpy as np
import pytest
import torch

from oracle import gdn_oracle as O
from paper_2609_23900_b200 import binding
from synthetic import workload as W
from synthetic.device_case import DeviceCase
from tests.harness import assert_close, ctx

pytestmark = pytest.mark.gpu


def _cycles(kind):
    """Previous and current cycle over the same sequences: same heads and state pool, different trees."""
    if kind == "cfg2":
        P, C = W.config2(B=4), W.config2(B=4, seed=W.BASE_SEED + 77)
    elif kind == "two_layers":
        P, C = W.config2(B=3, n_layers=2), W.config2(B=3, n_layers=2, seed=W.BASE_SEED + 78)
    elif kind == "paper_then_cfg3":     # padded permuted 28-of-32 tree, then 32-node trees (32-node MMA tile)
        P, C = W.config_paper(B=4), W.config3(B=4, n_layers=1)
    else:                               # 256-node trees: several groups per sequence, served by the two separate calls
        P, C = W.config2(B=2), W.make_case("big", [W.tree_star(200)] * 2, seed=9, Hk=16, Hv=32, d=128, in_dtype="bf16")
    C.state_row = P.state_row.copy()
    C.rows = P.rows
    for LP, LC in zip(P.layers, C.layers):
        LC.state = LP.state.copy()
        LC.hist = LP.hist.copy()
    return P, C


def _share_state(dcP, dcC):
    """Layers of the current cycle that name the previous cycle's state, history and row tensors."""
    c = dcC.case
    out = []
    for l, layer in enumerate(dcC.layers):
        t = dict(layer.tensors)
        t.update(state=dcP.t("state", l), conv_hist=dcP.t("conv_hist", l), state_row=dcP.state_row)
        out.append(binding.GdnLayer(Hk=c.Hk, Hv=c.Hv, d=c.d, scale=dcC.scale, qk_l2norm=dcC.qk_l2norm, l2_eps=dcC.l2_eps, **t))
    return out


def _bf16(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).to(torch.float64).numpy()


def _oracle(P, C, dcP, layersC, l, accepted, length):
    """commit(P) then conv + scan(C) in fp64, on the operands the GPU recorded."""
    LP, LC = P.layers[l], C.layers[l]
    f = lambda t: t.to(torch.float64).cpu().numpy()
    st1, hist1, status, _ = O.commit(P.parent, P.slot, P.state_row, dcP.np("q", l), dcP.np("k", l), dcP.np("v", l),
                                     LP.alpha, LP.beta, LP.state, accepted, length, x=LP.x, hist=LP.hist,
                                     l2norm=dcP.qk_l2norm, eps=dcP.l2_eps)
    # unrounded fp64 result: the recorded operands are compared with it element by element under the
    # quantised-output rule (1e-3 (1 + |ref|) plus half a bf16 ulp)
    y = O.conv(C.parent, C.slot, C.state_row, LC.x, LC.conv_w, LC.conv_b, hist1, C.Ns, out_dtype="none")
    tc = layersC[l].tensors
    o_ref, _, _ = O.scan(C.parent, C.slot, C.state_row, f(tc["q"]), f(tc["k"]), f(tc["v"]), LC.alpha, LC.beta, st1,
                         l2norm=True, eps=1e-6)
    return st1, hist1, status, y, o_ref


@pytest.fixture(params=["auto", "solve", "direct", "tensor"])
def algo(request):
    """Both tensor-core scans have a fused variant; every fused test runs on each."""
    yield request.param
    ctx("auto")


@pytest.mark.parametrize("kind", ["cfg2", "two_layers", "paper_then_cfg3", "fallback_many_groups"])
def test_commit_verify_equals_commit_then_verify(kind, algo):
    P, C = _cycles(kind)
    c = ctx(algo)
    dcP, dcC = DeviceCase(c, P), DeviceCase(c, C)
    dcP.verify()                                    # records the previous cycle's operands
    layersC = _share_state(dcP, dcC)
    c.commit_verify(dcP.desc, dcP.layers, dcP.accepted, dcP.accepted_len, dcC.desc, layersC)
    torch.cuda.synchronize()
    hk = C.Hk * C.d
    for l in range(len(C.layers)):
        st1, hist1, status, y, o_ref = _oracle(P, C, dcP, layersC, l, P.accepted, P.accepted_len)
        assert_close(dcP.np("state", l), st1, what=f"{kind} committed state, layer {l}")
        assert np.array_equal(dcP.np("conv_hist", l), hist1), "history"
        assert dcP.t("status", l).cpu().numpy().tolist() == status.tolist()
        f = lambda t: t.to(torch.float64).cpu().numpy()
        tc = layersC[l].tensors
        got = np.concatenate([f(tc["q"]).reshape(C.B, C.Ns, hk), f(tc["k"]).reshape(C.B, C.Ns, hk),
                              f(tc["v"]).reshape(C.B, C.Ns, C.Hv * C.d)], axis=-1)
        assert_close(got, y, bf16=True, what=f"{kind} recorded operands of the new tree (conv over the committed history), layer {l}")
        assert (got == _bf16(y)).mean() > 0.98      # and nearly all are the oracle's own rounding
        assert_close(f(tc["out"]), o_ref, what=f"{kind} outputs of the new tree, layer {l}")
        assert tc["status"].cpu().numpy().tolist() == [0] * C.B
    # against the two separate calls on fresh copies
    dcP2, dcC2 = DeviceCase(c, P), DeviceCase(c, C)
    dcP2.verify()
    layersC2 = _share_state(dcP2, dcC2)
    dcP2.commit()
    c.verify(dcC2.desc, layersC2)
    torch.cuda.synchronize()
    for l in range(len(C.layers)):
        a, b = dcP.np("state", l), dcP2.np("state", l)
        assert np.abs(a - b).max() <= 1e-5 * max(1.0, np.abs(b).max())
        assert torch.equal(dcP.t("conv_hist", l), dcP2.t("conv_hist", l))
        o1 = layersC[l].tensors["out"].to(torch.float64).cpu().numpy()
        o2 = layersC2[l].tensors["out"].to(torch.float64).cpu().numpy()
        assert np.abs(o1 - o2).max() <= 1e-4 * (1.0 + np.abs(o2).max())


def test_commit_verify_rejects_a_bad_path_and_skips_empty_ones(algo):
    P, C = _cycles("cfg2")
    acc, ln = P.accepted.copy(), P.accepted_len.copy()
    ln[1] = 0                                       # nothing accepted: state stays
    depth = W.tree_depths(P.parent[2].tolist())
    root = int(np.flatnonzero(P.parent[2] < 0)[0])
    acc[2, :2] = [root, next(i for i in range(P.N) if depth[i] == 3)]   # second entry is no child of the first
    ln[2] = 2
    c = ctx(algo)
    dcP, dcC = DeviceCase(c, P), DeviceCase(c, C)
    dcP.verify()
    layersC = _share_state(dcP, dcC)
    dev = dcP.accepted.device
    c.commit_verify(dcP.desc, dcP.layers, torch.from_numpy(acc).to(dev), torch.from_numpy(ln).to(dev), dcC.desc, layersC)
    torch.cuda.synchronize()
    st1, hist1, status, y, o_ref = _oracle(P, C, dcP, layersC, 0, acc, ln)
    assert status[2] != 0 and status[1] == 0
    assert dcP.t("status").cpu().numpy().tolist() == status.tolist()
    assert_close(dcP.np("state"), st1, what="state")
    row1, row2 = P.state_row[1], P.state_row[2]
    assert np.array_equal(dcP.np("state")[row1], P.layers[0].state[row1])      # bitwise untouched
    assert np.array_equal(dcP.np("state")[row2], P.layers[0].state[row2])
    assert np.array_equal(dcP.np("conv_hist"), hist1)
    assert_close(layersC[0].tensors["out"].to(torch.float64).cpu().numpy(), o_ref, what="outputs")


def test_commit_verify_every_mix_of_old_and_accepted_history_rows(algo):
    """Accepted lengths 0, 1, 2, 3, 4 and 5 in one batch: the three history rows the new tree's
    convolution reads are then 3, 2, 1 and 0 old rows followed by 0, 1, 2 and 3 accepted inputs.  The
    recorded operands (every row, depth-1 rows read all three history taps), the committed state and
    history and the outputs are compared with the composed oracles."""
    chain = W.tree_chain(6)
    parents = [chain + [0, 0, 1, 2, 3, 1, 6, 7, 7, 9] for _ in range(6)]      # 16 nodes, spine 0..5 plus branches
    P = W.make_case("hp", parents, seed=41, Hk=4, Hv=8, d=128, in_dtype="bf16", with_bias=True,
                    accepted=[list(range(n)) for n in range(6)], lmax=6)
    C = W.make_case("hc", [W.tree_random(W.IntStream(W.stream_key(43, b)), 24, 4) for b in range(6)], seed=42, Hk=4, Hv=8,
                    d=128, in_dtype="bf16", with_bias=True, Ns=29, permute_slots=True)
    assert P.accepted_len.tolist() == [0, 1, 2, 3, 4, 5]
    C.state_row, C.rows = P.state_row.copy(), P.rows
    C.layers[0].state, C.layers[0].hist = P.layers[0].state.copy(), P.layers[0].hist.copy()
    c = ctx(algo)
    dcP, dcC = DeviceCase(c, P), DeviceCase(c, C)
    dcP.verify()
    layersC = _share_state(dcP, dcC)
    c.commit_verify(dcP.desc, dcP.layers, dcP.accepted, dcP.accepted_len, dcC.desc, layersC)
    torch.cuda.synchronize()
    st1, hist1, status, y, o_ref = _oracle(P, C, dcP, layersC, 0, P.accepted, P.accepted_len)
    assert status.tolist() == [0] * 6 and dcP.t("status").cpu().numpy().tolist() == [0] * 6
    f = lambda t: t.to(torch.float64).cpu().numpy()
    tc = layersC[0].tensors
    hk = C.Hk * C.d
    got = np.concatenate([f(tc["q"]).reshape(C.B, C.Ns, hk), f(tc["k"]).reshape(C.B, C.Ns, hk),
                          f(tc["v"]).reshape(C.B, C.Ns, C.Hv * C.d)], axis=-1)
    for b in range(6):
        assert_close(got[b], y[b], bf16=True, what=f"accepted length {b}: recorded operands")
    # the history rows really differ between the lengths (a conv that ignored the path would fail above)
    assert not np.array_equal(hist1[P.state_row[1]], P.layers[0].hist[P.state_row[1]])
    assert np.array_equal(hist1[P.state_row[0]], P.layers[0].hist[P.state_row[0]])
    assert np.array_equal(dcP.np("conv_hist"), hist1)
    assert_close(dcP.np("state"), st1, what="committed state")
    assert_close(f(tc["out"]), o_ref, what="outputs of the new tree")


def test_commit_verify_argument_checks():
    P, C = _cycles("cfg2")
    c = ctx()
    dcP, dcC = DeviceCase(c, P), DeviceCase(c, C)
    with pytest.raises(binding.LumoError) as e:     # the two cycles name different state tensors
        c.commit_verify(dcP.desc, dcP.layers, dcP.accepted, dcP.accepted_len, dcC.desc, dcC.layers)
    assert e.value.code == 1
    with pytest.raises(binding.LumoError) as e:     # the previous operands must not be the new ones
        c.commit_verify(dcP.desc, dcP.layers, dcP.accepted, dcP.accepted_len, dcP.desc, dcP.layers)
    assert e.value.code == 1


def test_commit_verify_scan_only_cycle_updates_history_with_the_commit_kernel(algo):
    """The new cycle has no convolution (operands given): the history of the accepted path is then
    gathered by the commit kernel's history CTAs ahead of the fused scan."""
    P, C = _cycles("cfg2")
    c = ctx(algo)
    dcP, dcC = DeviceCase(c, P), DeviceCase(c, C, use_conv=False, qk_l2norm=True)
    dcP.verify()
    layersC = []
    for l, layer in enumerate(dcC.layers):
        t = dict(layer.tensors)
        t.update(state=dcP.t("state", l), state_row=dcP.state_row, conv_hist=dcP.t("conv_hist", l))
        layersC.append(binding.GdnLayer(Hk=C.Hk, Hv=C.Hv, d=C.d, scale=dcC.scale, qk_l2norm=True, l2_eps=dcC.l2_eps, **t))
    c.commit_verify(dcP.desc, dcP.layers, dcP.accepted, dcP.accepted_len, dcC.desc, layersC)
    torch.cuda.synchronize()
    LP, LC = P.layers[0], C.layers[0]
    st1, hist1, status, _ = O.commit(P.parent, P.slot, P.state_row, dcP.np("q"), dcP.np("k"), dcP.np("v"), LP.alpha, LP.beta,
                                     LP.state, P.accepted, P.accepted_len, x=LP.x, hist=LP.hist, l2norm=True, eps=dcP.l2_eps)
    f = lambda t: t.to(torch.float64).cpu().numpy()
    tc = layersC[0].tensors
    o_ref, _, _ = O.scan(C.parent, C.slot, C.state_row, f(tc["q"]), f(tc["k"]), f(tc["v"]), LC.alpha, LC.beta, st1,
                         l2norm=True, eps=dcC.l2_eps)
    assert_close(dcP.np("state"), st1, what="state")
    assert np.array_equal(dcP.np("conv_hist"), hist1)
    assert_close(f(tc["out"]), o_ref, what="outputs")


def test_commit_after_commit_verify_sees_the_rewritten_state(algo):
    """A plain commit right after a fused call (the last cycle of a generation) under kernel overlap:
    it must start from the state the fused scan wrote, cycle after cycle, bitwise as without overlap."""
    P, C = _cycles("cfg2")
    res = {}
    for on in (False, True):
        c = ctx(algo)
        c.set_overlap(on)
        dcP, dcC = DeviceCase(c, P), DeviceCase(c, C)
        dcP.verify()
        layersC = _share_state(dcP, dcC)
        for _ in range(3):
            c.commit_verify(dcP.desc, dcP.layers, dcP.accepted, dcP.accepted_len, dcC.desc, layersC)
            c.commit(dcC.desc, layersC, dcC.accepted, dcC.accepted_len)
        torch.cuda.synchronize()
        res[on] = (dcP.t("state").clone(), dcP.t("conv_hist").clone(), layersC[0].tensors["out"].clone())
    ctx().set_overlap(True)
    for a, b in zip(res[False], res[True]):
        assert torch.equal(a, b)


def test_commit_verify_randomized_sweep():
    """Seeded sweep: tree sizes around the tile sizes, depths up to 16, padded and permuted slots, bias,
    head ratios 1..3, empty and invalid accepted paths; state, history, status, recorded operands and
    outputs against the composed oracles."""
    import random
    rng = random.Random(2024)

    def rand_tree(N, maxd):
        p, d = [], []
        for i in range(N):
            while True:
                q = rng.randint(-1, i - 1)
                dq = 0 if q < 0 else d[q]
                if dq < maxd:
                    break
            p.append(q)
            d.append(dq + 1)
        return p

    c = ctx()
    worst = 0.0
    for it in range(24):
        B = rng.choice([1, 2, 3])
        Hk = rng.choice([1, 2])
        Hv = Hk * rng.choice([1, 2, 3])
        bias = rng.random() < 0.3
        cases = []
        for _ in range(2):
            N = rng.choice([1, 2, 3, 17, 31, 32, 33, 63, 64])
            parents = [rand_tree(N, rng.choice([2, 5, 9, 16])) for _ in range(B)]
            Ns = N + rng.choice([0, 0, 7])
            cases.append(W.make_case("f", parents, seed=rng.getrandbits(30), Hk=Hk, Hv=Hv, d=128, in_dtype="bf16", Ns=Ns,
                                     permute_slots=Ns > N or rng.random() < 0.5, alpha_lo=rng.choice([0.5, 0.9]),
                                     beta_uniform=rng.random() < 0.5, with_bias=bias))
        P, C = cases
        C.state_row, C.rows = P.state_row.copy(), P.rows
        C.layers[0].state, C.layers[0].hist = P.layers[0].state.copy(), P.layers[0].hist.copy()
        acc, ln = P.accepted.copy(), P.accepted_len.copy()
        if rng.random() < 0.3:
            ln[rng.randrange(B)] = 0
        if rng.random() < 0.25 and P.N > 2:
            acc[rng.randrange(B), 0] = P.N - 1            # (mostly) not a child of the pre-tree state
        dcP, dcC = DeviceCase(c, P), DeviceCase(c, C)
        dcP.verify()
        layersC = _share_state(dcP, dcC)
        dev = dcP.accepted.device
        c.commit_verify(dcP.desc, dcP.layers, torch.from_numpy(acc).to(dev), torch.from_numpy(ln).to(dev), dcC.desc, layersC)
        torch.cuda.synchronize()
        st1, hist1, status, y, o_ref = _oracle(P, C, dcP, layersC, 0, acc, ln)
        f = lambda t: t.to(torch.float64).cpu().numpy()
        tc = layersC[0].tensors
        hk = C.Hk * C.d
        got = np.concatenate([f(tc["q"]).reshape(C.B, C.Ns, hk), f(tc["k"]).reshape(C.B, C.Ns, hk),
                              f(tc["v"]).reshape(C.B, C.Ns, C.Hv * C.d)], axis=-1)
        what = f"case {it}: nodes {P.N} -> {C.N}, batch {B}, heads {Hk}/{Hv}, lengths {ln.tolist()}"
        worst = max(worst, assert_close(dcP.np("state"), st1, what=what + " state"),
                    assert_close(f(tc["out"]), o_ref, what=what + " outputs"))
        assert np.array_equal(dcP.np("conv_hist"), hist1), what
        assert dcP.t("status").cpu().numpy().tolist() == status.tolist(), what
        assert_close(got, y, bf16=True, what=what + " recorded operands")
        assert (got == _bf16(y)).mean() > 0.98, what
    assert worst < 1e-4
