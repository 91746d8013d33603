"""Device-resident acceptance walk (lumo_tree_accept) against its oracle: accepted path, length,
pending token and final node must match bit for bit, in greedy and in rejection-sampling mode; and the
walk's device outputs must drive lumo_gdn_commit with no host round trip."""
import numpy as np
import pytest
import torch

from oracle import accept_oracle as A
from oracle import gdn_oracle as O
from synthetic import workload as W
from synthetic.device_case import DeviceCase
from tests.harness import assert_close, ctx

pytestmark = pytest.mark.gpu


def make_inputs(parents, slot, Ns, V, seed, agree=0.6):
    """Synthetic target/proposal rows: the proposal of a node is a perturbed copy of its parent's
    target row, so that a fair share of candidates is accepted."""
    rs = np.random.default_rng(seed)
    B, N = parents.shape
    p = rs.dirichlet(np.full(V, 0.05), size=(B, Ns + 1)).astype(np.float32)
    q = rs.dirichlet(np.full(V, 0.05), size=(B, Ns)).astype(np.float32)
    token = rs.integers(0, V, size=(B, Ns)).astype(np.int32)
    for b in range(B):
        for i in range(N):
            prow = Ns if parents[b, i] < 0 else slot[b, parents[b, i]]
            mix = (agree * p[b, prow] + (1 - agree) * q[b, slot[b, i]]).astype(np.float32)
            q[b, slot[b, i]] = mix / mix.sum(dtype=np.float32)
            token[b, slot[b, i]] = rs.choice(V, p=q[b, slot[b, i]].astype(np.float64) / q[b, slot[b, i]].astype(np.float64).sum())
            if rs.uniform() < 0.5:   # some candidates are the target's favourite: greedy accepts them
                token[b, slot[b, i]] = int(np.argmax(p[b, prow]))
    u = rs.uniform(size=(B, Ns)).astype(np.float32)
    noise = rs.exponential(size=(B, V)).astype(np.float32) + np.float32(1e-6)
    return token, p, q, u, noise


def run_device(desc, Ns, token, p, q, u, noise, mode, lmax):
    dev = torch.device("cuda", 0)
    B, V = p.shape[0], p.shape[-1]
    up = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    acc = torch.full((B, lmax), 99, dtype=torch.int32, device=dev)
    ln, nxt, fin = (torch.full((B,), 99, dtype=torch.int32, device=dev) for _ in range(3))
    work = torch.empty((B, V), dtype=torch.float32, device=dev)
    ctx().accept(desc, token=up(token), p_target=up(p), q_draft=up(q), uniforms=up(u), noise=up(noise), work=work,
                 accepted=acc, length=ln, next_token=nxt, final_node=fin, mode=mode)
    return acc, ln, nxt, fin


@pytest.mark.parametrize("mode", ["greedy", "rejection"])
@pytest.mark.parametrize("shape", ["tiny", "cfg2", "paper", "star", "chains"])
def test_accept_matches_oracle_bit_exactly(mode, shape):
    if shape == "tiny":
        c, V = W.make_case("t", [W.tree_tiny()] * 3, seed=1, Hk=1, Hv=1, d=64, in_dtype="f32"), 37
    elif shape == "cfg2":
        c, V = W.config2(B=4), 4099
    elif shape == "paper":
        c, V = W.config_paper(B=3), 32000
    elif shape == "chains":  # the largest tree; a vocabulary that does not divide over the cluster
        c, V = W.make_case("w", [W.tree_chains(32, 8)] * 2, seed=3, Hk=1, Hv=1, d=64, in_dtype="f32"), 8191
    else:
        c, V = W.make_case("s", [W.tree_star(40)] * 2, seed=2, Hk=1, Hv=1, d=64, in_dtype="f32", Ns=48, permute_slots=True), 1000
    token, p, q, u, noise = make_inputs(c.parent, c.slot, c.Ns, V, seed={"tiny": 11, "cfg2": 12, "paper": 13, "star": 14, "chains": 15}[shape])
    lmax = max(max(W.tree_depths(pp.tolist())) for pp in c.parent) + 1
    desc = ctx().tree_desc(c.parent, slot=c.slot, n_slots=c.Ns)
    acc, ln, nxt, fin = run_device(desc, c.Ns, token, p, q, u, noise, mode, lmax)
    torch.cuda.synchronize()
    ref = A.accept(c.parent, c.slot, c.Ns, token, p, q, u, noise, mode=A.GREEDY if mode == "greedy" else A.REJECTION, lmax=lmax)
    assert acc.cpu().numpy().tolist() == ref[0].tolist()
    assert ln.cpu().numpy().tolist() == ref[1].tolist()
    assert nxt.cpu().numpy().tolist() == ref[2].tolist()
    assert fin.cpu().numpy().tolist() == ref[3].tolist()
    assert (ref[1] > 0).any()            # the inputs do exercise acceptance


def test_verify_accept_commit_without_host_round_trip():
    c = W.config2(B=4)
    V = 2048
    token, p, q, u, noise = make_inputs(c.parent, c.slot, c.Ns, V, seed=5)
    lmax = 9
    dc = DeviceCase(ctx("auto"), c)
    dc.verify()
    acc, ln, nxt, fin = run_device(dc.desc, c.Ns, token, p, q, u, noise, "rejection", lmax)
    dc.commit(acc, ln)                   # consumes the device products directly
    torch.cuda.synchronize()
    ref = A.accept(c.parent, c.slot, c.Ns, token, p, q, u, noise, mode=A.REJECTION, lmax=lmax)
    assert acc.cpu().numpy().tolist() == ref[0].tolist() and dc.np("status").tolist() == [0] * c.B
    L = c.layers[0]
    st_ref, hist_ref, _, _ = O.commit(c.parent, c.slot, c.state_row, dc.np("q"), dc.np("k"), dc.np("v"), dc.np("alpha"),
                                      dc.np("beta"), L.state, ref[0], ref[1], l2norm=True, x=L.x, hist=L.hist)
    assert_close(dc.np("state"), st_ref, what="state committed along the device-selected path")
    assert np.array_equal(dc.np("conv_hist"), hist_ref)


@pytest.mark.parametrize("V", [4096, 4099, 151936])
def test_greedy_ties_take_the_lowest_token_on_every_load_path(V):
    """Target rows whose maximum occurs several times, spread over the slices of the cluster and over
    the ragged ends of the 16-byte body: the pending token must be the lowest such index."""
    c = W.make_case("t", [W.tree_tiny()] * 3, seed=1, Hk=1, Hv=1, d=64, in_dtype="f32")
    rs = np.random.default_rng(V)
    p = rs.uniform(0.0, 0.5, size=(c.B, c.Ns + 1, V)).astype(np.float32)
    for b in range(c.B):
        for r in range(c.Ns + 1):
            pos = rs.choice(V, size=5, replace=False)
            if r % 3 == 0:
                pos = np.concatenate([pos, [1, V - 1, V - 2]])      # ragged ends
            p[b, r, pos] = 0.75
    token = rs.integers(0, V, size=(c.B, c.Ns)).astype(np.int32)
    for b in range(c.B):                                            # let the walk take a few steps
        for i in range(c.N):
            prow = c.Ns if c.parent[b, i] < 0 else c.slot[b, c.parent[b, i]]
            token[b, c.slot[b, i]] = int(np.flatnonzero(p[b, prow] == p[b, prow].max())[0]) if i % 2 == 0 else token[b, c.slot[b, i]]
    lmax = max(W.tree_depths(c.parent[0].tolist())) + 1
    desc = ctx().tree_desc(c.parent, slot=c.slot, n_slots=c.Ns)
    q = np.zeros((c.B, c.Ns, 1), np.float32)
    acc, ln, nxt, fin = run_device(desc, c.Ns, token, p, q, np.zeros((c.B, c.Ns), np.float32), np.ones((c.B, V), np.float32), "greedy", lmax)
    torch.cuda.synchronize()
    ref = A.accept(c.parent, c.slot, c.Ns, token, p, None, None, None, mode=A.GREEDY, lmax=lmax)
    assert acc.cpu().numpy().tolist() == ref[0].tolist() and ln.cpu().numpy().tolist() == ref[1].tolist()
    assert nxt.cpu().numpy().tolist() == ref[2].tolist() and fin.cpu().numpy().tolist() == ref[3].tolist()
    assert (ref[1] > 0).any()
