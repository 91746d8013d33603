"""Pins for the fp64 oracle's tree scan and commit (oracle/gdn_oracle.cpp).

Each test checks the oracle against something fixed by the paper's Eq. 2-3 or by
mathematics, computed by another route: closed forms, invariants, a library
triangular solve of the ancestor-masked system, a library linear solve, products of
explicit transition matrices.  None of them re-types the oracle's loop.
"""
import numpy as np
import pytest
import scipy.linalg

from oracle import gdn_oracle as O
from oracle import tree_tables as T
from synthetic import workload as W

TINY = [-1, -1, 0, 0, 1, 1, 2]


def small_case(parents, seed=7, d=16, Hk=1, Hv=2, Ns=None, permute=False, **kw):
    return W.make_case("t", parents, seed=seed, Hk=Hk, Hv=Hv, d=d, in_dtype="f32", Ns=Ns,
                       permute_slots=permute, **kw)


def run_scan(c, L=None, **kw):
    L = L or c.layers[0]
    return O.scan(c.parent, c.slot, c.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state, **kw)


def all_nodes(c):
    return np.tile(np.arange(c.N, dtype=np.int32), (c.B, 1))


def rand_parents(seed, n, B=1):
    rs = np.random.default_rng(seed)
    return [[int(rs.integers(-1, i)) for i in range(n)] for _ in range(B)]


# ---------------------------------------------------------------- the sequential recurrence
def test_chain_tree_equals_the_sequential_gated_delta_rule():
    """A chain-shaped tree is an ordinary token sequence: the oracle must reproduce the sequential gated
    delta rule in its matrix form S_t = alpha_t S_{t-1} (I - beta_t k_t k_t^T) + beta_t v_t k_t^T,
    o_t = S_t q_t (Eq. 2-3 multiplied out), written here with library matrix products only."""
    n, d = 9, 16
    c = small_case([W.tree_chain(n)] * 2, seed=21, d=d, Hk=2, Hv=4, Ns=n + 3, permute=True)
    L = c.layers[0]
    o, snap, _ = run_scan(c, snap_nodes=all_nodes(c), mode="walk")
    I = np.eye(d)
    for b in range(c.B):
        for h in range(c.Hv):
            g = h // (c.Hv // c.Hk)
            S = L.state[c.state_row[b], h].astype(np.float64)
            for t in range(n):
                r = c.slot[b, t]
                k, q, v = (a.astype(np.float64) for a in (L.k[b, r, g], L.q[b, r, g], L.v[b, r, h]))
                a_t, b_t = float(L.alpha[b, r, h]), float(L.beta[b, r, h])
                S = a_t * S @ (I - b_t * np.outer(k, k)) + b_t * np.outer(v, k)
                np.testing.assert_allclose(snap[b, t, h], S, rtol=1e-12, atol=1e-15)
                np.testing.assert_allclose(o[b, r, h], S @ q, rtol=1e-11, atol=1e-15)


# ---------------------------------------------------------------- closed forms
def test_beta_zero_is_pure_decay():
    c = small_case(rand_parents(1, 12, B=2))
    L = c.layers[0]
    L.beta[:] = 0.0
    o, snap, _ = run_scan(c, snap_nodes=all_nodes(c), mode="walk")
    for b in range(c.B):
        S0 = L.state[c.state_row[b]].astype(np.float64)
        for i in range(c.N):
            g = np.prod([float(L.alpha[b, c.slot[b, t], 0]) for t in T.ancestry(c.parent[b].tolist(), i)])
            np.testing.assert_allclose(snap[b, i, 0], g * S0[0], rtol=1e-14, atol=0)
            np.testing.assert_allclose(o[b, c.slot[b, i], 0], g * (S0[0] @ L.q[b, c.slot[b, i], 0].astype(np.float64)),
                                       rtol=1e-12, atol=1e-16)


def test_alpha_one_beta_zero_leaves_state_bitwise_unchanged():
    c = small_case(rand_parents(2, 10))
    L = c.layers[0]
    L.alpha[:] = 1.0
    L.beta[:] = 0.0
    _, snap, _ = run_scan(c, snap_nodes=all_nodes(c))
    S0 = L.state[c.state_row[0]].astype(np.float64)
    for i in range(c.N):
        assert np.array_equal(snap[0, i], S0)
    acc, ln, _ = T.path_from_node(c.parent[0].tolist(), c.N - 1, c.N)
    st, _, status, _ = O.commit(c.parent, c.slot, c.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state,
                                [acc], [ln])
    assert status[0] == 0 and np.array_equal(st, L.state.astype(np.float64))


def test_orthonormal_keys_overwrite_single_columns():
    # keys e_j, alpha = 1: column j becomes (1 - b_j) S0[:, j] + b_j v_j, the rest stay
    d = 8
    c = small_case([W.tree_chain(d)], d=d, Hk=1, Hv=1)
    L = c.layers[0]
    L.alpha[:] = 1.0
    perm = np.random.default_rng(0).permutation(d)
    L.k[:] = 0.0
    for i in range(d):
        L.k[0, i, 0, perm[i]] = 1.0
    _, snap, _ = run_scan(c, snap_nodes=all_nodes(c))
    S = L.state[c.state_row[0], 0].astype(np.float64).copy()
    for i in range(d):
        j = perm[i]
        b = float(L.beta[0, i, 0])
        S[:, j] = S[:, j] + b * (L.v[0, i, 0].astype(np.float64) - S[:, j])
        np.testing.assert_allclose(snap[0, i, 0], S, rtol=1e-15, atol=1e-18)


def test_beta_one_full_orthonormal_chain_solves_SK_equals_V():
    # alpha = beta = 1, keys = columns of an orthogonal matrix: after d updates S K = V exactly,
    # i.e. S = V K^{-1} (library linear solve), whatever S0 was.
    d = 12
    c = small_case([W.tree_chain(d)], d=d, Hk=1, Hv=1)
    L = c.layers[0]
    L.alpha[:] = 1.0
    L.beta[:] = 1.0
    Q, _ = np.linalg.qr(np.random.default_rng(3).normal(size=(d, d)))
    kk = Q.T.copy()                      # node i's key = column i of Q (float64, not rounded)
    k64 = kk.reshape(1, d, 1, d)
    o, snap, _ = O.scan(c.parent, c.slot, c.state_row, L.q, k64, L.v, L.alpha, L.beta, L.state,
                        snap_nodes=[[d - 1]])
    V = L.v[0, :, 0, :].astype(np.float64).T   # [dv, nodes]: column i = v_i
    K = kk.T                                    # [dk, nodes]: column i = k_i
    S_expect = np.linalg.solve(K.T, V.T).T      # S K = V
    np.testing.assert_allclose(snap[0, 0, 0], S_expect, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- invariants
@pytest.mark.parametrize("seed", range(4))
def test_retrieval_invariant_any_tree(seed):
    # unit k: S_i k_i = (1 - b_i) a_i S_p k_i + b_i v_i (fails if the state is transposed,
    # if alpha is applied after the write, or if the parent is mistaken for the previous row)
    c = small_case(rand_parents(10 + seed, 14), Hk=2, Hv=4, Ns=20, permute=True)
    L = c.layers[0]
    rep = c.Hv // c.Hk
    # exactly unit keys, supplied in float64
    k64 = L.k.astype(np.float64)
    k64 /= np.linalg.norm(k64, axis=-1, keepdims=True)
    _, snap, _ = O.scan(c.parent, c.slot, c.state_row, L.q, k64, L.v, L.alpha, L.beta, L.state,
                        snap_nodes=all_nodes(c), mode="walk")
    for i in range(c.N):
        s, p = c.slot[0, i], c.parent[0, i]
        for h in range(c.Hv):
            k = k64[0, s, h // rep]
            Sp = L.state[c.state_row[0], h].astype(np.float64) if p < 0 else snap[0, p, h]
            a, b = float(L.alpha[0, s, h]), float(L.beta[0, s, h])
            lhs = snap[0, i, h] @ k
            rhs = (1 - b) * a * (Sp @ k) + b * L.v[0, s, h].astype(np.float64)
            np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-13)


@pytest.mark.parametrize("seed", range(4))
def test_walk_equals_memo_bitwise(seed):
    c = small_case(rand_parents(20 + seed, 17, B=2), Hk=2, Hv=4)
    o1, s1, _ = run_scan(c, snap_nodes=all_nodes(c), mode="walk")
    o2, s2, _ = run_scan(c, snap_nodes=all_nodes(c), mode="memo")
    assert np.array_equal(o1, o2) and np.array_equal(s1, s2)


# ---------------------------------------------------------------- other algebra, library routines
def _transition_product(c, L, b, h, i):
    """S_i = S0 M + W with M, W from explicit per-node affine maps
    S -> a S (I - beta k k^T) + beta v k^T, multiplied out along the ancestry."""
    d = c.d
    rep = c.Hv // c.Hk
    M = np.eye(d)
    Wm = np.zeros((d, d))
    for t in T.ancestry(c.parent[b].tolist(), i):
        s = c.slot[b, t]
        k = L.k[b, s, h // rep].astype(np.float64)
        v = L.v[b, s, h].astype(np.float64)
        a, be = float(L.alpha[b, s, h]), float(L.beta[b, s, h])
        A = a * (np.eye(d) - be * np.outer(k, k))
        M = M @ A
        Wm = Wm @ A + be * np.outer(v, k)
    return L.state[c.state_row[b], h].astype(np.float64) @ M + Wm


@pytest.mark.parametrize("parents", [[TINY], rand_parents(31, 11)])
def test_against_explicit_transition_matrices(parents):
    c = small_case(parents, Hk=1, Hv=2, d=16)
    L = c.layers[0]
    o, snap, _ = run_scan(c, snap_nodes=all_nodes(c), mode="walk")
    for i in range(c.N):
        for h in range(c.Hv):
            S = _transition_product(c, L, 0, h, i)
            np.testing.assert_allclose(snap[0, i, h], S, rtol=0, atol=1e-13)
            np.testing.assert_allclose(o[0, c.slot[0, i], h], S @ L.q[0, c.slot[0, i], h // 2].astype(np.float64),
                                       rtol=0, atol=1e-13)


@pytest.mark.parametrize("seed", range(3))
def test_against_ancestor_masked_triangular_solve(seed):
    """Related-work form (a triangular system over strict-ancestor interactions): with
    G(t,s) = product of alpha over the nodes after s up to t and g_t = G from the root,
    (I + A) Delta = rhs where A[t,s] = beta_t G(t,s) (k_s . k_t) for strict ancestors s and
    rhs_t = beta_t (v_t - g_t S0 k_t); then o_t = g_t S0 q_t + sum_{s anc-or-self} G(t,s) (k_s . q_t) Delta_s.
    Solved with scipy's triangular solver."""
    c = small_case(rand_parents(40 + seed, 15), Hk=1, Hv=1, d=16)
    L = c.layers[0]
    par = c.parent[0].tolist()
    N, d = c.N, c.d
    K = L.k[0, :, 0].astype(np.float64)
    Q = L.q[0, :, 0].astype(np.float64)
    V = L.v[0, :, 0].astype(np.float64)
    al = L.alpha[0, :, 0].astype(np.float64)
    be = L.beta[0, :, 0].astype(np.float64)
    S0 = L.state[c.state_row[0], 0].astype(np.float64)
    G = np.zeros((N, N))      # G[t, s] for s in ancestors-or-self of t
    g = np.zeros(N)
    for t in range(N):
        anc = T.ancestry(par, t)
        g[t] = np.prod(al[anc])
        for j, s in enumerate(anc):
            G[t, s] = np.prod(al[anc[j + 1:]])
    strict = G.copy()
    np.fill_diagonal(strict, 0.0)
    A = be[:, None] * strict * (K @ K.T)
    rhs = be[:, None] * (V - g[:, None] * (K @ S0.T))
    Delta = scipy.linalg.solve_triangular(np.eye(N) + A, rhs, lower=True)
    o_expect = g[:, None] * (Q @ S0.T) + (G * (Q @ K.T)) @ Delta
    o, _, _ = run_scan(c, mode="walk")
    np.testing.assert_allclose(o[0, :, 0], o_expect, rtol=0, atol=1e-12)


def test_leaf_shortcut_identity():
    # o_i = a_i (S_p q_i) + delta_i (k_i . q_i): an output needs only the parent's state
    c = small_case([TINY], Hk=1, Hv=1)
    L = c.layers[0]
    o, snap, _ = run_scan(c, snap_nodes=all_nodes(c))
    for i in range(c.N):
        p = c.parent[0, i]
        Sp = L.state[c.state_row[0], 0].astype(np.float64) if p < 0 else snap[0, p, 0]
        k, q, v = (x[0, i, 0].astype(np.float64) for x in (L.k, L.q, L.v))
        a, b = float(L.alpha[0, i, 0]), float(L.beta[0, i, 0])
        dl = b * (v - a * (Sp @ k))
        np.testing.assert_allclose(o[0, i, 0], a * (Sp @ q) + dl * (k @ q), rtol=0, atol=1e-14)


# ---------------------------------------------------------------- topology independence
def test_off_path_poison_leaves_results_bitwise_unchanged_and_sibling_swap_changes_them():
    c = small_case([TINY], Hk=1, Hv=2)
    L = c.layers[0]
    o_ref, s_ref, _ = run_scan(c, snap_nodes=[[6]])
    # poison every node not on 0 -> 2 -> 6
    for arr in (L.q, L.k, L.v, L.alpha, L.beta):
        for n in (1, 3, 4, 5):
            arr[0, n] = 1e30
    o_p, s_p, _ = run_scan(c, snap_nodes=[[6]])
    for n in (0, 2, 6):
        assert np.array_equal(o_p[0, n], o_ref[0, n])
    assert np.array_equal(s_p, s_ref)
    # negative control: substituting sibling 3 for node 2 in the ancestry of 6 must be detected
    c2 = small_case([[-1, -1, 0, 0, 1, 1, 3]], Hk=1, Hv=2)
    o_s, _, _ = run_scan(c2)
    assert np.abs(o_s[0, 6] - o_ref[0, 6]).max() > 1e-3


def test_slot_permutation_leaves_logical_results_bitwise_unchanged():
    par = rand_parents(50, 13)
    c = small_case(par, Hk=2, Hv=4, Ns=13)
    L = c.layers[0]
    o_ref, s_ref, _ = run_scan(c, snap_nodes=all_nodes(c))
    Ns = 19
    rs = np.random.default_rng(5)
    slot = rs.permutation(Ns)[: c.N].astype(np.int32).reshape(1, -1)

    def scatter(a, fill):
        out = np.full((1, Ns) + a.shape[2:], fill, dtype=a.dtype)
        out[0, slot[0]] = a[0]
        return out
    o, s, _ = O.scan(c.parent, slot, c.state_row, scatter(L.q, 9e9), scatter(L.k, 9e9), scatter(L.v, 9e9),
                     scatter(L.alpha, 9e9), scatter(L.beta, 9e9), L.state, snap_nodes=all_nodes(c))
    assert np.array_equal(o[0, slot[0]], o_ref[0])
    assert np.array_equal(s, s_ref)
    pad = sorted(set(range(Ns)) - set(slot[0].tolist()))
    assert np.all(o[0, pad] == 0.0)       # padding rows are zero


def test_value_heads_share_their_qk_head_and_skipped_sequences_are_zero():
    c = small_case(rand_parents(60, 9, B=2), Hk=2, Hv=6)
    L = c.layers[0]
    o, _, _ = run_scan(c)
    rep = 3
    for h in range(c.Hv):
        g = h // rep
        o1, _, _ = O.scan(c.parent, c.slot, c.state_row, L.q[:, :, g:g + 1], L.k[:, :, g:g + 1],
                          L.v[:, :, h:h + 1], L.alpha[:, :, h:h + 1], L.beta[:, :, h:h + 1],
                          L.state[:, h:h + 1])
        assert np.array_equal(o1[:, :, 0], o[:, :, h])
    row = c.state_row.copy()
    row[1] = -1
    o2, _, _ = O.scan(c.parent, c.slot, row, L.q, L.k, L.v, L.alpha, L.beta, L.state)
    assert np.array_equal(o2[0], o[0]) and np.all(o2[1] == 0.0)


def test_l2norm_flag_and_scale():
    c = small_case([TINY], Hk=1, Hv=2)
    L = c.layers[0]
    rs = np.random.default_rng(1)
    qraw = rs.normal(size=L.q.shape) * 3.0
    kraw = rs.normal(size=L.k.shape) * 0.3
    eps = 1e-6
    qn = qraw / np.sqrt((qraw ** 2).sum(-1, keepdims=True) + eps)
    kn = kraw / np.sqrt((kraw ** 2).sum(-1, keepdims=True) + eps)
    o_a, _, _ = O.scan(c.parent, c.slot, c.state_row, qraw, kraw, L.v, L.alpha, L.beta, L.state,
                       l2norm=True, eps=eps, scale=0.25)
    o_b, _, _ = O.scan(c.parent, c.slot, c.state_row, qn, kn, L.v, L.alpha, L.beta, L.state)
    np.testing.assert_allclose(o_a, 0.25 * o_b, rtol=1e-13, atol=1e-15)


# ---------------------------------------------------------------- commit
def test_commit_equals_scan_state_at_last_accepted_node():
    c = small_case(rand_parents(70, 16, B=3), Hk=2, Hv=4)
    L = c.layers[0]
    _, snap, _ = run_scan(c, snap_nodes=all_nodes(c))
    ends = [15, 7, 0]
    acc, ln = [], []
    for b in range(3):
        a, l, _ = T.path_from_node(c.parent[b].tolist(), ends[b], c.N)
        acc.append(a)
        ln.append(l)
    st, _, status, _ = O.commit(c.parent, c.slot, c.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state, acc, ln)
    assert np.all(status == 0)
    for b in range(3):
        assert np.array_equal(st[c.state_row[b]], snap[b, ends[b]])
    untouched = sorted(set(range(c.rows)) - set(c.state_row.tolist()))
    assert np.array_equal(st[untouched], L.state[untouched].astype(np.float64))


def test_commit_len_zero_poisoned_tail_invalid_path_and_zero_replay_control():
    c = small_case([TINY], Hk=1, Hv=2)
    L = c.layers[0]
    args = (c.parent, c.slot, c.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state)
    S0 = L.state.astype(np.float64)
    st, hist, status, _ = O.commit(*args, [[0, 2, 6]], [0], x=L.x, hist=L.hist)
    assert status[0] == 0 and np.array_equal(st, S0) and np.array_equal(hist, L.hist.astype(np.float64))
    st_full, _, _, _ = O.commit(*args, [[0, 2, 6]], [3])
    st_two, _, _, _ = O.commit(*args, [[0, 2, 123456]], [2])       # entry beyond len is ignored
    _, snap, _ = run_scan(c, snap_nodes=[[2, 6]])
    assert np.array_equal(st_two[c.state_row[0]], snap[0, 0]) and np.array_equal(st_full[c.state_row[0]], snap[0, 1])
    # zero-replay control: a commit that did nothing is distinguishable from the accepted state
    assert np.abs(S0[c.state_row[0]] - snap[0, 1]).max() > 1e-2
    for bad, code in (([0, 4, 6], T.PATH_BAD_LINK), ([2, 6, -1], T.PATH_BAD_ROOT), ([0, 9, 6], T.PATH_BAD_NODE)):
        st, hist, status, _ = O.commit(*args, [bad], [3], x=L.x, hist=L.hist)
        assert status[0] == code and np.array_equal(st, S0) and np.array_equal(hist, L.hist.astype(np.float64))
    st, _, status, _ = O.commit(*args, [[0, 2, 6]], [4])
    assert status[0] == T.PATH_BAD_LEN and np.array_equal(st, S0)


def test_two_cycles_equal_one_longer_chain():
    # verify -> commit -> verify: a 6-chain equals a 3-chain committed and then another 3-chain
    c = small_case([W.tree_chain(6)], Hk=1, Hv=2)
    L = c.layers[0]
    o_full, snap, _ = run_scan(c, snap_nodes=[[5]])
    c3 = small_case([W.tree_chain(3)], Hk=1, Hv=2)
    first = tuple(a[:, :3] for a in (L.q, L.k, L.v, L.alpha, L.beta))
    second = tuple(a[:, 3:] for a in (L.q, L.k, L.v, L.alpha, L.beta))
    st, _, status, _ = O.commit(c3.parent, c3.slot, c.state_row, *first, L.state, [[0, 1, 2]], [3])
    o2, snap2, _ = O.scan(c3.parent, c3.slot, c.state_row, *second, st, snap_nodes=[[2]])
    assert np.array_equal(o2[0], o_full[0, 3:]) and np.array_equal(snap2, snap)


def test_commit_history_is_last_three_of_old_plus_accepted_inputs():
    c = small_case([TINY], Hk=1, Hv=2)
    L = c.layers[0]
    args = (c.parent, c.slot, c.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state)
    r = c.state_row[0]
    x = L.x.astype(np.float64)
    h0 = L.hist.astype(np.float64)
    _, h, _, _ = O.commit(*args, [[0, 2, 6]], [3], x=L.x, hist=L.hist)
    assert np.array_equal(h[r], x[0, [0, 2, 6]])
    _, h, _, _ = O.commit(*args, [[1, 5, -1]], [2], x=L.x, hist=L.hist)
    assert np.array_equal(h[r], np.stack([h0[r, 2], x[0, 1], x[0, 5]]))
    _, h, _, _ = O.commit(*args, [[1, -1, -1]], [1], x=L.x, hist=L.hist)
    assert np.array_equal(h[r], np.stack([h0[r, 1], h0[r, 2], x[0, 1]]))


# ------------------------------------------------------------------ raw gate inputs
def test_raw_gate_activation_closed_forms_and_identities():
    import scipy.special
    one = lambda v: np.full((1, 1, 1), v)
    # softplus(0) = ln 2, a_log = 0: alpha = exp(-ln 2) = 1/2; sigmoid(0) = 1/2
    a, b = O.gates_from_raw(one(0.3), one(0.0), [0.0], [-0.3])
    assert a[0, 0, 0] == pytest.approx(0.5, abs=1e-15) and b[0, 0, 0] == 0.5
    # a_log = ln 3: alpha = 2^-3
    a, _ = O.gates_from_raw(one(0.0), one(0.0), [np.log(3.0)], [0.0])
    assert a[0, 0, 0] == pytest.approx(0.125, rel=1e-14)
    # limits: a very negative input leaves the state undecayed, a large one decays like exp(-x e^a_log)
    a, b = O.gates_from_raw(np.array([[[-60.0], [40.0]]]), np.array([[[-60.0], [60.0]]]), [0.5], [0.0])
    assert a[0, 0, 0] == pytest.approx(1.0, abs=1e-15) and a[0, 1, 0] == pytest.approx(np.exp(-40.0 * np.exp(0.5)), rel=1e-12)
    assert b[0, 0, 0] < 1e-25 and b[0, 1, 0] == pytest.approx(1.0, abs=1e-15)
    # identities and the library routines, per head (a_log and dt_bias index the last axis)
    rs = np.random.default_rng(3)
    g, r = rs.standard_normal((2, 5, 3)) * 4, rs.standard_normal((2, 5, 3)) * 4
    a_log, dt = rs.uniform(-1, 1, 3), rs.uniform(-1, 1, 3)
    a, b = O.gates_from_raw(g, r, a_log, dt)
    assert np.all((a > 0) & (a <= 1)) and np.all((b > 0) & (b < 1))
    np.testing.assert_allclose(b, scipy.special.expit(r), rtol=1e-14)
    np.testing.assert_allclose(-np.log(a) / np.exp(a_log), np.logaddexp(0.0, g + dt), rtol=1e-9, atol=1e-14)
    b_neg = O.gates_from_raw(g, -r, a_log, dt)[1]
    np.testing.assert_allclose(b + b_neg, 1.0, rtol=1e-14)                       # sigmoid(x) + sigmoid(-x) = 1
    sp = lambda x: -np.log(O.gates_from_raw(x, r, np.zeros(3), np.zeros(3))[0])
    np.testing.assert_allclose(sp(g) - sp(-g), g, rtol=1e-9, atol=1e-12)        # softplus(x) - softplus(-x) = x
    a_up = O.gates_from_raw(g + 0.1, r, a_log, dt)[0]
    assert np.all(a_up < a)                                                      # decay is monotone in the input
