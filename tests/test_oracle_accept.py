"""Pins of the acceptance-walk oracle (oracle/accept_oracle.py): a hand-worked greedy walk, special
cases with known answers, and Monte-Carlo checks that rejection sampling preserves the target
distribution (the property the scheme exists for) and that the exponential race samples r / Z."""
import numpy as np

from oracle import accept_oracle as A

TINY = [-1, -1, 0, 0, 1, 1, 2]
IDENT = list(range(7))


def test_greedy_walk_by_hand():
    V = 5
    token = np.array([3, 1, 4, 0, 2, 2, 1])
    p = np.full((8, V), 0.1, np.float32)
    p[7, 3] = 0.6      # after the pre-tree state: token 3 -> node 0 (its token is 3)
    p[0, 4] = 0.6      # after node 0: token 4 -> node 2
    p[2, 1] = 0.6      # after node 2: token 1 -> node 6
    p[6, 2] = 0.6      # after node 6 (leaf): bonus token 2
    acc, ln, nxt, fin = A.accept_one(TINY, IDENT, 7, token, p, None, None, None, A.GREEDY, 3)
    assert (acc, ln, nxt, fin) == ([0, 2, 6], 3, 2, 6)
    p[0, 4] = 0.1
    p[0, 2] = 0.6      # after node 0 the target wants token 2; no child of 0 carries it: correction token
    assert A.accept_one(TINY, IDENT, 7, token, p, None, None, None, A.GREEDY, 3) == ([0, -1, -1], 1, 2, 0)
    p[7] = 0.2         # a flat row: ties go to the lowest token index, which no child of the root carries
    assert A.accept_one(TINY, IDENT, 7, token, p, None, None, None, A.GREEDY, 3) == ([-1, -1, -1], 0, 0, -1)


def test_rejection_special_cases():
    rs = np.random.default_rng(0)
    V = 11
    token = rs.integers(0, V, 7)
    p = rs.dirichlet(np.ones(V), 8).astype(np.float32)
    u = rs.uniform(size=7).astype(np.float32) * 0.999
    noise = rs.exponential(size=V).astype(np.float32)
    # q == p at every node: the first child is always accepted (u < 1), down to a leaf
    q = np.stack([p[7 if TINY[i] < 0 else TINY[i]] for i in range(7)])
    acc, ln, nxt, fin = A.accept_one(TINY, IDENT, 7, token, p, q, u, noise, A.REJECTION, 3)
    assert acc == [0, 2, 6] and ln == 3 and fin == 6
    assert nxt == A.argmax_lowest(p[6] / noise)       # bonus token: race on the leaf's target row
    # zero target mass on both candidates of the root: both rejected, residual = p off the proposals
    p2 = p.copy()
    p2[7, token[0]] = 0.0
    p2[7, token[1]] = 0.0
    q2 = np.zeros((7, V), np.float32)
    q2[0, token[0]] = 1.0
    q2[1, token[1]] = 1.0
    acc, ln, nxt, fin = A.accept_one(TINY, IDENT, 7, token, p2, q2, u, noise, A.REJECTION, 3)
    assert ln == 0 and fin == -1 and nxt == A.argmax_lowest(p2[7] / noise)


def test_rejection_sampling_preserves_the_target_distribution():
    # root with three candidates drawn independently from q; the first emitted token (an accepted
    # candidate's token, or the residual draw) must be distributed as p, whatever q is
    rs = np.random.default_rng(1)
    V, trials = 6, 60000
    p_root = np.array([0.35, 0.05, 0.25, 0.15, 0.12, 0.08], np.float32)
    qd = np.array([0.10, 0.40, 0.10, 0.10, 0.10, 0.20], np.float32)
    parent, slot = [-1, -1, -1], [0, 1, 2]
    p = np.zeros((4, V), np.float32)
    p[3] = p_root
    p[:3] = 1.0 / V
    counts = np.zeros(V)
    for _ in range(trials):
        token = rs.choice(V, size=3, p=qd / qd.sum())
        q = np.tile(qd, (3, 1))
        u = rs.uniform(size=3).astype(np.float32)
        noise = rs.exponential(size=V).astype(np.float32)
        acc, ln, nxt, fin = A.accept_one(parent, slot, 3, token, p, q, u, noise, A.REJECTION, 1)
        counts[token[acc[0]] if ln else nxt] += 1
    freq = counts / trials
    assert np.abs(freq - p_root).max() < 0.008, freq          # ~4 sigma at 60000 trials


def test_exponential_race_samples_the_normalised_residual():
    rs = np.random.default_rng(2)
    r = np.array([0.0, 0.5, 0.2, 0.0, 1.3], np.float32)
    trials = 40000
    wins = np.zeros(5)
    for _ in range(trials):
        wins[A.argmax_lowest(r / rs.exponential(size=5).astype(np.float32))] += 1
    assert np.abs(wins / trials - r / r.sum()).max() < 0.01
    assert wins[0] == wins[3] == 0
