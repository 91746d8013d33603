"""Oracle of the device-resident acceptance walk (tree speculative sampling).

TEST INFRASTRUCTURE ONLY (see oracle/gdn_oracle.cpp): plain NumPy, one sequence at a time,
shares nothing with the CUDA library.

What it computes (Algorithm 1, "Select one continuation": the accepted materialized path A and
the pending token b* from sampling with the target probabilities p and the proposal probabilities
q; Sec. "One device-selected path drives native continuation": accepted node indices, path length,
emitted token and the selected final row are fixed-shape device products).  Starting at the
pre-tree state, the walk looks at the children of the current node in ascending logical index:

greedy      the child whose token equals argmax of the current node's target row is accepted
            (lowest index wins ties, the reference argmax convention of Sec. "Fuse draft selection
            without changing proposals"); if there is none the walk stops and b* is that argmax.
rejection   ordinary rejection sampling per candidate (Appendix "Serving configuration and
            measurement": accepted mass min(p, q), residual mass proportional to (p - q)+): child c
            with token x is accepted iff u_c q_c(x) < r(x) / Z, where r is the current unnormalised
            residual target (r = p at first) and Z its sum; after a rejection r <- (r - Z q_c)+.  If
            every child is rejected (or there is none) b* is drawn from r / Z by an exponential
            race, b* = argmax_i r_i / e_i with e_i ~ Exp(1), lowest index on ties.

Readings where the paper is silent: children are tried in ascending logical index; each child
carries the proposal row it was drawn from; all random numbers (one uniform per node, one
exponential variate per vocabulary entry) are inputs; the acceptance test and the residual update
are taken in float64 and the residual is stored in float32, the race keys are float32 quotients
(the CUDA kernel takes the same decisions in the same precisions); if a residual sums to zero the
target row is restored.

Pins (tests/test_oracle_accept.py): a hand-worked greedy walk; q = p accepts the first child;
zero target mass on every candidate rejects them all; Monte-Carlo distribution preservation (the
first emitted token is distributed as p whatever q is) and the exponential race against r / Z.
"""
from __future__ import annotations

from typing import Optional, Sequence, Tuple

import numpy as np

GREEDY, REJECTION = 0, 1


def _children(parent: Sequence[int], node: int):
    return [i for i, p in enumerate(parent) if p == node]


def argmax_lowest(a: np.ndarray) -> int:
    return int(np.flatnonzero(a == a.max())[0])


def accept_one(parent: Sequence[int], slot: Sequence[int], n_slots: int, token: np.ndarray, p: np.ndarray,
               q: Optional[np.ndarray], uniforms: Optional[np.ndarray], noise: Optional[np.ndarray], mode: int,
               lmax: int) -> Tuple[list, int, int, int]:
    """One sequence.  token [Ns]; p [Ns+1, V] float32 (row Ns = after the pre-tree state); q [Ns, V];
    uniforms [Ns]; noise [V].  Returns (accepted padded with -1 to lmax, length, next token, final node)."""
    cur, path = -1, []
    while True:
        prow = n_slots if cur < 0 else slot[cur]
        kids = _children(parent, cur)
        if mode == GREEDY:
            best = argmax_lowest(p[prow])
            hit = [c for c in kids if int(token[slot[c]]) == best]
            if hit and len(path) < lmax:
                cur = hit[0]
                path.append(cur)
                continue
            nxt = best
            break
        r = p[prow].astype(np.float32).copy()
        Z = float(np.sum(r.astype(np.float64)))
        took = None
        for c in kids:
            if len(path) >= lmax:
                break
            x = int(token[slot[c]])
            qrow = q[slot[c]].astype(np.float64)
            u = float(uniforms[slot[c]])
            if (u * qrow[x]) * Z < float(r[x]):
                took = c
                break
            r_new = np.maximum(r.astype(np.float64) - Z * qrow, 0.0).astype(np.float32)
            Z_new = float(np.sum(r_new.astype(np.float64)))
            if Z_new > 0.0:
                r, Z = r_new, Z_new
            else:                      # empty residual: restore the target row
                r = p[prow].astype(np.float32).copy()
                Z = float(np.sum(r.astype(np.float64)))
        if took is not None:
            cur = took
            path.append(cur)
            continue
        keys = r / noise.astype(np.float32)          # float32 quotients
        nxt = argmax_lowest(keys)
        break
    return path + [-1] * (lmax - len(path)), len(path), nxt, cur


def accept(parent, slot, n_slots, token, p, q=None, uniforms=None, noise=None, mode=GREEDY, lmax=16):
    """Batch wrapper: parent, slot [B, N]; token [B, Ns]; p [B, Ns+1, V]; q [B, Ns, V]; uniforms [B, Ns];
    noise [B, V] -> accepted [B, lmax], len [B], next_token [B], final_node [B] (int32)."""
    B = len(parent)
    acc = np.full((B, lmax), -1, np.int32)
    ln = np.zeros(B, np.int32)
    nxt = np.zeros(B, np.int32)
    fin = np.zeros(B, np.int32)
    for b in range(B):
        a, l, t, f = accept_one(list(parent[b]), list(slot[b]), n_slots, token[b], p[b],
                                None if q is None else q[b], None if uniforms is None else uniforms[b],
                                None if noise is None else noise[b], mode, lmax)
        acc[b], ln[b], nxt[b], fin[b] = a, l, t, f
    return acc, ln, nxt, fin
