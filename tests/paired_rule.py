"""The paper's paired error rule as an executable check (Sec. "Numerical and candidate-selection
validation", Table "GDN component checks"; Appendix, "Direct GDN comparisons").

A cell fixes (sequence, output node, value head); errors are reduced over the 128 output entries.  For
every cell both the root-mean-square and the maximum absolute error of the tree scan against the
float64 recurrence must satisfy

    E_tree <= 1.10 E_native + 2^-24 M_64 + 2^-149,

where E_native is the same error of the native sequential update and M_64 the root-mean-square (or the
maximum magnitude) of the reference.  Two native sides are evaluated:

  "sequential kernel": the library's own sequential recurrence with outputs, i.e. the rank-1 fp32 scan,
      whose per-token arithmetic is the commit kernel's (its node states equal the commit kernel's chain
      states bit for bit, see tests/test_gpu_paired_rule.py) and whose output product is fp32 as well.
      This is the reading of "the sequential comparator is the native GPU recurrence".
  "commit chain": the commit kernel run as a chain, for every node the accepted path that ends there
      replayed from the pre-tree state (lumo_gdn_commit); the node's output is the product of that fp32
      state with the query taken in float64 on the host, so the output product adds no error of its own.
      A stricter comparator than any fp32 kernel can be: reported, not required.

TEST INFRASTRUCTURE: uses the fp64 oracle; imported by the tests and by the CPU-baseline leg of
bench.py only.
"""
import numpy as np
import torch

from oracle import gdn_oracle as O
from synthetic import workload as W
from synthetic.device_case import DeviceCase


def native_chain_outputs(ctx, dc, layer=0):
    """o_native [B, Ns, Hv, d] (float64): the commit kernel replays the path to every node in turn."""
    c = dc.case
    dev = dc.dev
    state = dc.t("state", layer)
    S0 = state.clone()
    lmax = max(max(W.tree_depths(p.tolist())) for p in c.parent)
    acc = torch.zeros((c.B, lmax), dtype=torch.int32, device=dev)
    ln = torch.zeros((c.B,), dtype=torch.int32, device=dev)
    rep = c.Hv // c.Hk
    q = dc.np("q", layer)                                            # [B, Ns, Hk, d] float64
    out = np.zeros((c.B, c.Ns, c.Hv, c.d))
    rows = torch.from_numpy(c.state_row.astype(np.int64)).to(dev)
    for i in range(c.N):
        node = torch.full((c.B,), i, dtype=torch.int32, device=dev)
        ctx.path_from_node(dc.desc, node, lmax, acc, ln)
        state.copy_(S0)
        ctx.commit(dc.desc, [dc.layers[layer]], acc, ln)
        S = state[rows].to(torch.float64).cpu().numpy()             # [B, Hv, d, d]
        for b in range(c.B):
            r = c.slot[b, i]
            qh = np.repeat(q[b, r], rep, axis=0) * dc.scale         # [Hv, d]
            out[b, r] = np.einsum("hvk,hk->hv", S[b], qh)
    state.copy_(S0)
    return out


def _cell_errors(x, ref):
    e = x - ref
    return np.sqrt((e ** 2).mean(-1)), np.abs(e).max(-1)


def paired_rule(ctx, case, algos=("gram", "direct", "tensor", "solve"), layer=0, with_commit_chain=True):
    """Per scan kernel: cells (sequence, node, value head) inside the paired bound against each native
    side, with the error levels behind the counts."""
    active = np.zeros((case.B, case.Ns), dtype=bool)
    for b in range(case.B):
        active[b, case.slot[b]] = True
    L = case.layers[layer]
    outs = {}
    for algo in ("rank1",) + tuple(a for a in algos if a != "rank1"):
        ctx.set_scan_algo(algo)
        dc = DeviceCase(ctx, case, use_conv=False, qk_l2norm=False)
        dc.verify()
        torch.cuda.synchronize()
        outs[algo] = dc.np("out", layer)
    ctx.set_scan_algo("auto")
    ref, _, _ = O.scan(case.parent, case.slot, case.state_row, dc.np("q", layer), dc.np("k", layer),
                       dc.np("v", layer), dc.np("alpha", layer), dc.np("beta", layer), L.state)
    m_rms, m_max = np.sqrt((ref ** 2).mean(-1)), np.abs(ref).max(-1)
    natives = {"sequential_kernel": _cell_errors(outs["rank1"], ref)}
    if with_commit_chain:
        natives["commit_chain"] = _cell_errors(native_chain_outputs(ctx, dc, layer), ref)
    act = active[:, :, None] & np.ones(m_rms.shape, dtype=bool)
    res = {"cells": int(act.sum()), "native": {}, "kernels": {}}
    for name, (rms_n, max_n) in natives.items():
        res["native"][name] = {"median_cell_rms_error": float(np.median(rms_n[act])), "max_abs_error": float(max_n[act].max())}
    for algo, out in outs.items():
        rms_t, max_t = _cell_errors(out, ref)
        entry = {"median_cell_rms_error": float(np.median(rms_t[act])), "max_abs_error": float(max_t[act].max())}
        for name, (rms_n, max_n) in natives.items():
            ok = (rms_t <= 1.10 * rms_n + 2.0 ** -24 * m_rms + 2.0 ** -149) & \
                 (max_t <= 1.10 * max_n + 2.0 ** -24 * m_max + 2.0 ** -149)
            entry["passed_vs_" + name] = int((ok & act).sum())
        res["kernels"][algo] = entry
    return res
