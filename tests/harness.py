"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI on a
synthetic case, run the fp64 oracle on the same rounded arrays, compare."""
import numpy as np
import torch

from oracle import gdn_oracle as O
from paper_2609_23900_b200 import binding
from synthetic.device_case import DeviceCase

_ctx = None


def ctx(algo="auto"):
    """Shared context; `algo` selects the scan kernel ("auto", "rank1", "gram", "solve", "direct", "tensor") for the calls that follow."""
    global _ctx
    if _ctx is None:
        _ctx = binding.Context(0)
    _ctx.set_scan_algo(algo)
    return _ctx


def gram_eligible(c) -> bool:
    """Shapes the tensor-core Gram-form scan takes: d = 128, bf16 operands, depth <= 16."""
    from synthetic import workload as W
    depth = max(max(W.tree_depths(p.tolist())) for p in c.parent)
    return c.d == 128 and c.in_dtype == "bf16" and depth <= 16


def ulp_bf16(ref):
    a = np.maximum(np.abs(ref), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(a)) - 7)


def assert_close(got, ref, *, bf16=False, what=""):
    """|d| <= 1e-3 (1 + |ref|); bf16-typed results may add half a bf16 ulp of the reference."""
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    tol = 1e-3 * (1.0 + np.abs(ref))
    if bf16:
        tol = tol + 0.5 * ulp_bf16(ref)
    err = np.abs(got - ref)
    bad = err > tol
    assert np.all(np.isfinite(got)), f"{what}: non-finite values"
    assert not bad.any(), (f"{what}: {bad.sum()} of {bad.size} outside tolerance; worst |d|={err.max():.3e} "
                           f"at ref={ref.flat[err.argmax()]:.3e}")
    return float((err / (1.0 + np.abs(ref))).max())


def device_gates(dc: DeviceCase, layer=0):
    """The gates the recurrence consumes, from the arrays the GPU reads (raw-gate layers: activated in fp64)."""
    a, b = dc.np("alpha", layer), dc.np("beta", layer)
    if dc.t("a_log", layer) is not None:
        a, b = O.gates_from_raw(a, b, dc.np("a_log", layer), dc.np("dt_bias", layer))
    return a, b


def oracle_scan_from_device(dc: DeviceCase, layer=0, **kw):
    """Oracle scan on the operands the GPU recorded (same rounded arrays on both sides)."""
    c = dc.case
    alpha, beta = device_gates(dc, layer)
    return O.scan(c.parent, c.slot, c.state_row, dc.np("q", layer), dc.np("k", layer), dc.np("v", layer),
                  alpha, beta, c.layers[layer].state, scale=dc.scale,
                  l2norm=dc.qk_l2norm, eps=dc.l2_eps, **kw)


def oracle_commit_from_device(dc: DeviceCase, layer=0, accepted=None, length=None, with_hist=True, **kw):
    c = dc.case
    L = c.layers[layer]
    acc = c.accepted if accepted is None else accepted
    ln = c.accepted_len if length is None else length
    x, hist = (L.x, L.hist) if with_hist else (None, None)
    alpha, beta = device_gates(dc, layer)
    return O.commit(c.parent, c.slot, c.state_row, dc.np("q", layer), dc.np("k", layer), dc.np("v", layer),
                    alpha, beta, L.state, acc, ln, x=x, hist=hist,
                    l2norm=dc.qk_l2norm, eps=dc.l2_eps, **kw)
