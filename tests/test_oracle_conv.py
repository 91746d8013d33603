"""Pins for the oracle's ancestry-gathered convolution (oracle/gdn_oracle.cpp: oracle_conv).

The chain case must equal a library causal depthwise conv1d over [history ; chain]
followed by the library SiLU; the other tests use closed forms and properties of the
ancestry gather (Sec. "Precompute branch histories while preserving arithmetic").
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import gdn_oracle as O
from synthetic import workload as W

TINY = [-1, -1, 0, 0, 1, 1, 2]


def case(parents, **kw):
    return W.make_case("t", parents, seed=11, Hk=1, Hv=2, d=8, in_dtype="f32", **kw)


def run(c, L=None, **kw):
    L = L or c.layers[0]
    return O.conv(c.parent, c.slot, c.state_row, L.x, L.conv_w, L.conv_b, L.hist, c.Ns, **kw)


@pytest.mark.parametrize("with_bias", [False, True])
def test_chain_equals_library_causal_depthwise_conv1d(with_bias):
    n = 9
    c = case([W.tree_chain(n), W.tree_chain(n)], with_bias=with_bias)
    L = c.layers[0]
    y = run(c)
    for b in range(c.B):
        seq = np.concatenate([L.hist[c.state_row[b]], L.x[b]], axis=0).astype(np.float64)   # [3+n, C]
        inp = torch.from_numpy(seq.T.copy()).unsqueeze(0)                                    # [1, C, 3+n]
        w = torch.from_numpy(L.conv_w.astype(np.float64)).unsqueeze(1)                       # [C, 1, 4]
        bias = None if L.conv_b is None else torch.from_numpy(L.conv_b.astype(np.float64))
        ref = F.silu(F.conv1d(inp, w, bias=bias, groups=c.C))[0].T.numpy()                   # [n, C]
        np.testing.assert_allclose(y[b], ref, rtol=1e-13, atol=1e-15)


def test_identity_tap_gives_silu_of_input():
    c = case([TINY])
    L = c.layers[0]
    L.conv_w[:] = 0.0
    L.conv_w[:, 3] = 1.0
    y = run(c)
    x = L.x.astype(np.float64)
    np.testing.assert_allclose(y, x / (1.0 + np.exp(-x)), rtol=1e-15, atol=0)


def test_each_tap_reads_the_right_ancestor_or_history_row():
    # one-hot taps turn the conv into a gather: tap j of node i reads window entry j
    c = case([TINY])
    L = c.layers[0]
    x = L.x.astype(np.float64)
    h = L.hist[c.state_row[0]].astype(np.float64)
    silu = lambda a: a / (1.0 + np.exp(-a))
    # (node, tap) -> expected source row, written by hand for parents [-1,-1,0,0,1,1,2]
    expect = {
        (0, 2): h[2], (0, 1): h[1], (0, 0): h[0],
        (1, 2): h[2], (5, 2): x[0, 1], (5, 1): h[2], (5, 0): h[1],
        (6, 2): x[0, 2], (6, 1): x[0, 0], (6, 0): h[2], (3, 2): x[0, 0], (4, 2): x[0, 1],
    }
    for tap in range(3):
        L.conv_w[:] = 0.0
        L.conv_w[:, tap] = 1.0
        y = run(c)
        for (node, t), src in expect.items():
            if t == tap:
                np.testing.assert_allclose(y[0, node], silu(src), rtol=1e-15, atol=0)


def test_siblings_differ_only_through_the_current_tap():
    c = case([TINY])
    L = c.layers[0]
    L.conv_w[:, 3] = 0.0
    y = run(c)
    assert np.array_equal(y[0, 2], y[0, 3]) and np.array_equal(y[0, 4], y[0, 5]) and np.array_equal(y[0, 0], y[0, 1])
    assert not np.array_equal(y[0, 2], y[0, 4])


def test_slot_permutation_padding_and_skipped_sequence():
    c = case([TINY, TINY])
    L = c.layers[0]
    y_ref = run(c)
    Ns = 10
    slot = np.stack([np.random.default_rng(s).permutation(Ns)[:7] for s in (1, 2)]).astype(np.int32)
    x = np.full((2, Ns, c.C), 7e7, dtype=np.float32)
    for b in range(2):
        x[b, slot[b]] = L.x[b]
    y = O.conv(c.parent, slot, c.state_row, x, L.conv_w, None, L.hist, Ns)
    for b in range(2):
        assert np.array_equal(y[b, slot[b]], y_ref[b])
        pad = sorted(set(range(Ns)) - set(slot[b].tolist()))
        assert np.all(y[b, pad] == 0.0)
    row = c.state_row.copy()
    row[0] = -1
    y2 = O.conv(c.parent, c.slot, row, L.x, L.conv_w, None, L.hist, c.Ns)
    assert np.all(y2[0] == 0.0) and np.array_equal(y2[1], y_ref[1])


def test_recorded_operand_rounding_is_rne():
    c = case([TINY])
    y = run(c)
    y16 = run(c, out_dtype="bf16")
    y32 = run(c, out_dtype="f32")
    assert np.array_equal(y32, y.astype(np.float32).astype(np.float64))
    # bf16: representable, and the nearest representable value
    t = torch.from_numpy(y16).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(t, y16)
    ulp = 2.0 ** (np.floor(np.log2(np.abs(y))) - 7)
    assert np.all(np.abs(y16 - y) <= ulp / 2 * (1 + 1e-12))
    # ties go to even; fp32-representable inputs agree with the library's fp32 -> bf16 cast
    assert O.round_bf16(1.0 + 2.0 ** -8) == 1.0
    assert O.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2.0 ** -6
    v = np.random.default_rng(0).normal(size=2000).astype(np.float32)
    lib = torch.from_numpy(v).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(np.array([O.round_bf16(float(a)) for a in v]), lib)
