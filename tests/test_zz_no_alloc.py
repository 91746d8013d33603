"""The scan entry point that allocates nothing (lumo_gdn_tree_scan_static).

Collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test.  It calls the entry point through the C ABI twice in a row and checks both
results against the allocating entry point (lumo_gdn_tree_verify) on the same inputs; the two
run the same kernel on different stack memory, so the outputs must agree bit for bit, which is
inside the 1e-3 (1 + |ref|) rule the other parity tests use.
"""
import numpy as np
import pytest
import torch

from paper_2609_23900_b200 import binding
from synthetic import workload as W
from synthetic.device_case import DeviceCase

pytestmark = pytest.mark.gpu


def test_static_stack_scan_matches_allocating_verify_twice():
    ctx = binding.Context(0)
    ctx.set_scan_algo("rank1")      # compare like with like: the entry point under test runs the rank-1 kernel
    # a tree with several branching internal nodes so that the stack is really used
    parents = [W.tree_random(W.IntStream(W.stream_key(77, b)), 64, 8) for b in range(4)]
    case = W.make_case("noalloc", parents, seed=77, Hk=4, Hv=8, d=128, in_dtype="bf16")
    ref = DeviceCase(ctx, case, use_conv=False)
    assert len(ref.desc.table("schedule", 0)) > case.N          # pushes / pops present
    ref.verify()
    torch.cuda.synchronize()
    expect = ref.t("out").clone()
    assert torch.isfinite(expect).all() and expect.abs().max() > 0

    dc = DeviceCase(ctx, case, use_conv=False)
    for trial in range(2):
        dc.t("out").fill_(float("nan"))
        ctx.scan_static(dc.desc, dc.layers)
        torch.cuda.synchronize()
        got = dc.t("out")
        err = (got - expect).abs() / (1 + expect.abs())
        assert torch.isfinite(got).all() and float(err.max()) <= 1e-3, (trial, float(err.max()))
        assert torch.equal(got, expect), trial                    # same kernel, same arithmetic
        assert dc.np("status").tolist() == [0] * case.B
    assert binding.Context.static_stack_bytes() == 64 << 20


def test_static_stack_scan_refuses_shapes_beyond_its_capacity():
    ctx = binding.Context(0)
    # a comb: a 40-node spine whose every node also has a later-numbered internal child (a side
    # branch with one leaf).  The walk descends the spine first and must keep every spine state
    # for the side branch, so the schedule needs ~40 stack levels per CTA: 256 CTAs x 40 x 16 KiB
    # is beyond 64 MiB.
    depth = 40
    parent = [i - 1 for i in range(depth)]
    for sp in range(depth):
        parent.append(sp)                  # side branch head (internal)
        parent.append(len(parent) - 1)     # its leaf
    case = W.make_case("deep", [parent] * 8, seed=78, Hk=4, Hv=8, d=128, in_dtype="bf16")
    dc = DeviceCase(ctx, case, use_conv=False)
    dc.t("out").fill_(7.0)
    with pytest.raises(binding.LumoError) as e:
        ctx.scan_static(dc.desc, dc.layers)
    assert e.value.code == 4 and "built-in stack holds" in str(e.value)
    torch.cuda.synchronize()
    assert torch.all(dc.t("out") == 7.0)                           # nothing was enqueued
    dc.verify()                                                    # the allocating path still takes it
    torch.cuda.synchronize()
    assert torch.isfinite(dc.t("out")).all()
