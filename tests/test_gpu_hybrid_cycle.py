"""One verification cycle of a hybrid model under ONE tree descriptor (Sec. "Coordinating recurrent
state and attention under one descriptor"): a Gated DeltaNet layer and a full-attention layer verify the
same candidate tree through the same slot map, the acceptance walk selects a path on the device, and
both publishers consume that device-resident path: the recurrent committer replays it into the running
state, the KV publisher re-linearises it in the cache.  No host round trip between the calls.  The check:
every consumer ends on the SAME materialised prefix, and each matches its oracle for the path the walk
chose."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import accept_oracle as AC
from oracle import attn_oracle as A
from oracle import gdn_oracle as O
from synthetic import workload as W
from synthetic.device_case import DeviceAttnCase, DeviceCase
from tests.harness import assert_close, ctx
from tests.test_gpu_accept import make_inputs, run_device
from tests.test_gpu_attn import check_attention

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("mode", ["greedy", "rejection"])
def test_one_descriptor_drives_both_verifiers_and_both_publishers(mode):
    B, V = 4, 4099
    g = W.config_paper(B=B)                                   # 28 active rows in 32 slots, slots permuted
    a = W.make_attn_case("hybrid", [p.tolist() for p in g.parent], [700, 45, 1999, 128], seed=W.BASE_SEED + 77,
                         Hq=8, Hkv=2, Ns=g.Ns)
    a = dataclasses.replace(a, slot=g.slot.copy())            # the attention layer follows the SAME slot map
    token, p, q, u, noise = make_inputs(g.parent, g.slot, g.Ns, V, seed=33)   # accepts 0 to 12 nodes
    lmax = max(max(W.tree_depths(pp.tolist())) for pp in g.parent) + 1

    c = ctx("auto")
    dg = DeviceCase(c, g, out_dtype="bf16")
    da = DeviceAttnCase(c, a, n_splits=0)
    desc = dg.desc                                            # one descriptor for every call below
    S0 = dg.np("state").copy()

    c.verify(desc, dg.layers)                                 # recurrent verifier
    c.kv_write_tree(desc, da.packed)                          # attention verifier
    c.tree_attention(desc, da.packed)
    acc, ln, nxt, fin = run_device(desc, g.Ns, token, p, q, u, noise, mode, lmax)
    c.commit(desc, dg.layers, acc, ln)                        # both publishers take the walk's device outputs
    c.kv_publish(desc, da.packed, acc, ln, da.ctx_len_out)
    torch.cuda.synchronize()

    ref = AC.accept(g.parent, g.slot, g.Ns, token, p, q, u, noise, mode=AC.GREEDY if mode == "greedy" else AC.REJECTION,
                    lmax=lmax)
    acc_h, ln_h = acc.cpu().numpy(), ln.cpu().numpy()
    assert acc_h.tolist() == ref[0].tolist() and ln_h.tolist() == ref[1].tolist()
    assert len(set(ln_h.tolist())) > 1, "the sequences should accept prefixes of different lengths"

    # attention verifier against its oracle
    k1, v1 = A.kv_write(a.slot, a.k_new, a.v_new, a.k_cache, a.v_cache, a.ctx_len, a.cache_row)
    check_attention(da, a, k1, v1, "hybrid cycle")

    # recurrent publisher: the state of the chosen path
    L = g.layers[0]
    st_ref, hist_ref, status_ref, _ = O.commit(g.parent, g.slot, g.state_row, dg.np("q"), dg.np("k"), dg.np("v"),
                                               dg.np("alpha"), dg.np("beta"), L.state, ref[0], ref[1], l2norm=True,
                                               x=L.x, hist=L.hist)
    assert dg.np("status").tolist() == status_ref.tolist() == [0] * B
    assert_close(dg.np("state"), st_ref, what="state published along the walk's path")
    assert np.array_equal(dg.np("conv_hist"), hist_ref)

    # KV publisher: the same path, re-linearised
    k2, v2, ctx2, st = A.kv_publish(a.parent, a.slot, k1, v1, a.ctx_len, a.cache_row, ref[0], ref[1])
    assert da.t("status").tolist() == st.tolist() == [0] * B
    assert np.array_equal(da.np("k_cache"), k2) and np.array_equal(da.np("v_cache"), v2)

    # every consumer selected the same materialised prefix
    assert da.ctx_len_out.tolist() == ctx2.tolist() == (a.ctx_len + ln_h).tolist()
    for b in range(B):
        n, row, cx = int(ln_h[b]), int(a.cache_row[b]), int(a.ctx_len[b])
        path = acc_h[b, :n]
        # the published cache rows are the K/V entries of exactly the nodes whose updates the state received
        assert np.array_equal(da.np("k_cache")[row, cx:cx + n], a.k_new[b, path])
        # a sequence that accepted nothing keeps its state; one that accepted something does not
        srow = g.state_row[b]
        changed = not np.array_equal(dg.np("state")[srow], S0[srow])
        assert changed == (n > 0)
        # and the pending token was drawn at the node both publishers stopped at
        assert int(fin.cpu()[b]) == (int(path[-1]) if n else -1)
