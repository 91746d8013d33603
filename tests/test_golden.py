"""The stored oracle values of configuration 0 (tests/golden/cfg0_oracle.json, written by
tests/golden/make_golden.py from the oracle alone) are reproduced by the oracle and, on a GPU,
matched by the CUDA path within the parity tolerance."""
import importlib.util
import json
import os

import numpy as np
import pytest

HERE = os.path.dirname(os.path.abspath(__file__))
GOLD = json.load(open(os.path.join(HERE, "golden", "cfg0_oracle.json")))


def test_oracle_reproduces_stored_values():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.compute()
    assert now["accepted_path"] == GOLD["accepted_path"] == [0, 2, 6]
    assert now["tables"] == GOLD["tables"] and now["status"] == GOLD["status"] == [0]
    assert GOLD["committed_equals_node6_state"] and now["committed_equals_node6_state"]
    for key, val in GOLD.items():
        if isinstance(val, float):
            assert abs(now[key] - val) <= 1e-12 * (1 + abs(val)), key
        elif isinstance(val, list) and val and isinstance(val[0], float):
            np.testing.assert_allclose(now[key], val, rtol=1e-12, atol=1e-15, err_msg=key)


@pytest.mark.gpu
def test_cuda_path_matches_stored_values():
    import torch
    from synthetic import workload as W
    from synthetic.device_case import DeviceCase
    from tests.harness import ctx
    c = W.config0()
    dc = DeviceCase(ctx("auto"), c, use_conv=False, snapshot_mode=1, snap_nodes=[[6]])
    dc.verify()
    dc.commit()
    torch.cuda.synchronize()
    o, st, snap = dc.np("out"), dc.np("state"), dc.np("snap_out")
    tol = lambda ref: 1e-3 * (1 + np.abs(np.asarray(ref)))
    assert np.all(np.abs(o[0, 6, 0, :8] - GOLD["out_node6_head0_first8"]) <= tol(GOLD["out_node6_head0_first8"]))
    assert np.all(np.abs(o[0, 3, 1, :8] - GOLD["out_node3_head1_first8"]) <= tol(GOLD["out_node3_head1_first8"]))
    assert np.all(np.abs(snap[0, 0, 0, 0, :4] - GOLD["state_node6_head0_row0_first4"]) <= tol(GOLD["state_node6_head0_row0_first4"]))
    assert abs(np.abs(o).sum() - GOLD["out_abs_sum"]) <= 1e-3 * GOLD["out_abs_sum"]
    assert abs(np.abs(st).sum() - GOLD["committed_state_abs_sum"]) <= 1e-3 * GOLD["committed_state_abs_sum"]
    dcv = DeviceCase(ctx("auto"), c)          # conv pipeline, operands recorded in fp32
    dcv.verify()
    torch.cuda.synchronize()
    hk = c.Hk * c.d
    y = np.concatenate([dcv.np("q").reshape(1, 7, hk), dcv.np("k").reshape(1, 7, hk), dcv.np("v").reshape(1, 7, -1)], -1)
    assert np.all(np.abs(y[0, 6, :6] - GOLD["conv_row6_first6"]) <= tol(GOLD["conv_row6_first6"]))
