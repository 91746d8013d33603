"""Writes tests/golden/cfg0_oracle.json: values of the fp64 oracle on the smallest configuration.

The paper prints no worked numeric example, so these are not the paper's numbers: they are a
tripwire for unintended changes of the oracle's arithmetic or of the input generator (a deliberate
change regenerates the file and says why in its commit message).  Calls only oracle/ and the input
generator; nothing here comes from the CUDA path.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import gdn_oracle as O          # noqa: E402
from oracle import tree_tables as T         # noqa: E402
from synthetic import workload as W   # noqa: E402


def compute():
    c = W.config0()
    L = c.layers[0]
    y = O.conv(c.parent, c.slot, c.state_row, L.x, L.conv_w, L.conv_b, L.hist, c.Ns, out_dtype="f32")
    o, snap, _ = O.scan(c.parent, c.slot, c.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state,
                        mode="walk", snap_nodes=[[6]])
    st, hist, status, _ = O.commit(c.parent, c.slot, c.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state,
                                   c.accepted, c.accepted_len, x=L.x, hist=L.hist)
    return {
        "what": "fp64 oracle on configuration 0 (7-node tree, 2 heads, d=64, fp32 inputs), scan-only operands",
        "accepted_path": c.accepted[0].tolist(),
        "tables": T.all_tables(c.parent[0].tolist(), c.slot[0].tolist(), c.Ns),
        "out_node6_head0_first8": o[0, 6, 0, :8].tolist(),
        "out_node3_head1_first8": o[0, 3, 1, :8].tolist(),
        "out_abs_sum": float(np.abs(o).sum()),
        "state_node6_head0_row0_first4": snap[0, 0, 0, 0, :4].tolist(),
        "committed_state_abs_sum": float(np.abs(st).sum()),
        "committed_equals_node6_state": bool(np.array_equal(st[c.state_row[0]], snap[0, 0])),
        "conv_row6_first6": y[0, 6, :6].tolist(),
        "conv_abs_sum": float(np.abs(y).sum()),
        "status": status.tolist(),
    }


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg0_oracle.json")
    with open(path, "w") as f:
        json.dump(compute(), f, indent=1)
    print("wrote", path)
