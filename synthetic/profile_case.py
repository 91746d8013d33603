"""One synthetic case through the tree scan alone, three times, each behind a 256 MiB fill that evicts L2:
the command to put under a profiler (the third launch is the one to capture).

    python -m synthetic.profile_case cfg2 gram
    python -m synthetic.profile_case cfgP direct

The operands are uploaded as recorded q, k, v (no convolution launch), q and k are normalised inside the
scan, outputs are bf16, launches do not overlap."""
import sys

import torch

from paper_2609_23900_b200 import binding
from synthetic import workload as W
from synthetic.device_case import DeviceCase

CASES = {
    "cfg2": W.config2,
    "cfg3": lambda: W.config3(n_layers=8),
    "cfg4": lambda: W.config4("random", B=8),
    "cfgP": lambda: W.config_paper(B=8),
}


def main(argv):
    cfg = argv[1] if len(argv) > 1 else "cfg2"
    algo = argv[2] if len(argv) > 2 else "auto"
    ctx = binding.Context(0)
    ctx.set_scan_algo(algo)
    ctx.set_overlap(False)
    dc = DeviceCase(ctx, CASES[cfg](), use_conv=False, qk_l2norm=True, out_dtype="bf16")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(3):
        flush.zero_()
        dc.verify()
        torch.cuda.synchronize()
    print("ok", cfg, algo)


if __name__ == "__main__":
    main(sys.argv)
