"""The N>1 launch path of bench.py on CPU: two gloo ranks agree on the max-over-ranks time,
own different sequences (weak scaling, no data-path collective) and only rank 0 reports."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, os.environ["LUMO_ROOT"])
import torch, torch.distributed as dist
import bench
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
case = bench.make_case("cfg1", seed_offset=bench.rank_seed_offset(rank))
ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
agg = bench.aggregate_value(case.B * case.N * len(case.layers), ms, world)
print(json.dumps({"rank": rank, "ms": ms, "value": agg, "seed": case.seed,
                  "parent": case.parent.tolist(), "reports": bench.is_reporting_rank(rank)}))
dist.barrier()
dist.destroy_process_group()
"""


def test_two_gloo_ranks_shard_by_sequence_and_reduce_time_by_max(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, LUMO_ROOT=ROOT, MASTER_ADDR="127.0.0.1", MASTER_PORT="29533", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    a, b = sorted(outs, key=lambda o: o["rank"])
    assert a["ms"] == b["ms"] == 15.0                       # max over ranks
    assert a["value"] == b["value"] == 2 * 16 / 15e-3       # whole-job nodes per second
    assert a["seed"] != b["seed"]                           # each rank owns its own sequences
    assert a["reports"] and not b["reports"]
