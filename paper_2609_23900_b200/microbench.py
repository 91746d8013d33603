"""Device-time microbenchmarks of the two steps around the verifier: the fused draft selection
(lumo_select_spine_top3) and the acceptance walk (lumo_tree_accept).

    python -m paper_2609_23900_b200.microbench select [--rows R] [--vocab V] [--dtype bf16|f32] [--split S]
    python -m paper_2609_23900_b200.microbench accept [--vocab V] [--mode greedy|rejection]

Each call is captured in a CUDA graph over several input sets (together larger than L2 when the
workload allows it) and timed with CUDA events on the launch stream; prints one JSON line."""
import argparse
import json

import numpy as np
import torch

from . import binding
from . import workload as W


def _time_graph(launch_all, n_calls, reps):
    for _ in range(2):
        launch_all()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        launch_all()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / (reps * n_calls)          # us per call


def bench_select(args):
    ctx = binding.Context(0)
    dev = torch.device("cuda", 0)
    dtype = {"bf16": torch.bfloat16, "f32": torch.float32}[args.dtype]
    nbytes = args.rows * args.vocab * (2 if args.dtype == "bf16" else 4)
    n_sets = int(min(16, max(2, 400e6 // nbytes + 1)))          # rotate over > 3 x L2 when rows are many
    gen = torch.Generator(device=dev).manual_seed(1)
    sets = [torch.randn((args.rows, args.vocab), device=dev, generator=gen).to(dtype) for _ in range(n_sets)]
    spine = torch.zeros((args.rows,), dtype=torch.int32, device=dev)
    cand = torch.zeros((args.rows, 3), dtype=torch.int32, device=dev)

    def launch_all():
        st = torch.cuda.current_stream()
        for s in sets:
            ctx.select_spine_top3(s, spine, cand, split=args.split, stream=st)

    us = _time_graph(launch_all, n_sets, args.reps)
    print(json.dumps({"kernel": "select_spine_top3", "rows": args.rows, "vocab": args.vocab, "dtype": args.dtype,
                      "split": args.split, "us_per_call": us, "bytes_per_call": nbytes, "GBps": nbytes / us / 1e3,
                      "input_sets": n_sets}))


def bench_accept(args):
    ctx = binding.Context(0)
    dev = torch.device("cuda", 0)
    c = W.config2()
    V, B, Ns = args.vocab, c.B, c.Ns
    rs = np.random.default_rng(0)
    # cheap synthetic rows at full vocabulary size: normalised squares of normals
    p = rs.standard_normal((B, Ns + 1, V)).astype(np.float32) ** 2
    p /= p.sum(-1, keepdims=True)
    q = rs.standard_normal((B, Ns, V)).astype(np.float32) ** 2
    q /= q.sum(-1, keepdims=True)
    token = rs.integers(0, V, size=(B, Ns)).astype(np.int32)
    for b in range(B):
        for i in range(c.N):
            prow = Ns if c.parent[b, i] < 0 else c.slot[b, c.parent[b, i]]
            if rs.uniform() < 0.6:                                # a fair share of candidates is accepted
                token[b, c.slot[b, i]] = int(np.argmax(p[b, prow]))
    u = rs.uniform(size=(B, Ns)).astype(np.float32)
    noise = rs.exponential(size=(B, V)).astype(np.float32) + np.float32(1e-6)
    up = lambda a: torch.from_numpy(a).to(dev)
    desc = ctx.tree_desc(c.parent, slot=c.slot, n_slots=c.Ns)
    t = dict(token=up(token), p_target=up(p), q_draft=up(q), uniforms=up(u), noise=up(noise),
             work=torch.empty((B, V), device=dev))
    lmax = max(max(W.tree_depths(pp.tolist())) for pp in c.parent) + 1
    acc = torch.zeros((B, lmax), dtype=torch.int32, device=dev)
    ln, nx, fn = (torch.zeros((B,), dtype=torch.int32, device=dev) for _ in range(3))

    def launch_all():
        st = torch.cuda.current_stream()
        for _ in range(8):
            ctx.accept(desc, accepted=acc, length=ln, next_token=nx, final_node=fn, mode=args.mode, stream=st, **t)

    us = _time_graph(launch_all, 8, args.reps)
    print(json.dumps({"kernel": "tree_accept", "mode": args.mode, "batch": B, "nodes": c.N, "vocab": V,
                      "us_per_call": us, "accepted_lengths": ln.tolist()}))


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    sub = ap.add_subparsers(dest="which", required=True)
    s = sub.add_parser("select")
    s.add_argument("--rows", type=int, default=32)
    s.add_argument("--vocab", type=int, default=151936)
    s.add_argument("--dtype", choices=["bf16", "f32"], default="bf16")
    s.add_argument("--split", type=int, default=0)
    s.add_argument("--reps", type=int, default=20)
    a = sub.add_parser("accept")
    a.add_argument("--vocab", type=int, default=151936)
    a.add_argument("--mode", choices=["greedy", "rejection"], default="greedy")
    a.add_argument("--reps", type=int, default=20)
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("microbench needs a CUDA device")
    (bench_select if args.which == "select" else bench_accept)(args)


if __name__ == "__main__":
    main()
