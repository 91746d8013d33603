#!/usr/bin/env python
"""Benchmark of the GDN tree verify + commit hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg2] [--impl reference]

One "step" = the whole hot path over one batch of synthetic input: tree conv + tree scan
(lumo_gdn_tree_verify) and accepted-path replay + conv-history gather (lumo_gdn_commit).
The metric is tree nodes verified per second per layer, B * N * n_layers / step time, summed
over ranks (each rank owns its own sequences: weak scaling, no collective on the data path).

Prints ONE JSON line.  `value` is timed with inputs resident in HBM (CUDA-graph replay of the
C-ABI calls, rotating over buffer sets larger than L2); `e2e` repeats the measurement through
the C-ABI calls with the step's inputs copied from pinned host memory and its outputs copied
back inside the timed region; `roofline` is the scan kernel's algorithmic bytes over its own
device time (CUDA events around each launch, taken in a second pass of K steps);
`cpu_baseline` is the fp64 oracle timed on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "gdn_tree_nodes_verified_per_s_per_layer"
UNIT = "nodes/s"
L2_BYTES = 126 * 2 ** 20


def make_case(name: str, seed_offset: int = 0):
    from synthetic import workload as W
    if name == "cfg1":
        return W.config1(seed=W.BASE_SEED + 1 + 1000 * seed_offset)
    if name == "cfg2":
        return W.config2(seed=W.BASE_SEED + 2 + 1000 * seed_offset)
    if name == "cfg3":
        return W.config3(seed=W.BASE_SEED + 3 + 1000 * seed_offset)
    if name.startswith("cfg4_"):
        return W.config4(name[5:], seed=W.BASE_SEED + 4 + 1000 * seed_offset)
    if name == "cfgP":
        return W.config_paper(seed=W.BASE_SEED + 5 + 1000 * seed_offset, B=8, n_layers=1)
    raise SystemExit(f"unknown config {name}")


WORKLOAD_TEXT = {
    "cfg1": "config 1: batch 1, 16/32 heads, d=128, 16-node MTP-spine tree, 1 layer",
    "cfg2": "config 2: serving batch 8, 16/32 heads, d=128, random 64-node trees (depth<=8), 1 layer",
    "cfg3": "config 3: 48 layers back to back, batch 4, 32-node trees (depth<=6)",
    "cfg4_chains": "config 4: batch 32, 256-node trees, 16 chains of depth 16",
    "cfg4_star": "config 4: batch 32, 256-node trees, 255-child star",
    "cfg4_random": "config 4: batch 32, 256-node trees, random depth<=12",
    "cfgP": "paper geometry: 28 active rows padded to 32, batch 8, 1 layer",
}


def rank_seed_offset(rank: int) -> int:
    """Each rank owns its own sequences (weak scaling): disjoint seed ranges per rank."""
    return rank * 64


def is_reporting_rank(rank: int) -> bool:
    return rank == 0


def max_over_ranks(ms: float, world: int, device) -> float:
    """A step is as slow as its slowest rank."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(nodes_per_rank_step: int, ms_step: float, world: int) -> float:
    """Whole-job nodes per second: every rank processed its own batch in the (max) step time."""
    return world * nodes_per_rank_step / (ms_step / 1e3)


def algorithmic_bytes(c, out_bytes=2):
    """Per layer: state read once, operands read once, outputs written once (verify);
    state read+written, accepted operands read, history rewritten (commit)."""
    B, N, Hk, Hv, d = c.B, c.N, c.Hk, c.Hv, c.d
    s_in = 2 if c.in_dtype == "bf16" else 4
    C = c.C
    state = 4 * B * Hv * d * d
    operands = B * N * C * s_in
    gates = 2 * B * N * Hv * s_in
    out = B * N * Hv * d * out_bytes
    Lsum = int(c.accepted_len.sum())
    scan = state + operands + gates + out
    conv = 2 * B * N * C * s_in + 4 * C * s_in + 3 * B * C * s_in
    commit = 2 * state + Lsum * ((Hk * d + Hv * d) * s_in + 2 * Hv * s_in) + 2 * 3 * B * C * s_in
    return dict(scan=scan, conv=conv, commit=commit)


def rank1_fma(c):
    """fp32 FMAs of the rank-1 form per layer: 2 d^2 per leaf, 3 d^2 per internal node-head."""
    total = 0
    for b in range(c.B):
        par = c.parent[b]
        internal = set(int(p) for p in par if p >= 0)
        total += (2 * (c.N - len(internal)) + 3 * len(internal)) * c.Hv * c.d * c.d
    return total


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the GPU is under load."""

    def __init__(self, index: int, period: float = 0.01):
        super().__init__(daemon=True)
        self.period, self.samples, self.reasons, self.stop_flag = period, [], set(), False
        self.max_mhz = None
        self.windows = {}
        self._tag = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def tag(self, name):
        self._tag = name

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
        }
        while not self.stop_flag:
            try:
                mhz = nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                if self._tag:
                    self.windows.setdefault(self._tag, []).append(mhz)
                    for n, bit in names.items():
                        if r & bit:
                            self.reasons.add(n)
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self):
        timed = self.windows.get("timed", [])
        allw = [m for w in self.windows.values() for m in w]
        use = timed if len(timed) >= 3 else allw
        return {"sm_mhz": statistics.median(use) if use else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(use),
                "window": "timed region" if use is timed and timed else "all load phases of this run"}


def run_oracle_steps(case, seconds: float, threads: int = 0):
    """Times the oracle, as it stands, on whole steps of the workload (conv, memo-mode scan,
    commit) for about `seconds`; returns (nodes/s/layer, steps, cores, seconds)."""
    from oracle import gdn_oracle as O
    O.build()
    n_layers = len(case.layers)
    t0 = time.perf_counter()
    steps, used = 0, 1
    while True:
        for L in case.layers:
            y = O.conv(case.parent, case.slot, case.state_row, L.x, L.conv_w, L.conv_b, L.hist, case.Ns,
                       out_dtype=case.in_dtype, threads=threads)
            hk = case.Hk * case.d
            q = y[..., :hk].reshape(case.B, case.Ns, case.Hk, case.d)
            k = y[..., hk:2 * hk].reshape(case.B, case.Ns, case.Hk, case.d)
            v = y[..., 2 * hk:].reshape(case.B, case.Ns, case.Hv, case.d)
            _, _, used = O.scan(case.parent, case.slot, case.state_row, q, k, v, L.alpha, L.beta, L.state,
                                l2norm=True, mode="memo", threads=threads)
            O.commit(case.parent, case.slot, case.state_row, q, k, v, L.alpha, L.beta, L.state, case.accepted,
                     case.accepted_len, l2norm=True, x=L.x, hist=L.hist, threads=threads)
        steps += 1
        dt = time.perf_counter() - t0
        if dt >= seconds or steps >= 1000:
            break
    return case.B * case.N * n_layers * steps / dt, steps, used, dt


def oracle_walk_mode():
    """The oracle in its literal form (every node recomputed from the pre-tree state along its ancestry,
    "walk" mode), scan only, on configs 0-2: nodes per second."""
    from oracle import gdn_oracle as O
    from synthetic import workload as W
    out = {}
    for name, case in (("cfg0", W.config0()), ("cfg1", W.config1()), ("cfg2", W.config2())):
        L = case.layers[0]
        best = None
        for _ in range(3):
            t0 = time.perf_counter()
            O.scan(case.parent, case.slot, case.state_row, L.q, L.k, L.v, L.alpha, L.beta, L.state, mode="walk")
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        out[name] = case.B * case.N / best
    return out


def reference_arm(args, rank):
    """The oracle, as it stands, on the host cores (rank 0 only)."""
    if rank != 0:
        return
    case = make_case(args.config)
    if len(case.layers) > 4:          # bounded sample: a few layers of the stack
        case.layers = case.layers[:4]
    per_step = []
    cores = 1
    for i in range(args.warmup + args.steps):
        v, steps, cores, dt = run_oracle_steps(case, seconds=0.0)
        if i >= args.warmup:
            per_step.append(dt)
        if sum(per_step) > 150:
            break
    ms = 1e3 * statistics.mean(per_step)
    nodes = case.B * case.N * len(case.layers)
    value = nodes / (ms / 1e3)
    sample = f"whole batch of {WORKLOAD_TEXT[args.config]}" + (f", first {len(case.layers)} layers" if args.config == "cfg3" else "")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(per_step), "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.config], "name": args.config},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def read_ncu_traffic(config_name):
    """dram__bytes_read.sum + dram__bytes_write.sum of one scan launch, from the ncu summary under
    profiles/ -- used only when the kernel source is still the one that capture was taken from (the
    summary records a hash of the source file); otherwise None."""
    import hashlib
    import re
    path = os.path.join(ROOT, "profiles", "scan_gram_traffic.md")
    src = os.path.join(ROOT, "paper_2609_23900_b200", "csrc", "scan_gram.cu")
    if not (os.path.exists(path) and os.path.exists(src)):
        return None
    text = open(path).read()
    sha = hashlib.sha256(open(src, "rb").read()).hexdigest()[:16]
    m = re.search(r"source-sha256:\s*([0-9a-f]{16})", text)
    t = re.search(r"traffic %s:\s*(\d+)" % re.escape(config_name), text)
    if not (m and t) or m.group(1) != sha:
        return None
    return int(t.group(1))


def measure_extra_config(ctx, name, out_dtype, peak_gbs, steps=20, warmup=3, snapshot_mode=0, n_sets=2):
    """One more configuration of the benchmark spec in the same run: whole-step throughput, per-kernel device
    time, the scan alone and the verify (conv + scan) alone from back-to-back launches, and the two
    roofline fractions.  Fewer steps than the headline so that the whole run stays within minutes."""
    import torch
    from paper_2609_23900_b200 import binding
    from synthetic.device_case import DeviceCase
    cases = [make_case(name, seed_offset=i) for i in range(n_sets)]
    c0 = cases[0]
    sets = [DeviceCase(ctx, c, out_dtype=out_dtype, snapshot_mode=snapshot_mode) for c in cases]
    packed = [binding.Context.pack(s.layers) for s in sets]
    n_layers = len(c0.layers)
    nodes = c0.B * c0.N * n_layers
    ab = algorithmic_bytes(c0, out_bytes=2 if out_dtype == "bf16" else 4)

    def run_step(i):
        s = sets[i % n_sets]
        ctx.verify(s.desc, packed[i % n_sets])
        ctx.commit(s.desc, packed[i % n_sets], s.accepted, s.accepted_len)

    for i in range(max(warmup, n_sets)):
        run_step(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        run_step(i)
    e1.record()
    torch.cuda.synchronize()
    ms_step = e0.elapsed_time(e1) / steps
    ctx.timing_enable(True)
    ctx.timing_read(reset=True)
    for i in range(steps):
        run_step(i)
    torch.cuda.synchronize()
    per_kernel = ctx.timing_read(reset=True)
    ctx.timing_enable(False)
    kern = {k: {"launches": n, "avg_us": 1e3 * ms / n} for k, (n, ms) in per_kernel.items() if n}

    def back_to_back(arrs):
        for i in range(warmup):
            ctx.verify(sets[i % n_sets].desc, arrs[i % n_sets])
        torch.cuda.synchronize()
        e0.record()
        for i in range(steps):
            ctx.verify(sets[i % n_sets].desc, arrs[i % n_sets])
        e1.record()
        torch.cuda.synchronize()
        return 1e3 * e0.elapsed_time(e1) / steps

    verify_us = back_to_back(packed)                  # conv + scan, launched as the library launches them
    scan_only = []
    for s_ in sets:
        arr = binding.Context.pack(s_.layers)
        for a in arr:
            a.x = None
        scan_only.append(arr)
    scan_us = back_to_back(scan_only)
    out = {"workload": WORKLOAD_TEXT[name], "value": nodes / (ms_step * 1e-3), "unit": UNIT, "ms_per_step": ms_step,
           "steps": steps, "warmup": max(warmup, n_sets), "buffer_sets": n_sets,
           "kernels": kern, "scan_us_back_to_back": scan_us, "verify_us_back_to_back": verify_us,
           "scan_frac_of_hbm_peak": n_layers * ab["scan"] / (scan_us * 1e-6) / 1e9 / peak_gbs,
           "verify_frac_of_hbm_peak": n_layers * ab["scan"] / (verify_us * 1e-6) / 1e9 / peak_gbs,
           "algorithmic_bytes_verify": n_layers * ab["scan"],
           "verify_nodes_per_s_per_layer": nodes / (verify_us * 1e-6),
           "commit_us_per_layer": kern["commit"]["avg_us"] / n_layers if "commit" in kern else None}
    if snapshot_mode == 2:
        snap = c0.Hv * c0.d * c0.d * 4
        out["snapshots"] = {"mode": "cached: every node state exported (snapshot_mode 2, sequential fp32 kernel)",
                            "extra_state_bytes_per_node": snap,
                            "extra_state_bytes_per_launch": snap * nodes,
                            "algorithmic_bytes_per_node": n_layers * ab["scan"] / nodes}
    del sets, packed, scan_only, cases
    torch.cuda.empty_cache()
    return out


def measure_attention(ctx, peak_gbs, steps=30, warmup=4, B=8, context=16384, Hq=32, Hkv=8, n_sets=2, with_oracle=False):
    """The attention half of the verifier on the paper's tree geometry (28 candidates + root padded to 32
    rows, spine-first slots): tree KV write, ancestry-masked decode attention and KV publication of one
    full-attention layer, timed back to back over rotating cache sets larger than L2.  The paper states no
    head counts or context lengths for its model: 32 query / 8 KV heads of 128 and a 16k-token context per
    sequence stand in for a coding-agent request.  Inputs are drawn on the
    device; parity with the oracle is the tests' business."""
    import numpy as np
    import torch
    from paper_2609_23900_b200 import binding
    from synthetic import workload as W
    dev = torch.device("cuda", ctx.device)
    tree = W.tree_paper_geometry()
    N, Ns, dh = len(tree), 32, 128
    parent = np.asarray([tree] * B, dtype=np.int32)
    slot = np.asarray([W.spine_first_slots(tree)] * B, dtype=np.int32)
    desc = ctx.tree_desc(parent, slot=slot, n_slots=Ns)
    S = context + Ns
    ctx_len = torch.full((B,), context, dtype=torch.int32, device=dev)
    ctx_out = torch.zeros((B,), dtype=torch.int32, device=dev)
    rows = torch.arange(B, dtype=torch.int32, device=dev)
    spine = [i for i in range(N) if slot[0][i] < 6][:6]                 # six accepted spine nodes: already in place
    branch = []
    i = N - 1                                                           # and a rescue branch for the odd sequences
    while i >= 0:
        branch.append(i)
        i = tree[i]
    branch = branch[::-1]
    lmax = max(len(spine), len(branch))
    acc = np.full((B, lmax), -1, dtype=np.int32)
    ln = np.zeros(B, dtype=np.int32)
    for b in range(B):
        path = spine if b % 2 == 0 else branch
        acc[b, :len(path)] = path
        ln[b] = len(path)
    acc_d, ln_d = torch.from_numpy(acc).to(dev), torch.from_numpy(ln).to(dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(20260923)
    rnd = lambda *shape: torch.randn(*shape, device=dev, dtype=torch.float32, generator=gen).to(torch.bfloat16)
    layers, packs = [], []
    for _ in range(n_sets):
        L = binding.AttnLayer(Hq=Hq, Hkv=Hkv, k_cache=rnd(B, S, Hkv, dh), v_cache=rnd(B, S, Hkv, dh), ctx_len=ctx_len,
                              cache_row=rows, scale=dh ** -0.5, q=rnd(B, N, Hq, dh), k_new=rnd(B, N, Hkv, dh),
                              v_new=rnd(B, N, Hkv, dh), out=torch.empty(B, N, Hq, dh, device=dev),
                              lse=torch.empty(B, N, Hq, device=dev), status=torch.zeros(B, dtype=torch.int32, device=dev))
        layers.append(L)
        packs.append(ctx.pack_attn([L]))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed(fn):
        # the calls are captured into one CUDA graph and the replay is timed: the short kernels (write,
        # publish) would otherwise be timed at the rate of the Python binding, not of the device
        for i in range(warmup):
            fn(i)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for i in range(steps):
                fn(i)
        g.replay()                      # once untimed
        torch.cuda.synchronize()
        e0.record()
        g.replay()
        e1.record()
        torch.cuda.synchronize()
        return 1e3 * e0.elapsed_time(e1) / steps

    attn_us = timed(lambda i: ctx.tree_attention(desc, packs[i % n_sets]))
    write_us = timed(lambda i: ctx.kv_write_tree(desc, packs[i % n_sets]))
    publish_us = timed(lambda i: ctx.kv_publish(desc, packs[i % n_sets], acc_d, ln_d, ctx_out))
    cycle_us = timed(lambda i: (ctx.kv_write_tree(desc, packs[i % n_sets]), ctx.tree_attention(desc, packs[i % n_sets]),
                                ctx.kv_publish(desc, packs[i % n_sets], acc_d, ln_d, ctx_out)))
    ctx.timing_enable(True)
    ctx.timing_read(reset=True)
    for i in range(steps):
        ctx.tree_attention(desc, packs[i % n_sets])
    torch.cuda.synchronize()
    per_kernel = ctx.timing_read(reset=True)
    ctx.timing_enable(False)
    ok = all(int(L.tensors["status"].abs().sum()) == 0 for L in layers) and all(bool(torch.isfinite(L.tensors["out"]).all()) for L in layers)
    # algorithmic bytes of one attention launch: every key and value of context and suffix once, queries, outputs
    kv = 2 * B * S * Hkv * dh * 2
    alg = kv + B * N * Hq * dh * (2 + 4) + B * N * Hq * 4
    out = {"workload": f"one full-attention layer: batch {B}, {Hq}/{Hkv} heads of {dh}, {context}-token context per sequence, "
                       f"paper tree ({N} nodes in {Ns} rows, spine-first slots), bf16 cache",
           "attention_us": attn_us, "kv_write_us": write_us, "kv_publish_us": publish_us, "write_attend_publish_us": cycle_us,
           "kernels": {k: {"launches": n, "avg_us": 1e3 * ms / n} for k, (n, ms) in per_kernel.items() if n},
           "algorithmic_bytes": alg, "achieved_gbs": alg / (attn_us * 1e-6) / 1e9,
           "frac_of_hbm_peak": alg / (attn_us * 1e-6) / 1e9 / peak_gbs,
           "tree_nodes_per_s_per_layer": B * N / (attn_us * 1e-6),
           "timing": f"{steps} back-to-back calls replayed from one CUDA graph between two CUDA events, {n_sets} cache sets of {kv // 2 ** 20} MiB each rotated (larger than L2)",
           "accepted": "even sequences accept six spine nodes (in place under the spine-first map: no bytes move), odd ones a rescue branch",
           "status_ok_and_finite": ok}
    if with_oracle:
        # error of the timed launch against the fp64 oracle on sampled (sequence, query head) pairs, every node
        # (CPU-baseline leg only: the oracle is test infrastructure)
        from oracle import attn_oracle as A
        L = layers[0]
        ctx.kv_write_tree(desc, packs[0])
        ctx.tree_attention(desc, packs[0])
        torch.cuda.synchronize()
        f64 = lambda t: t.to(torch.float64).cpu().numpy()
        outs, lses, q = f64(L.tensors["out"]), f64(L.tensors["lse"]), f64(L.tensors["q"])
        G = Hq // Hkv
        max_abs, max_ratio, max_lse_ulp, n_el = 0.0, 0.0, 0.0, 0
        for b, h in ((0, 0), (B // 2, Hq // 2 + 1), (B - 1, Hq - 1)):
            g = h // G
            k1 = f64(L.tensors["k_cache"][b:b + 1, :, g:g + 1])
            v1 = f64(L.tensors["v_cache"][b:b + 1, :, g:g + 1])
            one = lambda a_: a_[b:b + 1]
            args_ = (one(parent), one(slot), q[b:b + 1, :, h:h + 1], k1, v1, np.asarray([context]), np.zeros(1, np.int32), dh ** -0.5)
            ref, rl = A.tree_attention(*args_)
            bound, _ = A.tree_attention(args_[0], args_[1], args_[2], k1, np.abs(v1), *args_[5:])
            err = np.abs(outs[b, :, h] - ref[0, :, 0])
            max_abs = max(max_abs, float(err.max()))
            max_ratio = max(max_ratio, float((err / (2.0 ** -8 * bound[0, :, 0] + 1e-30)).max()))
            ulp = np.spacing(np.abs(rl[0, :, 0]).astype(np.float32)).astype(np.float64)
            max_lse_ulp = max(max_lse_ulp, float((np.abs(lses[b, :, h] - rl[0, :, 0]) / ulp).max()))
            n_el += err.size
        out["error_vs_fp64_oracle"] = {"sampled_outputs": n_el, "max_abs_output_error": max_abs,
                                       "max_error_over_bf16_probability_bound": max_ratio,
                                       "max_lse_error_in_fp32_ulp": max_lse_ulp,
                                       "bound": "2^-8 * sum_p softmax_p |v_p| per element (probabilities rounded to bf16)"}
    del layers, packs
    torch.cuda.empty_cache()
    return out


def fused_arm(args):
    """The same workload through lumo_gdn_commit_verify (the previous cycle's commit folded into the
    verify), timed by a run of this script of its own; reported beside the headline, never as it."""
    import subprocess
    cmd = [sys.executable, os.path.abspath(__file__), "--config", args.config, "--steps", str(args.steps), "--warmup",
           str(args.warmup), "--out-dtype", args.out_dtype, "--no-cpu-baseline", "--fused-commit"]
    if args.no_overlap:
        cmd.append("--no-overlap")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    try:
        out = subprocess.run(cmd, capture_output=True, text=True, timeout=600, env=env).stdout
        d = json.loads([l for l in out.splitlines() if l.startswith("{")][-1])
        return {"value": d["value"], "unit": d["unit"], "ms_per_step": d["ms_per_step"], "step": d["config"]["step"]}
    except Exception as e:      # an extra figure only: its failure must not cost the headline
        return {"unavailable": f"{type(e).__name__}: {e}"[:200]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="cfg2", choices=sorted(WORKLOAD_TEXT))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--no-graph", action="store_true", help="launch through the C ABI every step instead of graph replay")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-overlap", action="store_true", help="plain stream order instead of programmatic dependent launch")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--sets", type=int, default=0, help="rotating buffer sets (0 = enough to exceed L2 twice)")
    ap.add_argument("--out-dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--extra-configs", dest="extra_configs", action="store_true", default=None,
                    help="also measure configs 3 (recomputed and cached) and 4 (three shapes) in the same run "
                         "(default: on for the default workload)")
    ap.add_argument("--no-extra-configs", dest="extra_configs", action="store_false")
    ap.add_argument("--scan-algo", default="auto", choices=["auto", "rank1", "gram", "solve", "direct", "tensor"],
                    help="which scan kernel verify uses (auto = the library's choice)")
    ap.add_argument("--attention-only", action="store_true",
                    help="time only the attention layer (the 'attention' block of the default line) and print it as its own JSON line")
    ap.add_argument("--attn-batch", type=int, default=8)
    ap.add_argument("--attn-context", type=int, default=16384)
    ap.add_argument("--fused-commit", action="store_true",
                    help="time lumo_gdn_commit_verify (the previous cycle's commit folded into the verify) instead of "
                         "verify + commit; every step still commits one accepted path and verifies one tree per sequence")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    if args.extra_configs is None:
        args.extra_configs = args.config == "cfg2" and not args.no_cpu_baseline

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        reference_arm(args, rank)
        return

    import torch
    import torch.distributed as dist
    from paper_2609_23900_b200 import binding
    from synthetic.device_case import DeviceCase

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the GDN tree verifier has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    ctx = binding.Context(local)
    ctx.set_overlap(not args.no_overlap)
    ctx.set_scan_algo(args.scan_algo)
    if args.attention_only:
        # the attention layer alone (used for profiling that kernel); not the headline metric
        if is_reporting_rank(rank):
            peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
            peak = float(json.load(open(peaks_path))["hbm_gbs"]) if os.path.exists(peaks_path) else 6650.0
            print(json.dumps({"attention": measure_attention(ctx, peak, steps=args.steps, warmup=args.warmup, B=args.attn_batch,
                                                             context=args.attn_context)}), flush=True)
        if world > 1:
            dist.destroy_process_group()
        return
    # ---- buffer sets: distinct seeds per set and per rank, together larger than L2 -----------
    case0 = make_case(args.config, seed_offset=rank_seed_offset(rank))
    n_layers = len(case0.layers)
    ab = algorithmic_bytes(case0, out_bytes=2 if args.out_dtype == "bf16" else 4)
    set_bytes = n_layers * (ab["scan"] + ab["conv"] // 2)
    n_sets = args.sets or max(2, min(16, -(-3 * L2_BYTES // set_bytes)))
    cases = [case0] + [make_case(args.config, seed_offset=rank_seed_offset(rank) + i) for i in range(1, n_sets)]
    sets = [DeviceCase(ctx, c, out_dtype=args.out_dtype, pinned_host=(i < 4)) for i, c in enumerate(cases)]
    packed = [binding.Context.pack(s.layers) for s in sets]
    nodes_per_step = case0.B * case0.N * n_layers

    prev_sets, prev_packed = [], []
    if args.fused_commit:
        # a previous cycle per set (another tree and other inputs over the same sequences), sharing the
        # set's state, history and row tensors; its operands are recorded once, outside the timed region
        for i, s_ in enumerate(sets):
            pc = make_case(args.config, seed_offset=rank_seed_offset(rank) + 1000 + i)
            pc.state_row = s_.case.state_row.copy()
            pd = DeviceCase(ctx, pc, out_dtype=args.out_dtype)
            shared = []
            for l, layer in enumerate(pd.layers):
                t = dict(layer.tensors)
                t.update(state=s_.t("state", l), conv_hist=s_.t("conv_hist", l), state_row=s_.state_row)
                shared.append(binding.GdnLayer(Hk=pc.Hk, Hv=pc.Hv, d=pc.d, scale=pd.scale, qk_l2norm=pd.qk_l2norm,
                                               l2_eps=pd.l2_eps, **t))
            pd.layers = shared
            pd.verify()
            prev_sets.append(pd)
            prev_packed.append(binding.Context.pack(shared))
        torch.cuda.synchronize()

    def run_step(i):
        s = sets[i % n_sets]
        if args.fused_commit:
            p_ = prev_sets[i % n_sets]
            ctx.commit_verify(p_.desc, prev_packed[i % n_sets], p_.accepted, p_.accepted_len, s.desc, packed[i % n_sets])
            return
        ctx.verify(s.desc, packed[i % n_sets])
        ctx.commit(s.desc, packed[i % n_sets], s.accepted, s.accepted_len)

    for i in range(n_sets):          # first calls size the library scratch
        run_step(i)
    torch.cuda.synchronize()

    launch_mode = "c_abi_direct"
    graphs = None
    if not args.no_graph:
        try:
            graphs = []
            for i in range(n_sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    run_step(i)
                graphs.append(g)
            launch_mode = "cuda_graph_replay_of_c_abi_calls"
        except Exception as e:  # capture is an optimisation of the launch path only
            graphs = None
            launch_mode = f"c_abi_direct (graph capture failed: {type(e).__name__})"
            torch.cuda.synchronize()

    def step(i):
        if graphs is not None:
            graphs[i % n_sets].replay()
        else:
            run_step(i)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()
    sampler.tag("warmup")
    for i in range(args.warmup):
        step(i)
    # ---- timed region: K steps, inputs resident in HBM ------------------------------------
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.tag("timed")
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    barrier()
    sampler.tag("per_kernel")
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), world, dev)
    ms_step = ms_total / args.steps
    value = aggregate_value(nodes_per_step, ms_step, world)

    # ---- per-kernel device time: second pass, events around every launch -------------------
    ctx.timing_enable(True)
    ctx.timing_read(reset=True)
    n_timed = min(args.steps, 2000)
    for i in range(n_timed):
        run_step(i)
    torch.cuda.synchronize()
    per_kernel = ctx.timing_read(reset=True)
    ctx.timing_enable(False)
    kern = {k: {"launches": n, "avg_us": 1e3 * ms / n} for k, (n, ms) in per_kernel.items() if n}
    # The event bracket adds a few microseconds to every launch.  The scan kernel can also be launched
    # alone (verify without x runs only the scan, on the operands the conv recorded), so its launch
    # duration is taken again from back-to-back launches between two events, same rotation of sets.
    scan_only = []
    for s_ in sets:
        arr = binding.Context.pack(s_.layers)
        for a in arr:
            a.x = None
        scan_only.append(arr)
    ctx.set_overlap(False)          # plain stream order: consecutive launches must not overlap here
    for i in range(args.warmup):
        ctx.verify(sets[i % n_sets].desc, scan_only[i % n_sets])
    torch.cuda.synchronize()
    k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    k0.record()
    for i in range(n_timed):
        ctx.verify(sets[i % n_sets].desc, scan_only[i % n_sets])
    k1.record()
    torch.cuda.synchronize()
    kern["scan"]["avg_us_back_to_back"] = 1e3 * k0.elapsed_time(k1) / n_timed
    ctx.set_overlap(not args.no_overlap)
    # the same launches as the library issues them by default (each a programmatic dependent of the one before:
    # its prologue and state requests run under the predecessor's tail); reported beside, never as, the figure above
    for i in range(args.warmup):
        ctx.verify(sets[i % n_sets].desc, scan_only[i % n_sets])
    torch.cuda.synchronize()
    k0.record()
    for i in range(n_timed):
        ctx.verify(sets[i % n_sets].desc, scan_only[i % n_sets])
    k1.record()
    torch.cuda.synchronize()
    kern["scan"]["avg_us_back_to_back_overlapped"] = 1e3 * k0.elapsed_time(k1) / n_timed
    # the whole verify (conv + scan as the library launches them, kernel overlap included), back to back
    for i in range(args.warmup):
        ctx.verify(sets[i % n_sets].desc, packed[i % n_sets])
    torch.cuda.synchronize()
    k0.record()
    for i in range(n_timed):
        ctx.verify(sets[i % n_sets].desc, packed[i % n_sets])
    k1.record()
    torch.cuda.synchronize()
    verify_b2b_us = 1e3 * k0.elapsed_time(k1) / n_timed

    # ---- end to end: inputs from pinned host memory, outputs back to the host --------------
    sampler.tag("e2e")
    hs = [s for s in sets if s.host]
    out_host = [[torch.empty_like(l.tensors["out"], device="cpu").pin_memory() for l in s.layers] for s in hs]
    st_host = [torch.empty((case0.B,), dtype=torch.int32).pin_memory() for _ in hs]
    acc_host = [(s.accepted.cpu().pin_memory(), s.accepted_len.cpu().pin_memory()) for s in hs]

    # three streams: copy-in, compute, copy-out; a buffer set is reused only after its previous
    # results have left the device, so step i+1's inputs arrive while step i computes and step i-1's
    # outputs leave
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in hs]
    ev_cmp = [torch.cuda.Event() for _ in hs]
    ev_out = [torch.cuda.Event() for _ in hs]

    def e2e_step(i):
        j = i % len(hs)
        s = hs[j]
        with torch.cuda.stream(s_in):
            s_in.wait_event(ev_out[j])
            for l, h in zip(s.layers, s.host):
                for name, src in h.items():
                    l.tensors[name].copy_(src, non_blocking=True)
            s.accepted.copy_(acc_host[j][0], non_blocking=True)
            s.accepted_len.copy_(acc_host[j][1], non_blocking=True)
            ev_in[j].record(s_in)
        with torch.cuda.stream(s_cmp):
            s_cmp.wait_event(ev_in[j])
            ctx.verify(s.desc, packed[j])
            ctx.commit(s.desc, packed[j], s.accepted, s.accepted_len)
            ev_cmp[j].record(s_cmp)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_cmp[j])
            for l, oh in zip(s.layers, out_host[j]):
                oh.copy_(l.tensors["out"], non_blocking=True)
            st_host[j].copy_(s.layers[-1].tensors["status"], non_blocking=True)
            ev_out[j].record(s_out)

    h2d = sum(sum(t.numel() * t.element_size() for t in h.values()) for h in hs[0].host) \
        + acc_host[0][0].numel() * 4 + acc_host[0][1].numel() * 4
    d2h = sum(o.numel() * o.element_size() for o in out_host[0]) + st_host[0].numel() * 4
    for i in range(2 * len(hs)):
        e2e_step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n_e2e = min(args.steps, 200)
    e0.record(s_in)
    for i in range(n_e2e):
        e2e_step(i)
    s_out.wait_stream(s_in)
    s_out.wait_stream(s_cmp)
    e1.record(s_out)
    barrier()
    ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev)
    e2e_value = aggregate_value(nodes_per_step, ms_e2e / n_e2e, world)
    sampler.stop_flag = True
    sampler.join(timeout=1.0)

    if not is_reporting_rank(rank):
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel -----------------------------------------------------
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        with open(peaks_path) as f:
            peak_gbs, peak_src = float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    else:
        peak_gbs, peak_src = 6650.0, "fallback (earlier measurement on this pool)"
    dominant = max(kern, key=lambda k: kern[k]["launches"] * kern[k]["avg_us"])
    dom_us = kern[dominant].get("avg_us_back_to_back", kern[dominant]["avg_us"])
    achieved = n_layers * ab[dominant] / (dom_us * 1e-6) / 1e9
    clocks = sampler.summary()
    fma = rank1_fma(case0) * n_layers
    sm_mhz = clocks["sm_mhz"] or 1965.0
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak_gbs, "unit": "GB/s",
                "frac": achieved / peak_gbs, "peak_source": peak_src,
                "traffic": read_ncu_traffic(args.config) if dominant == "scan" and args.scan_algo in ("auto", "gram") else None,
                "traffic_source": "profiles/scan_gram_traffic.md (one ncu capture of this kernel source; null when the source changed since)",
                "algorithmic_bytes_per_launch": n_layers * ab[dominant],
                "avg_launch_us": dom_us,
                "frac_of_8TBs_nominal": achieved / 8000.0,
                "timing": ("K back-to-back launches of this kernel alone between two CUDA events on the launch stream "
                           "(buffer sets rotated as in the timed region)") if "avg_us_back_to_back" in kern[dominant]
                else "CUDA events around each launch on the launch stream, second pass of the same steps",
                "fp32_fma_per_launch_rank1": fma,
                "alu_frac_at_sampled_clock": (fma / (kern["scan"]["avg_us"] * 1e-6)) / (148 * 128 * sm_mhz * 1e6)
                if "scan" in kern else None}
    commit_us = kern["commit"]["avg_us"] / n_layers if "commit" in kern else None
    verify_us = sum(kern[k]["avg_us"] for k in ("conv", "scan") if k in kern)
    # the metric's own unit: algorithmic bytes of the verify over the time of the whole verify (conv + scan)
    verify_achieved = n_layers * ab["scan"] / (verify_b2b_us * 1e-6) / 1e9
    if "avg_us_back_to_back_overlapped" in kern.get("scan", {}):
        ov_us = kern["scan"]["avg_us_back_to_back_overlapped"]
        roofline["scan_overlapped_launches"] = {
            "us": ov_us, "frac": n_layers * ab["scan"] / (ov_us * 1e-6) / 1e9 / peak_gbs,
            "note": "throughput of consecutive scan launches with the library's default launch overlap; "
                    "roofline.frac itself is taken from launches that do not overlap"}
    roofline["verify_level"] = {"algorithmic_bytes": n_layers * ab["scan"], "us": verify_b2b_us, "achieved": verify_achieved,
                                "frac": verify_achieved / peak_gbs, "unit": "GB/s",
                                "timing": "K back-to-back lumo_gdn_tree_verify calls (conv + scan) between two CUDA events"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.config], "name": args.config, "batch_per_gpu": case0.B,
                       "nodes_per_tree": case0.N, "layers": n_layers, "heads_qk_v": [case0.Hk, case0.Hv],
                       "d": case0.d, "in_dtype": case0.in_dtype, "out_dtype": args.out_dtype, "state": "f32",
                       "pipeline": "conv+silu -> l2norm(q,k) -> tree scan; commit state + conv history",
                       "l2": f"rotating over {n_sets} buffer sets ({n_sets * set_bytes / 2**20:.0f} MiB) larger than L2",
                       "launch": launch_mode, "step": ("commit of the previous cycle folded into the verify (lumo_gdn_commit_verify)" if args.fused_commit else "verify, then commit"), "kernel_overlap": "programmatic dependent launch" if not args.no_overlap else "off", "parallelism": "replicas" if world > 1 else "single gpu",
                       "mean_accepted_len": float(case0.accepted_len.mean())},
            "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons", "samples", "window")},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                    "ms_per_step": ms_e2e / n_e2e, "steps": n_e2e,
                    "how": "C-ABI calls with the step's x, gates and accepted path copied from pinned host memory and "
                           "outputs + status copied back, every step; copy-in, compute and copy-out on three streams"},
            "gpu_launches": int(args.steps * sum(1 for k in ("conv", "scan", "commit") if k in kern)),
            "roofline": roofline,
            "kernels": kern,
            "verify_nodes_per_s_per_layer": nodes_per_step / (verify_b2b_us * 1e-6),
            "verify_us_per_layer": verify_b2b_us / n_layers, "verify_us_per_layer_event_bracketed": verify_us / n_layers,
            "commit_us_per_layer": commit_us,
            "scratch_bytes": ctx.scratch_bytes}

    if world == 1 and not args.no_cpu_baseline:
        sample_case = case0
        sample = "whole batch of the same workload, every step = conv + memo-mode scan + commit"
        if n_layers > 2:
            import copy
            sample_case = copy.copy(case0)
            sample_case.layers = case0.layers[:2]
            sample += ", first 2 layers"
        # best of three slices of the time budget (the oracle as it stands, memo mode)
        runs = [run_oracle_steps(sample_case, args.cpu_seconds / 3.0) for _ in range(3)]
        v, steps, cores, dt = max(runs, key=lambda r: r[0])
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{sample}; best of 3 slices, {steps} steps in {dt:.1f} s",
                                "walk_mode_scan_nodes_per_s": oracle_walk_mode()}
        # the paper's paired error rule, counted for the tensor-core scans against the library's sequential
        # recurrence (needs the fp64 oracle, hence in this leg); one layer of the headline workload
        try:
            from tests.paired_rule import paired_rule
            pc = make_case(args.config, seed_offset=rank_seed_offset(rank))
            if len(pc.layers) > 1:
                pc.layers = pc.layers[:1]
            line["paired_rule"] = paired_rule(ctx, pc, with_commit_chain=False)
            line["paired_rule"]["rule"] = "E_tree <= 1.10 E_native + 2^-24 M_64 + 2^-149 per cell (sequence, node, value head), rms and max"
        except Exception as e:      # an extra figure only
            line["paired_rule"] = {"unavailable": f"{type(e).__name__}: {e}"[:200]}
    if world == 1 and not args.fused_commit and not args.no_cpu_baseline:
        line["fused_commit_verify"] = fused_arm(args)
    if world == 1 and args.extra_configs and not args.fused_commit:
        # the other configurations of the target in the same run (fewer steps each; configs 3 and 4)
        extra = {}
        plan = [("cfg3", "cfg3_recomputed", 0, 10, 2), ("cfg3", "cfg3_cached", 2, 4, 1),
                ("cfg4_chains", "cfg4_chains", 0, 15, 2), ("cfg4_star", "cfg4_star", 0, 15, 2),
                ("cfg4_random", "cfg4_random", 0, 15, 2)]
        for name, key, snap, k_steps, k_sets in plan:
            if name == args.config and snap == 0:
                continue
            try:
                extra[key] = measure_extra_config(ctx, name, args.out_dtype, peak_gbs, steps=k_steps, snapshot_mode=snap,
                                                  n_sets=k_sets)
            except Exception as e:
                extra[key] = {"unavailable": f"{type(e).__name__}: {e}"[:200]}
        line["configs"] = extra
        try:
            line["attention"] = measure_attention(ctx, peak_gbs, with_oracle=not args.no_cpu_baseline)
        except Exception as e:
            line["attention"] = {"unavailable": f"{type(e).__name__}: {e}"[:200]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
