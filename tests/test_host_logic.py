"""CPU-side checks of the C-ABI library: it loads, exports every symbol the header declares,
builds bit-exact integer tables on a host-only context, produces a valid scan schedule, returns
the documented error codes, and refuses to launch without a GPU (no CPU fallback)."""
import ctypes
import os
import random
import re

import numpy as np
import pytest

import __graft_entry__ as entry

entry.build()

from oracle import tree_tables as T                      # noqa: E402
from paper_2609_23900_b200 import binding               # noqa: E402
from synthetic import workload as W         # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "lumo_gdn.h")).read()
    declared = set(re.findall(r"\b(lumo_[a-z0-9_]+)\s*\(", hdr))
    assert {"lumo_tree_desc_create", "lumo_gdn_tree_verify", "lumo_gdn_commit"} <= declared
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} is declared in lumo_gdn.h but not exported"
    assert declared == set(binding.EXPORTS)


def _rand_tree(rng, n):
    return [rng.randint(-1, i - 1) for i in range(n)]


@pytest.mark.parametrize("seed", range(12))
def test_tables_bit_exact_against_oracle_on_host_only_context(seed):
    rng = random.Random(seed)
    ctx = binding.Context(-1)
    B = 3
    n = rng.choice([1, 2, 7, 31, 64, 200, 256])
    Ns = n + rng.choice([0, 0, 5])
    parents = [_rand_tree(rng, n) if seed % 3 else W.tree_random(W.IntStream(seed * 7 + b), n, 9) for b in range(B)]
    slots = [rng.sample(range(Ns), n) for _ in range(B)]
    desc = ctx.tree_desc(np.array(parents, dtype=np.int32), slot=np.array(slots, dtype=np.int32), n_slots=Ns,
                         depth=np.array([T.depth(p) for p in parents], dtype=np.int32))
    for b in range(B):
        ref = T.all_tables(parents[b], slots[b], Ns)
        for key, val in ref.items():
            assert desc.table(key, b).tolist() == val, (key, b)


def _simulate(parent, ops, full):
    """Symbolic run of the op list: registers hold 'the state of node X' (-1 = pre-tree)."""
    regs, stack, emitted, cached, states = -1, {}, [], set(), []
    for op in ops:
        kind, flag, arg = op >> 24, (op >> 20) & 1, op & 0xFFFF
        if kind in (0, 1):      # EMIT / EMIT_DESCEND
            assert parent[arg] == regs, "output computed from a state that is not the parent's"
            emitted.append(arg)
            if flag:
                cached.add(arg)
            if kind == 1:
                regs = arg
                states.append(arg)
        elif kind == 2:         # DESCEND
            assert parent[arg] == regs and arg in cached and arg in emitted
            cached.discard(arg)
            regs = arg
            states.append(arg)
        elif kind == 3:         # PUSH
            stack[arg] = regs
        elif kind == 4:         # POP
            regs = -1 if arg == 0xFFFF else stack[arg]
        else:
            raise AssertionError("unknown op")
    n = len(parent)
    assert sorted(emitted) == list(range(n)), "every node is emitted exactly once"
    internal = sorted(set(p for p in parent if p >= 0))
    assert sorted(states) == (list(range(n)) if full else internal)
    assert not cached


@pytest.mark.parametrize("seed", range(15))
def test_scan_schedule_is_a_valid_depth_first_walk(seed):
    rng = random.Random(100 + seed)
    n = rng.choice([1, 5, 16, 64, 256])
    parent = _rand_tree(rng, n) if seed % 2 else W.tree_random(W.IntStream(seed), n, 12)
    if seed == 0:
        parent = W.tree_star(64)
    if seed == 2:
        parent = W.tree_chains(16, 16)
    desc = binding.Context(-1).tree_desc(np.array([parent], dtype=np.int32))
    _simulate(parent, desc.table("schedule").tolist(), full=False)
    _simulate(parent, desc.table("schedule_full").tolist(), full=True)
    # leaves never materialise a state in the lean schedule: 2 passes instead of 3
    lean = desc.table("schedule").tolist()
    assert sum(1 for o in lean if (o >> 24) in (1, 2)) == len(set(p for p in parent if p >= 0))


@pytest.mark.parametrize("seed", range(12))
def test_gram_groups_partition_the_tree(seed):
    rng = random.Random(300 + seed)
    n = rng.choice([1, 40, 64, 65, 130, 256])
    shapes = [W.tree_star(n), W.tree_chains(max(1, n // 16), 16) if n >= 16 else W.tree_chain(n),
              W.tree_random(W.IntStream(seed), n, 12), W.tree_random(W.IntStream(seed + 50), n, 16, max_children=2)]
    parent = shapes[seed % 4]
    n = len(parent)
    desc = binding.Context(-1).tree_desc(np.array([parent], dtype=np.int32))
    tab = desc.table("gram_groups").tolist()
    depth = T.depth(parent)
    G, pos = tab[0], 1
    emitted = [0] * n
    member_once = [0] * n
    for _ in range(G):
        cnt = tab[pos]
        nodes, emit = tab[pos + 1:pos + 1 + cnt], tab[pos + 1 + cnt:pos + 1 + 2 * cnt]
        pos += 1 + 2 * cnt
        assert 1 <= cnt <= 64
        assert nodes == sorted(nodes, key=lambda x: (depth[x], x)) and len(set(nodes)) == cnt
        inside = set(nodes)
        for x, e in zip(nodes, emit):
            assert parent[x] == -1 or parent[x] in inside       # self-contained: all ancestors are members
            emitted[x] += e
    assert pos == len(tab) and emitted == [1] * n               # every node is written exactly once
    if n <= 64:
        assert G == 1
    # packing quality: prefix recomputation keeps the count near the lower bound ceil(n / 64)
    assert G <= (3 * ((n + 63) // 64) + 1) // 2 + 1
    # a tree deeper than 16 has no groups (the rank-1 kernel takes it)
    deep = binding.Context(-1).tree_desc(np.array([W.tree_chain(17)], dtype=np.int32))
    assert deep.table("gram_groups").tolist() == []


def test_error_codes_and_no_cpu_fallback():
    ctx = binding.Context(-1)
    for bad in ([[0]], [[-1, 1]], [[-1, -2]], [[-1, 0, 3, 1]]):
        with pytest.raises(binding.LumoError) as e:
            ctx.tree_desc(np.array(bad, dtype=np.int32))
        assert e.value.code == 2
    with pytest.raises(binding.LumoError) as e:
        ctx.tree_desc(np.array([[-1, 0]], dtype=np.int32), slot=np.array([[0, 0]], dtype=np.int32))
    assert e.value.code == 2
    with pytest.raises(binding.LumoError) as e:
        ctx.tree_desc(np.array([[-1, 0]], dtype=np.int32), depth=np.array([[1, 1]], dtype=np.int32))
    assert e.value.code == 2
    with pytest.raises(binding.LumoError) as e:
        ctx.tree_desc(np.zeros((1, 300), dtype=np.int32) - 1)
    assert e.value.code == 1
    # a host-only context refuses every launch; a device context without a GPU cannot be made
    desc = ctx.tree_desc(np.array([[-1, 0]], dtype=np.int32))
    arr = (binding._Args * 1)()
    rc = binding._lib.lumo_gdn_tree_verify(ctx._h, desc._h, arr, 1, None)
    assert rc == 4
    rc = binding._lib.lumo_gdn_commit(ctx._h, desc._h, arr, 1, None, None, 1, None)
    assert rc == 4
    rc = binding._lib.lumo_gdn_tree_scan_static(ctx._h, desc._h, arr, 1, None)
    assert rc == 4
    # a path bound beyond 256 nodes (the kernels stage the path in arrays of that size) or below 1 is
    # refused on the host, before anything is looked at or enqueued
    for bad_lmax in (0, -3, 257, 300, 1 << 20):
        assert binding._lib.lumo_gdn_commit(ctx._h, desc._h, arr, 1, None, None, bad_lmax, None) == 1
        assert b"lmax" in binding._lib.lumo_last_error(ctx._h)
        assert binding._lib.lumo_gdn_commit_verify(ctx._h, desc._h, arr, None, None, bad_lmax, desc._h, arr, 1, None) == 1
    assert binding._lib.lumo_gdn_commit(ctx._h, desc._h, arr, 1, None, None, 256, None) == 4
    assert binding._lib.lumo_conv_rows_per_cta(ctx._h, desc._h, 16, 32, 128, 1) == 0     # host-only context
    import torch
    if not torch.cuda.is_available():
        with pytest.raises(binding.LumoError):
            binding.Context(0)


def test_attention_visibility_table_matches_the_oracle_bit_for_bit():
    """The mask rows the attention kernel reads (bit s of node i = slot s holds i or an ancestor) against
    the oracle's visible positions, on permuted slot maps with padding."""
    from oracle import attn_oracle as A
    ctx = binding.Context(-1)
    for seed, N, Ns in ((1, 7, 7), (2, 28, 32), (3, 100, 131), (4, 256, 256)):
        parents = [W.tree_random(W.IntStream(W.stream_key(seed, b)), N, 9) for b in range(2)]
        c = W.make_attn_case("vis", parents, [0, 0], seed=seed, Hq=1, Hkv=1, dh=8, Ns=Ns, layout="permuted")
        desc = ctx.tree_desc(c.parent, slot=c.slot, n_slots=Ns)
        Wd = (Ns + 31) // 32
        for b in range(2):
            tab = desc.table("attn_vis", b).view(np.uint32).reshape(N, Wd)
            for i in range(N):
                want = np.zeros(Wd, dtype=np.uint32)
                for p in A.visible_positions(c.parent[b], c.slot[b], 0, i):
                    want[p >> 5] |= np.uint32(1 << (p & 31))
                assert np.array_equal(tab[i], want), (seed, b, i)
    wide = ctx.tree_desc(np.array([[-1, 0]], dtype=np.int32), n_slots=300)
    assert wide.table("attn_vis").size == 0          # beyond 256 slots the attention calls are refused


def test_spine_first_slot_map_is_contiguous_on_the_principal_chain():
    p = W.tree_paper_geometry()
    s = W.spine_first_slots(p)
    assert sorted(s) == list(range(len(p)))
    spine = [0, 1, 4, 7, 10, 13, 16, 17, 18, 19, 20, 21]
    assert [s[i] for i in spine] == list(range(12))


def test_attention_calls_refuse_to_launch_on_a_host_only_context():
    import ctypes as C
    ctx = binding.Context(-1)
    desc = ctx.tree_desc(np.array([[-1, 0, 1]], dtype=np.int32))
    arr = (binding._AttnArgs * 1)()
    for fn in (binding._lib.lumo_kv_write_tree, binding._lib.lumo_tree_attention):
        assert fn(ctx._h, desc._h, arr, 1, None) == 4            # LUMO_ERR_UNSUPPORTED: there is no CPU path
    assert binding._lib.lumo_kv_publish(ctx._h, desc._h, arr, 1, None, None, 4, None, None) == 4
    assert b"host-only" in binding._lib.lumo_last_error(ctx._h)
