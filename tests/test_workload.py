"""The seeded input generators: determinism, dtype exactness, tree-shape recipes."""
import numpy as np
import torch

from synthetic import workload as W


def test_streams_are_counter_based_and_reproducible():
    k = W.stream_key(1, 2, 3)
    a = W.uniforms(k, 100)
    assert np.array_equal(a[10:20], W.uniforms(k, 10, start=10))
    assert np.array_equal(a, W.uniforms(W.stream_key(1, 2, 3), 100))
    assert not np.array_equal(a, W.uniforms(W.stream_key(1, 2, 4), 100))
    assert a.min() >= 0.0 and a.max() < 1.0
    n = W.normals(k, 200000)
    assert abs(n.mean()) < 0.01 and abs(n.std() - 1.0) < 0.01


def test_splitmix64_known_answer():
    # published first outputs of splitmix64 seeded with 0 (Vigna's reference generator)
    assert W._mix_int(0) == 0xE220A8397B1DCDAF
    assert W._mix_int(W._GOLDEN) == 0x6E789E6AA1B965F4


def test_rounding_matches_library_casts():
    x = np.random.default_rng(0).normal(size=5000) * 3
    r = W.round_to(x, "bf16")
    lib = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(r, lib)
    assert np.array_equal(W.round_to(x, "f32"), x.astype(np.float32))


def test_tree_recipes():
    assert W.tree_tiny() == [-1, -1, 0, 0, 1, 1, 2]
    for seed in range(20):
        p = W.tree_mtp_spine(W.IntStream(seed))
        assert len(p) == 16 and p[:4] == [-1, 0, 1, 2] and all(-1 <= q < i for i, q in enumerate(p))
        for lvl in range(4):  # the spine node of this level plus its 2-3 single-node siblings
            assert 3 <= p.count(lvl - 1) <= 4
        p = W.tree_random(W.IntStream(seed), 64, 8)
        d = W.tree_depths(p)
        assert len(p) == 64 and max(d) <= 8 and all(-1 <= q < i for i, q in enumerate(p))
        assert max(p.count(i) for i in range(-1, 64)) <= 4
    p = W.tree_chains(16, 16)
    assert len(p) == 256 and max(W.tree_depths(p)) == 16 and p.count(-1) == 16
    p = W.tree_star(256)
    assert p.count(0) == 255 and W.tree_depths(p)[1:] == [2] * 255
    p = W.tree_paper_geometry()
    assert len(p) == 28 and max(W.tree_depths(p)) == 12   # root token + draft depth 11


def test_config0_recipe_statistics_and_accepted_path():
    c = W.config0()
    L = c.layers[0]
    assert (c.B, c.N, c.Hk, c.Hv, c.d, c.C) == (1, 7, 2, 2, 64, 384)
    assert c.accepted.tolist() == [[0, 2, 6]] and c.accepted_len.tolist() == [3]
    np.testing.assert_allclose(np.linalg.norm(L.q, axis=-1), 1.0, atol=1e-6)
    np.testing.assert_allclose(np.linalg.norm(L.k, axis=-1), 1.0, atol=1e-6)
    assert L.alpha.min() >= 0.9 and L.alpha.max() <= 1.0 and 0 < L.beta.min() and L.beta.max() < 1
    assert abs(L.state.std() - 0.02) < 0.002 and abs(L.conv_w.std() - 0.5) < 0.05


def test_accepted_paths_are_valid_prefix_walks():
    c = W.config2(B=4)
    for b in range(c.B):
        ln = c.accepted_len[b]
        a = c.accepted[b]
        assert ln >= 1 and c.parent[b, a[0]] == -1 and np.all(a[ln:] == -1)
        assert all(c.parent[b, a[t]] == a[t - 1] for t in range(1, ln))
    assert sorted(c.state_row.tolist()) == sorted(set(c.state_row.tolist()))
    for L in c.layers:   # bf16-exact
        for arr in (L.x, L.q, L.k, L.v, L.alpha, L.beta, L.hist, L.conv_w):
            t = torch.from_numpy(arr)
            assert torch.equal(t.to(torch.bfloat16).to(torch.float32), t)
