"""Fused draft selection (lumo_select_spine_top3) against its oracle: both output tensors must match
byte for byte, for every way of splitting a row over CTAs, on rows with planted ties."""
import numpy as np
import pytest
import torch

from oracle import select_oracle as S
from paper_2609_23900_b200 import binding
from tests.harness import ctx

pytestmark = pytest.mark.gpu


def make_logits(R, V, seed, dtype):
    """Synthetic logits rows with the tie patterns that matter: quantised rows (many ties), rows with
    the maximum planted two or three times, constant rows, masked (-inf) stretches."""
    rs = np.random.default_rng(seed)
    x = (rs.standard_normal((R, V)) * 3).astype(np.float32)
    for r in range(R):
        kind = r % 6
        if kind == 1:
            x[r] = np.round(x[r])                                   # few distinct values
        elif kind == 2:
            pos = rs.choice(V, size=min(3, V), replace=False)       # the maximum three times
            x[r, pos] = x[r].max() + 1
        elif kind == 3:
            x[r] = 0.5                                              # constant row
        elif kind == 4:
            x[r, rs.uniform(size=V) < 0.7] = -np.inf                # masked vocabulary
        elif kind == 5:
            pos = rs.choice(V, size=min(2, V), replace=False)       # tie for second place
            x[r, pos] = np.sort(x[r])[-1] - 0.25
    t = torch.from_numpy(x).to(dtype)
    return t


def run(t, split):
    dev = torch.device("cuda", 0)
    d = t.to(dev)
    R = d.shape[0]
    spine = torch.full((R,), -7, dtype=torch.int32, device=dev)
    cand = torch.full((R, 3), -7, dtype=torch.int32, device=dev)
    ctx().select_spine_top3(d, spine, cand, split=split)
    torch.cuda.synchronize()
    return spine.cpu().numpy(), cand.cpu().numpy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("R,V", [(5, 3), (6, 37), (12, 4099), (7, 32000), (6, 151936), (9, 8191)])
def test_select_matches_oracle_for_every_split(dtype, R, V):
    t = make_logits(R, V, seed=R * 1000 + V, dtype=dtype)
    ref = S.select(t.to(torch.float64).numpy())
    for split in (0, 1, 2, 4, 8, 16):
        spine, cand = run(t, split)
        assert spine.tobytes() == ref[0].tobytes(), f"spine, split {split}"
        assert cand.tobytes() == ref[1].tobytes(), f"candidates, split {split}"


def test_select_unaligned_rows():
    # V odd: rows start on every 2- and 4-byte offset, so the 16-byte body, head and tail all occur
    for dtype in (torch.float32, torch.bfloat16):
        t = make_logits(11, 1237, seed=3, dtype=dtype)
        ref = S.select(t.to(torch.float64).numpy())
        spine, cand = run(t, 4)
        assert np.array_equal(spine, ref[0]) and np.array_equal(cand, ref[1])


def test_select_negative_control():
    # a planted change of one logit must change the outputs (the comparison is not vacuous)
    t = make_logits(4, 5000, seed=9, dtype=torch.float32)
    a = run(t, 0)
    t2 = t.clone()
    t2[0, 4999] = 1e9
    b = run(t2, 0)
    assert b[0][0] == 4999 and b[1][0, 0] == 4999 and (a[0][0] != 4999)


def test_select_many_rows_and_graph_replay():
    dev = torch.device("cuda", 0)
    t = make_logits(300, 20000, seed=11, dtype=torch.bfloat16).to(dev)
    ref = S.select(t.cpu().to(torch.float64).numpy())
    spine = torch.zeros((300,), dtype=torch.int32, device=dev)
    cand = torch.zeros((300, 3), dtype=torch.int32, device=dev)
    c = ctx()
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        c.select_spine_top3(t, spine, cand, stream=st)          # warm-up outside capture
        st.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=st):
            c.select_spine_top3(t, spine, cand, stream=st)
        for _ in range(4):
            spine.fill_(-1); cand.fill_(-1)
            g.replay()
            st.synchronize()
            assert np.array_equal(spine.cpu().numpy(), ref[0]) and np.array_equal(cand.cpu().numpy(), ref[1])


def test_select_argument_errors():
    dev = torch.device("cuda", 0)
    t = torch.zeros((2, 2), device=dev)
    spine = torch.zeros((2,), dtype=torch.int32, device=dev)
    cand = torch.zeros((2, 3), dtype=torch.int32, device=dev)
    with pytest.raises(binding.LumoError) as e:
        ctx().select_spine_top3(t, spine, cand)                   # V < 3
    assert e.value.code == 1
    with pytest.raises(binding.LumoError) as e:
        ctx().select_spine_top3(torch.zeros((2, 8), device=dev), spine, cand, split=3)
    assert e.value.code == 1
