"""GPU parity: router and sort-scatter through moe_route, bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
from paper_2602_19128_b200.inputs import CONFIGS, zipf_bias
from tests.gpu_common import WEIGHT_TOL, Guarded

pytestmark = pytest.mark.gpu


def run_route(logits: torch.Tensor, k: int):
    """moe_route with every output array and the workspace between sentinel bands (checked after the call)."""
    T, E = logits.shape
    dev = logits.device
    A = T * k
    guards = [Guarded(n * 4, dev, fill=0xFF) for n in (A, A, E + 1, A, A)]
    ids, w, off, s2f, f2s = (g.inner[:n * 4].view(dt).view(shape) for g, n, dt, shape in zip(
        guards, (A, A, E + 1, A, A), (torch.int32, torch.float32, torch.int32, torch.int32, torch.int32),
        ((T, k), (T, k), (E + 1,), (A,), (A,))))
    wg = Guarded(moe.moe_route_workspace_bytes(T, E, k), dev)
    moe.moe_route(logits, k, ids, w, off, s2f, f2s, wg.inner)
    assert moe.moe_last_status(wg.inner) == moe.MOE_OK
    for g, name in zip(guards + [wg], ("topk_ids", "topk_weights", "expert_offsets", "sorted_to_flat", "flat_to_sorted",
                                       "workspace")):
        g.assert_bands_intact(f"moe_route {name}")
        if name != "workspace" and g.n > [A, A, E + 1, A, A][guards.index(g)] * 4:   # bytes past the array's end
            assert bool((g.inner[[A, A, E + 1, A, A][guards.index(g)] * 4:] == 0xFF).all()), name
    return [t.cpu().numpy() for t in (ids, w, off, s2f, f2s)]


def check_against_oracle(logits: torch.Tensor, k: int):
    E = logits.shape[1]
    ids, w, off, s2f, f2s = run_route(logits.cuda().contiguous(), k)
    o = moe_oracle.get("f32")
    rid, rw = o.route(logits.cpu().numpy(), k)
    roff, rs2f, rf2s = o.permute(rid, E)
    assert np.array_equal(ids, rid)
    assert np.array_equal(off, roff)
    assert np.array_equal(s2f, rs2f)
    assert np.array_equal(f2s, rf2s)
    np.testing.assert_allclose(w, rw, rtol=0, atol=WEIGHT_TOL)
    np.testing.assert_allclose(w.sum(axis=1), 1.0, atol=1e-5)


@pytest.mark.parametrize("name", list(CONFIGS))
def test_route_on_the_five_workloads(name):
    c = CONFIGS[name]
    g = torch.Generator().manual_seed(0)
    logits = torch.randn(c["T"], c["E"], generator=g)
    if c["skew"]:
        logits = logits + zipf_bias(c["E"])
    check_against_oracle(logits, c["top_k"])


@pytest.mark.parametrize("T,E,k", [(1, 1, 1), (1, 8, 8), (31, 5, 3), (32, 256, 8), (33, 256, 32), (1000, 97, 6),
                                   (257, 2, 1), (5000, 33, 4), (64, 200, 1)])
def test_route_odd_shapes(T, E, k):
    g = torch.Generator().manual_seed(T * 1000 + E)
    check_against_oracle(torch.randn(T, E, generator=g), k)


def test_route_constructed_ties():
    g = torch.Generator().manual_seed(5)
    T, E, k = 512, 64, 8
    logits = torch.randint(-2, 3, (T, E), generator=g).float()  # few distinct values: ties everywhere
    logits[7] = 0.75                                            # a whole row equal
    logits[8, ::2] = -0.0
    logits[8, 1::2] = 0.0                                       # signed zeros compare equal
    logits[9] = torch.arange(E, 0, -1).float()
    logits[9, 8] = logits[9, 7]                                 # tie exactly at the k-th / (k+1)-th boundary
    check_against_oracle(logits, k)


def test_route_all_tokens_to_one_expert_and_empty_experts():
    T, E, k = 300, 16, 1
    logits = torch.zeros(T, E)
    logits[:, 11] = 5.0
    check_against_oracle(logits, k)


def test_route_empty_batch_and_argument_errors():
    dev = "cuda"
    E, k = 8, 2
    off = torch.full((E + 1,), -1, dtype=torch.int32, device=dev)
    ws = moe.alloc_workspace(moe.moe_route_workspace_bytes(0, E, k), dev)
    empty_f = torch.empty((0, E), dtype=torch.float32, device=dev)
    empty_i = torch.empty((0, k), dtype=torch.int32, device=dev)
    flat = torch.empty((0,), dtype=torch.int32, device=dev)
    moe.moe_route(empty_f, k, empty_i, empty_f[:, :k].contiguous(), off, flat, flat, ws)
    torch.cuda.synchronize()
    assert (off == 0).all()
    # too-small workspace and top_k > E are rejected on the host
    logits = torch.zeros(64, E, device=dev)
    ids = torch.empty((64, k), dtype=torch.int32, device=dev)
    w = torch.empty((64, k), dtype=torch.float32, device=dev)
    s = torch.empty((64 * k,), dtype=torch.int32, device=dev)
    tiny_ws = moe.alloc_workspace(256, dev)
    assert moe.moe_route(logits, k, ids, w, off, s, s.clone(), tiny_ws, check=False) == -5
    big = moe.alloc_workspace(1 << 16, dev)
    assert moe.moe_route(logits, E + 1, ids, w, off, s, s.clone(), big, check=False) == -2


def test_route_large_batch_three_kernel_path_and_max_top_k():
    g = torch.Generator().manual_seed(21)
    check_against_oracle(torch.randn(100_000, 64, generator=g), 8)      # 800k assignments, 3125 chunks
    check_against_oracle(torch.randn(2_000, 64, generator=g), 32)       # the largest supported top_k


def test_route_non_finite_logits_terminate_with_in_range_distinct_ids():
    """NaN / inf logits are outside the contract, but the kernels must finish and stay in bounds."""
    g = torch.Generator().manual_seed(22)
    T, E, k = 300, 96, 8
    logits = torch.randn(T, E, generator=g)
    logits[0] = float("nan")
    logits[1, ::3] = float("inf")
    logits[2, 5:50] = float("-inf")
    logits[3, 7] = float("nan")
    logits[4] = float("-inf")
    ids, w, off, s2f, f2s = run_route(logits.cuda().contiguous(), k)
    assert ((ids >= 0) & (ids < E)).all()
    assert all(len(set(r.tolist())) == k for r in ids)
    assert off[0] == 0 and off[-1] == T * k and (np.diff(off) >= 0).all()
    assert np.array_equal(np.sort(s2f), np.arange(T * k)) and np.array_equal(s2f[f2s], np.arange(T * k))
    # rows without non-finite values are unaffected by their neighbours
    o = moe_oracle.get("f32")
    rid, _ = o.route(logits[5:].numpy(), k)
    assert np.array_equal(ids[5:], rid)
