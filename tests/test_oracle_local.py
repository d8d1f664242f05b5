"""Pins for the oracle's local-expert-subset variant (CPU only)."""
import numpy as np
import pytest

from oracle import moe_oracle
from tests.helpers import bits_to_f64, small_case

PRECISIONS = ["f32", "f64"]


def masked_bruteforce(c, k, lo, n):
    """Float64 dense evaluation in which only experts [lo, lo+n) contribute; weights are the softmax
    over the selected logits of ALL top-k experts (no renormalisation over the local ones)."""
    x = bits_to_f64(c["x"]); w13 = bits_to_f64(c["w13"]); w2 = bits_to_f64(c["w2"])
    l = c["logits"].astype(np.float64)
    T, E = l.shape
    I = w13.shape[1] // 2
    order = np.argsort(-l, axis=1, kind="stable")[:, :k]
    sel = np.take_along_axis(l, order, axis=1)
    z = np.exp(sel - sel.max(axis=1, keepdims=True))
    w = z / z.sum(axis=1, keepdims=True)
    dense = np.zeros((T, E)); np.put_along_axis(dense, order, w, axis=1)
    out = np.zeros_like(x)
    for e in range(lo, lo + n):
        g = x @ w13[e, :I].T; u = x @ w13[e, I:].T
        out += dense[:, e:e + 1] * ((g / (1 + np.exp(-g)) * u) @ w2[e].T)
    return out


@pytest.mark.parametrize("prec", PRECISIONS)
def test_all_experts_local_is_the_full_layer_bit_for_bit(prec):
    c = small_case(T=9, H=48, I=64, E=6, k=2, seed=1)
    o = moe_oracle.get(prec)
    full = o.forward(c["x"], c["logits"], c["w13"], c["w2"], 2)
    assert np.array_equal(o.forward_local(c["x"], c["logits"], c["w13"], c["w2"], 6, 2, 0), full)


@pytest.mark.parametrize("prec", PRECISIONS)
@pytest.mark.parametrize("lo,n", [(0, 2), (2, 3), (5, 1), (3, 0)])
def test_local_subset_matches_masked_bruteforce(prec, lo, n):
    c = small_case(T=14, H=40, I=56, E=6, k=3, seed=2)
    o = moe_oracle.get(prec)
    got = o.forward_local(c["x"], c["logits"], c["w13"][lo:lo + n], c["w2"][lo:lo + n], 6, 3, lo)
    ref = masked_bruteforce(c, 3, lo, n)
    assert (np.abs(got - ref) <= (1e-4 if prec == "f32" else 1e-11) * (1 + np.abs(ref))).all()
    if n == 0:
        assert not got.any()


def test_partial_outputs_of_a_partition_add_up_to_the_full_layer():
    c = small_case(T=20, H=64, I=96, E=8, k=4, seed=3)
    o = moe_oracle.get("f64")
    full = o.forward(c["x"], c["logits"], c["w13"], c["w2"], 4)
    parts = sum(o.forward_local(c["x"], c["logits"], c["w13"][lo:lo + 2], c["w2"][lo:lo + 2], 8, 4, lo)
                for lo in (0, 2, 4, 6))
    np.testing.assert_allclose(parts, full, rtol=0, atol=1e-12)


def test_permute_local_hand_example_and_invariants():
    # T=3, k=2, ids rows [2,0],[0,1],[2,1]; local experts 1..2 (offset 1, two of them):
    # expert 1 (local 0) has flat 3, 5; expert 2 (local 1) has flat 0, 4; flat 1, 2 (expert 0) are dropped.
    ids = np.array([[2, 0], [0, 1], [2, 1]], np.int32)
    off, s2f, f2s = moe_oracle.get("f32").permute_local(ids, 1, 2)
    assert off.tolist() == [0, 2, 4]
    assert s2f.tolist() == [3, 5, 0, 4, -1, -1]
    assert f2s.tolist() == [2, -1, -1, 0, 3, 1]
    # with every expert local it is the ordinary sort-scatter
    rng = np.random.default_rng(0)
    ids = np.stack([rng.permutation(16)[:4] for _ in range(50)]).astype(np.int32)
    a = moe_oracle.get("f32").permute(ids, 16)
    b = moe_oracle.get("f32").permute_local(ids, 0, 16)
    assert all(np.array_equal(u, v) for u, v in zip(a, b))
    # a strict subset: kept assignments are exactly those with a local id, in stable order
    off, s2f, f2s = moe_oracle.get("f32").permute_local(ids, 4, 5)
    flat = ids.ravel()
    keep = (flat >= 4) & (flat < 9)
    assert off[-1] == keep.sum() and (f2s[~keep] == -1).all() and (s2f[off[-1]:] == -1).all()
    kept_sorted = s2f[:off[-1]]
    assert (kept_sorted == np.flatnonzero(keep)[np.argsort(flat[keep], kind="stable")]).all()
