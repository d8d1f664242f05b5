"""Pins for the oracle's router and sort-scatter (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle
from tests.helpers import read_golden

PRECISIONS = ["f32", "f64"]


@pytest.mark.parametrize("prec", PRECISIONS)
def test_router_closed_forms(prec):
    o = moe_oracle.get(prec)
    for name, c in read_golden("router_closed_forms.txt").items():
        logits = np.array([c["logits"]], dtype=np.float32)
        ids, w = o.route(logits, int(c["k"][0]))
        assert ids[0].tolist() == [int(v) for v in c["ids"]], name
        # the fixture's logits are rounded to fp32 on the way in, which moves the weights by ~1e-8
        np.testing.assert_allclose(w[0], c["w"], rtol=0, atol=2e-7, err_msg=name)
    # k = 1 gives a weight of exactly one
    ids, w = o.route(np.array([[-3.0, 7.5, 2.0]], np.float32), 1)
    assert w[0, 0] == 1.0


@pytest.mark.parametrize("prec", PRECISIONS)
@pytest.mark.parametrize("T,E,k", [(64, 8, 2), (200, 256, 8), (33, 128, 8), (17, 5, 5), (9, 1, 1)])
def test_router_matches_torch_softmax_topk(prec, T, E, k):
    """Library reduction: torch.softmax + torch.topk on tie-free rows."""
    g = torch.Generator().manual_seed(1234 + E)
    logits = torch.randn(T, E, generator=g, dtype=torch.float32)
    ids, w = moe_oracle.get(prec).route(logits.numpy(), k)
    p = torch.softmax(logits.double(), dim=1)
    tv, ti = torch.topk(p, k, dim=1)
    tie_free = np.array([len(set(r.tolist())) == E for r in logits])
    assert tie_free.sum() >= T - 1
    assert (ids[tie_free] == ti.numpy()[tie_free]).all()
    wref = (tv / tv.sum(dim=1, keepdim=True)).numpy()
    np.testing.assert_allclose(w[tie_free], wref[tie_free], rtol=0, atol=3e-7 if prec == "f32" else 1e-12)


@pytest.mark.parametrize("prec", PRECISIONS)
def test_router_invariants(prec):
    g = torch.Generator().manual_seed(7)
    T, E, k = 300, 64, 6
    logits = torch.randn(T, E, generator=g).numpy()
    o = moe_oracle.get(prec)
    ids, w = o.route(logits, k)
    assert ((ids >= 0) & (ids < E)).all()
    assert all(len(set(r.tolist())) == k for r in ids)               # distinct experts
    np.testing.assert_allclose(w.sum(axis=1), 1.0, atol=1e-6)          # weights sum to one
    assert (w > 0).all() and (np.diff(w, axis=1) <= 0).all()           # positive, non-increasing in rank
    sel = np.take_along_axis(logits, ids, axis=1)
    assert (np.diff(sel, axis=1) <= 0).all()                           # rank order = descending logit
    rest_max = np.where(np.isin(np.arange(E)[None, :].repeat(T, 0), ids), -np.inf, logits)
    for t in range(T):
        mask = np.ones(E, bool); mask[ids[t]] = False
        assert logits[t, mask].max() <= sel[t, -1]                     # nothing left out beats the k-th
    # k = E: weights are the softmax itself
    ids_all, w_all = o.route(logits[:20], E)
    p = torch.softmax(torch.from_numpy(logits[:20]).double(), dim=1).numpy()
    np.testing.assert_allclose(w_all, np.take_along_axis(p, ids_all, axis=1), atol=3e-7)
    # shifting every logit of a row by a constant changes nothing that is exact
    ids_shift, _ = o.route(logits + np.float32(4.0), k)
    same = np.take_along_axis(logits + np.float32(4.0), ids, 1) - np.take_along_axis(logits, ids, 1)
    assert (ids_shift == ids).mean() > 0.99 and np.isfinite(same).all()


def test_router_constructed_ties():
    """Ties are rare in random data, so build them: duplicates at the k-th boundary, inside the
    top-k, and whole rows equal.  Expected ids come from a stable argsort on the negated logits."""
    rng = np.random.default_rng(3)
    T, E, k = 128, 32, 4
    logits = rng.integers(-3, 4, size=(T, E)).astype(np.float32)  # many exact duplicates
    logits[5, :] = 1.25
    logits[6, ::2] = -0.0
    logits[6, 1::2] = 0.0
    expect = np.argsort(-logits.astype(np.float64), axis=1, kind="stable")[:, :k]
    for prec in PRECISIONS:
        ids, w = moe_oracle.get(prec).route(logits, k)
        assert (ids == expect).all()
        np.testing.assert_allclose(w[5], 0.25, atol=1e-7)


def test_permute_hand_example():
    c = read_golden("permute_hand_example.txt")["hand"]
    T, k, E = int(c["T"][0]), int(c["k"][0]), int(c["E"][0])
    ids = np.array(c["ids"], np.int32).reshape(T, k)
    off, s2f, f2s = moe_oracle.get("f32").permute(ids, E)
    assert off.tolist() == [int(v) for v in c["offsets"]]
    assert s2f.tolist() == [int(v) for v in c["sorted_to_flat"]]
    assert f2s.tolist() == [int(v) for v in c["flat_to_sorted"]]


@pytest.mark.parametrize("T,E,k,seed", [(1, 4, 2, 0), (37, 8, 2, 1), (128, 256, 8, 2), (1000, 128, 8, 3), (64, 7, 7, 4)])
def test_permute_matches_stable_argsort_and_invariants(T, E, k, seed):
    g = torch.Generator().manual_seed(seed)
    logits = torch.randn(T, E, generator=g)
    if seed == 3:
        logits = logits - 2.2 * torch.log(torch.arange(1, E + 1, dtype=torch.float32))
    o = moe_oracle.get("f32")
    ids, _ = o.route(logits.numpy(), k)
    off, s2f, f2s = o.permute(ids, E)
    flat = ids.ravel()
    A = T * k
    assert (s2f == np.argsort(flat, kind="stable")).all()                 # library reduction
    assert (off == np.concatenate([[0], np.cumsum(np.bincount(flat, minlength=E))])).all()
    assert off[E] == A
    assert (s2f[f2s] == np.arange(A)).all() and (f2s[s2f] == np.arange(A)).all()   # inverse permutations
    assert (np.diff(flat[s2f]) >= 0).all()                                # expert-contiguous
    for e in range(E):                                                    # stable: flat index increases inside a segment
        seg = s2f[off[e]:off[e + 1]]
        assert (flat[seg] == e).all() and (np.diff(seg) > 0).all()
        assert (np.diff(seg // k) > 0).all()                              # hence token index strictly increases too
