"""Pins for the oracle's grouped sigmoid router: the fixed exp recipe against libm, a hand-derived case, a NumPy
float64 brute force written with sorts and masks, and the properties the rule fixes."""
import math

import numpy as np
import pytest

from oracle import moe_oracle
from paper_2602_19128_b200.inputs import bf16_bits, make_inputs
from tests.helpers import bits_to_f64, read_golden


def brute_grouped(logits, k, n_group, topk_group, bias, scale):
    """Float64, independent formulation: stable argsorts and a boolean mask instead of selection passes."""
    l = np.asarray(logits, dtype=np.float64)
    T, E = l.shape
    G = E // n_group
    score = 1.0 / (1.0 + np.exp(-l))
    choice = score + (0.0 if bias is None else np.asarray(bias, dtype=np.float64))
    grouped = np.sort(choice.reshape(T, n_group, G), axis=2)
    gscore = grouped[:, :, -2:].sum(axis=2) if G >= 2 else grouped[:, :, -1]
    keep_groups = np.argsort(-gscore, axis=1, kind="stable")[:, :topk_group]
    mask = np.zeros((T, n_group), bool)
    np.put_along_axis(mask, keep_groups, True, axis=1)
    masked = np.where(np.repeat(mask, G, axis=1), choice, -np.inf)
    ids = np.argsort(-masked, axis=1, kind="stable")[:, :k]
    sel = np.take_along_axis(score, ids, axis=1)
    return ids.astype(np.int32), sel / sel.sum(axis=1, keepdims=True) * scale


def test_fixed_exp_recipe_tracks_libm():
    o = moe_oracle.get("f32")
    xs = np.concatenate([np.linspace(-87, 88, 4001), np.linspace(-1, 1, 2001), [0.0, -0.0, 1e-8, -1e-8]]).astype(np.float32)
    for x in xs:
        assert abs(o.exp_fixed(float(x)) / math.exp(float(x)) - 1) < 2.5e-7
    assert o.exp_fixed(-1000.0) == o.exp_fixed(-87.0) and o.exp_fixed(1000.0) == o.exp_fixed(88.0)  # clamped
    assert o.sigmoid_fixed(0.0) == 0.5
    for v in (-30.0, -3.0, -0.1, 0.2, 5.0, 40.0):
        assert abs(o.sigmoid_fixed(v) - 1 / (1 + math.exp(-v))) < 1.5e-7
    vals = [o.sigmoid_fixed(float(v)) for v in np.linspace(-20, 20, 2001)]
    assert all(b >= a for a, b in zip(vals, vals[1:]))  # never decreasing


@pytest.mark.parametrize("prec", ["f32", "f64"])
def test_hand_derived_case(prec):
    c = read_golden("grouped_router.txt")["groups_of_two"]
    p = np.array(c["p"])
    logits = np.log(p / (1 - p)).astype(np.float32)[None, :]
    ids, w = moe_oracle.get(prec).route_grouped(logits, 2, 4, 2, bias=np.array(c["bias"], np.float32), scale=2.5)
    assert ids[0].tolist() == [int(v) for v in c["ids"]]
    assert np.allclose(w[0], c["weights"], rtol=0, atol=1e-6)


@pytest.mark.parametrize("T,E,k,n_group,topk_group", [(64, 64, 6, 8, 3), (40, 256, 8, 8, 4), (30, 32, 4, 32, 5),
                                                        (50, 48, 5, 3, 2), (20, 16, 16, 1, 1), (33, 128, 8, 4, 1)])
def test_matches_float64_brute_force(T, E, k, n_group, topk_group):
    rng = np.random.default_rng(E + k)
    logits = rng.normal(0, 1.5, (T, E)).astype(np.float32)
    bias = rng.normal(0, 0.2, E).astype(np.float32)
    want_ids, want_w = brute_grouped(logits, k, n_group, topk_group, bias, 2.5)
    for prec in ("f32", "f64"):
        ids, w = moe_oracle.get(prec).route_grouped(logits, k, n_group, topk_group, bias=bias, scale=2.5)
        assert np.array_equal(ids, want_ids)
        assert np.allclose(w, want_w, rtol=0, atol=2e-6)


def test_one_group_without_bias_selects_like_the_softmax_router():
    """sigmoid is increasing, so with a single group and no bias the chosen experts are those of the largest logits."""
    rng = np.random.default_rng(1)
    logits = rng.normal(size=(200, 32)).astype(np.float32)
    o = moe_oracle.get("f32")
    ids, w = o.route_grouped(logits, 4, 1, 1)
    ids_softmax, _ = o.route(logits, 4)
    assert np.array_equal(ids, ids_softmax)
    assert np.allclose(w.sum(axis=1), 1.0, atol=1e-6)


def test_properties_fixed_by_the_rule():
    rng = np.random.default_rng(2)
    T, E, k, n_group, topk_group = 300, 64, 6, 8, 2
    logits = rng.normal(size=(T, E)).astype(np.float32)
    bias = rng.normal(0, 0.3, E).astype(np.float32)
    o = moe_oracle.get("f32")
    ids, w = o.route_grouped(logits, k, n_group, topk_group, bias=bias, scale=1.7)
    assert all(len(set(r)) == k for r in ids.tolist())                       # k distinct experts
    assert all(len({e // (E // n_group) for e in r}) <= topk_group for r in ids.tolist())  # from at most topk_group groups
    assert np.allclose(w.sum(axis=1), 1.7, atol=1e-5)                        # weights sum to the scale
    # rank order: the choice values (score + bias) of the selected experts never increase
    score = np.array([[o.sigmoid_fixed(float(v)) for v in row] for row in logits[:20]], np.float32)
    choice = score + bias
    for t in range(20):
        c = choice[t, ids[t]]
        assert np.all(c[:-1] >= c[1:])
    # a large bias forces selection but does not enter the weight
    big = np.zeros(E, np.float32)
    big[5] = 10.0
    ids2, w2 = o.route_grouped(logits, k, n_group, topk_group, bias=big, scale=1.0)
    assert np.all(ids2[:, 0] == 5)
    s5 = np.array([o.sigmoid_fixed(float(v)) for v in logits[:, 5]])
    assert np.all(w2[:, 0] < 1.0) and np.allclose(w2[:, 0] * np.array(
        [sum(o.sigmoid_fixed(float(logits[t, e])) for e in ids2[t]) for t in range(T)]), s5, atol=1e-5)


def test_ties_go_to_the_lower_index():
    logits = np.zeros((1, 16), np.float32)
    ids, w = moe_oracle.get("f32").route_grouped(logits, 4, 4, 2)
    assert ids[0].tolist() == [0, 1, 2, 3]      # groups 0 and 1 win the group tie; experts in index order
    assert np.allclose(w, 0.25)


def test_invalid_group_settings_are_rejected():
    o = moe_oracle.get("f32")
    l = np.zeros((1, 16), np.float32)
    for n_group, topk_group, k in ((3, 1, 2), (4, 5, 2), (4, 1, 5), (0, 1, 1)):
        with pytest.raises(RuntimeError):
            o.route_grouped(l, k, n_group, topk_group)


def test_layer_with_the_grouped_router_matches_a_dense_float64_evaluation():
    cfg = dict(T=10, H=64, I=32, E=16, top_k=3, skew=False)
    inp = make_inputs(cfg, seed=3)
    logits = inp["router_logits"].numpy()
    bias = np.linspace(-0.2, 0.2, 16).astype(np.float32)
    ids, wsel = brute_grouped(logits, 3, 4, 2, bias, 2.5)
    x, w13, w2 = (bits_to_f64(bf16_bits(inp[n])) for n in ("x", "w13", "w2"))
    dense_w = np.zeros((10, 16))
    np.put_along_axis(dense_w, ids.astype(np.int64), wsel, axis=1)
    want = np.zeros_like(x)
    for e in range(16):
        g, u = x @ w13[e, :32].T, x @ w13[e, 32:].T
        want += dense_w[:, e:e + 1] * ((g / (1 + np.exp(-g)) * u) @ w2[e].T)
    experts = {e: (bf16_bits(inp["w13"][e]), bf16_bits(inp["w2"][e])) for e in range(16)}
    got = moe_oracle.get("f64").forward_sampled_grouped(bf16_bits(inp["x"]), logits, experts, 32, 3, np.arange(10), 4, 2,
                                                        bias=bias, scale=2.5)
    assert np.allclose(got, want, rtol=1e-5, atol=1e-6)
