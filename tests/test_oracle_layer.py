"""Pins for the oracle's expert FFN and the whole layer (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle
from tests.helpers import bits_to_f64, bruteforce_dense_moe, f32_to_bf16_bits, read_golden, small_case

PRECISIONS = ["f32", "f64"]


@pytest.mark.parametrize("prec", PRECISIONS)
def test_ffn_scalar_closed_form(prec):
    c = read_golden("ffn_scalar_closed_form.txt")["scalar"]
    x = f32_to_bf16_bits([c["x"]])
    w13 = f32_to_bf16_bits([[c["w_gate"]], [c["w_up"]]]).reshape(1, 2, 1)
    w2 = f32_to_bf16_bits([[c["w_down"]]]).reshape(1, 1, 1)
    o = moe_oracle.get(prec)
    y = o.expert_ffn(x.reshape(1), w13[0], w2[0])
    np.testing.assert_allclose(y, c["out"], rtol=3e-7 if prec == "f32" else 1e-14)
    out = o.forward(x.reshape(1, 1), np.zeros((1, 1), np.float32), w13, w2, 1)
    np.testing.assert_allclose(out, [c["out"]], rtol=3e-7 if prec == "f32" else 1e-14)


@pytest.mark.parametrize("prec", PRECISIONS)
def test_ffn_matches_torch_library_ops(prec):
    """Library reduction: F.silu(x W1^T) * (x W3^T) W2^T in float64 on the same bf16 values."""
    c = small_case(T=5, H=96, I=160, E=3, k=1, seed=11)
    o = moe_oracle.get(prec)
    for e in range(3):
        w13 = torch.from_numpy(bits_to_f64(c["w13"][e]))
        w2 = torch.from_numpy(bits_to_f64(c["w2"][e]))
        for t in range(5):
            xr = torch.from_numpy(bits_to_f64(c["x"][t]))
            ref = (torch.nn.functional.silu(w13[:160] @ xr) * (w13[160:] @ xr)) @ w2.T
            y = o.expert_ffn(c["x"][t], c["w13"][e], c["w2"][e])
            np.testing.assert_allclose(y, ref.numpy(), rtol=0, atol=2e-5 if prec == "f32" else 1e-12)


@pytest.mark.parametrize("prec", PRECISIONS)
@pytest.mark.parametrize("T,H,I,E,k,skew", [(16, 256, 512, 8, 2, False), (24, 64, 96, 16, 4, True),
                                           (7, 32, 48, 5, 5, False), (9, 40, 24, 6, 1, False)])
def test_layer_matches_dense_bruteforce(prec, T, H, I, E, k, skew):
    c = small_case(T, H, I, E, k, seed=0, skew=skew)
    out = moe_oracle.get(prec).forward(c["x"], c["logits"], c["w13"], c["w2"], k)
    ref = bruteforce_dense_moe(c["x"], c["logits"], c["w13"], c["w2"], k)
    tol = 1e-4 if prec == "f32" else 1e-11
    assert (np.abs(out - ref) <= tol * (1 + np.abs(ref))).all()
    assert np.abs(ref).max() > 0.05            # the comparison is not vacuous


def test_f32_build_is_within_its_error_bar_of_f64():
    c = small_case(16, 256, 512, 8, 2, seed=0)
    a = moe_oracle.get("f32").forward(c["x"], c["logits"], c["w13"], c["w2"], 2)
    b = moe_oracle.get("f64").forward(c["x"], c["logits"], c["w13"], c["w2"], 2)
    assert np.abs(a - b).max() <= 2e-5 * (1 + np.abs(b).max())


@pytest.mark.parametrize("prec", PRECISIONS)
def test_identical_experts_with_k_equal_E_is_one_dense_mlp(prec):
    """Invariant: if all E experts are the same and every expert is selected, the weights sum to
    one and the layer is a single SwiGLU MLP, whatever the router says."""
    c = small_case(T=6, H=64, I=80, E=8, k=8, seed=5)
    w13 = np.repeat(c["w13"][:1], 8, axis=0)
    w2 = np.repeat(c["w2"][:1], 8, axis=0)
    out = moe_oracle.get(prec).forward(c["x"], c["logits"], w13, w2, 8)
    x = bits_to_f64(c["x"]); a = bits_to_f64(w13[0]); b = bits_to_f64(w2[0])
    g = x @ a[:80].T; u = x @ a[80:].T
    ref = (g / (1 + np.exp(-g)) * u) @ b.T
    np.testing.assert_allclose(out, ref, rtol=0, atol=2e-5 if prec == "f32" else 1e-12)
    # E = 1, k = 1 is the same statement
    out1 = moe_oracle.get(prec).forward(c["x"], c["logits"][:, :1], w13[:1], w2[:1], 1)
    np.testing.assert_allclose(out1, ref, rtol=0, atol=2e-5 if prec == "f32" else 1e-12)


def test_token_permutation_equivariance_is_bit_exact():
    c = small_case(T=12, H=64, I=96, E=8, k=3, seed=9)
    o = moe_oracle.get("f32")
    perm = np.random.default_rng(0).permutation(12)
    a = o.forward(c["x"], c["logits"], c["w13"], c["w2"], 3)
    b = o.forward(c["x"][perm], c["logits"][perm], c["w13"], c["w2"], 3)
    assert np.array_equal(a[perm], b)


def test_zero_gate_or_up_gives_exact_zero_and_pow2_scaling_is_exact():
    c = small_case(T=4, H=32, I=48, E=4, k=2, seed=2)
    o = moe_oracle.get("f32")
    w13 = c["w13"].copy(); w13[:, :48, :] = 0          # gate rows zero -> SiLU(0) = 0
    assert not o.forward(c["x"], c["logits"], w13, c["w2"], 2).any()
    w13 = c["w13"].copy(); w13[:, 48:, :] = 0          # up rows zero
    assert not o.forward(c["x"], c["logits"], w13, c["w2"], 2).any()
    base = o.forward(c["x"], c["logits"], c["w13"], c["w2"], 2)
    w2x4 = f32_to_bf16_bits(bits_to_f64(c["w2"]) * 4.0)
    assert np.array_equal(o.forward(c["x"], c["logits"], c["w13"], w2x4, 2), base * np.float32(4.0))


def test_gate_and_up_are_not_interchangeable():
    """Swapping the two halves of w13 must change the result (guards the gate/up row convention)."""
    c = small_case(T=4, H=32, I=48, E=2, k=1, seed=3)
    o = moe_oracle.get("f64")
    swapped = np.concatenate([c["w13"][:, 48:], c["w13"][:, :48]], axis=1)
    a = o.forward(c["x"], c["logits"], c["w13"], c["w2"], 1)
    b = o.forward(c["x"], c["logits"], swapped, c["w2"], 1)
    assert np.abs(a - b).max() > 1e-3


@pytest.mark.parametrize("prec", PRECISIONS)
def test_sampled_forward_and_sorted_intermediates_agree_with_full_forward(prec):
    c = small_case(T=10, H=48, I=64, E=6, k=2, seed=4)
    o = moe_oracle.get(prec)
    full = o.forward(c["x"], c["logits"], c["w13"], c["w2"], 2)
    ids, w = o.route(c["logits"], 2)
    tokens = [7, 0, 3]
    need = {int(e) for t in tokens for e in ids[t]}
    experts = {e: (c["w13"][e], c["w2"][e]) for e in need}
    part = o.forward_sampled(c["x"], c["logits"], experts, 64, 2, tokens)
    assert np.array_equal(part, full[tokens])
    off, s2f, f2s = o.permute(ids, 6)
    h, y = o.sorted_intermediates(c["x"], c["w13"], c["w2"], ids, s2f)
    comb = np.zeros_like(full)
    for t in range(10):
        for j in range(2):
            comb[t] += w[t, j] * y[f2s[t * 2 + j]]
    assert np.array_equal(comb, full)
    # h row r is SiLU(gate)*up of the token that assignment sorted_to_flat[r] belongs to
    r = 5; a = s2f[r]; t = a // 2; e = ids.ravel()[a]
    x = bits_to_f64(c["x"][t]); w13 = bits_to_f64(c["w13"][e])
    g = w13[:64] @ x; u = w13[64:] @ x
    np.testing.assert_allclose(h[r], g / (1 + np.exp(-g)) * u, atol=2e-5)
