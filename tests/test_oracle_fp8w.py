"""Pins for the oracle's FP8-block-scaled-weights variant (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle
from paper_2602_19128_b200.inputs import bf16_bits
from tests.weight_quantizers import make_fp8w_inputs
from tests.helpers import bits_to_f64, f32_to_bf16_bits

PRECISIONS = ["f32", "f64"]


def all_codes_as_float():
    return torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy()


def test_e4m3_decode_matches_the_library_conversion_for_all_256_codes():
    ref = all_codes_as_float()
    for prec in PRECISIONS:
        got = np.array([moe_oracle.get(prec).e4m3_decode(c) for c in range(256)], dtype=np.float32)
        assert np.array_equal(np.isnan(got), np.isnan(ref))
        assert np.array_equal(got[~np.isnan(ref)], ref[~np.isnan(ref)])
    # landmarks of the format, from its definition: largest finite 448, smallest subnormal 2^-9, 1.0 = 0x38
    o = moe_oracle.get("f32")
    assert o.e4m3_decode(0x7E) == 448.0 and o.e4m3_decode(0x01) == 2.0 ** -9 and o.e4m3_decode(0x38) == 1.0
    assert o.e4m3_decode(0xB8) == -1.0 and o.e4m3_decode(0x00) == 0.0 and np.isnan(o.e4m3_decode(0x7F))


def dequant(codes, scales):
    vals = all_codes_as_float().astype(np.float64)[codes]
    return vals * np.repeat(np.repeat(scales.astype(np.float64), 128, axis=1), 128, axis=2)


@pytest.mark.parametrize("prec", PRECISIONS)
@pytest.mark.parametrize("T,H,I,E,k", [(6, 128, 128, 4, 2), (5, 256, 128, 3, 3)])
def test_layer_matches_float64_bruteforce_on_dequantised_weights(prec, T, H, I, E, k):
    inp = make_fp8w_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=False), seed=1)
    x = bits_to_f64(bf16_bits(inp["x"]))
    l = inp["router_logits"].numpy()
    w13 = dequant(inp["w13_q"].numpy(), inp["w13_scale"].numpy())
    w2 = dequant(inp["w2_q"].numpy(), inp["w2_scale"].numpy())
    order = np.argsort(-l.astype(np.float64), axis=1, kind="stable")[:, :k]
    sel = np.take_along_axis(l.astype(np.float64), order, axis=1)
    z = np.exp(sel - sel.max(axis=1, keepdims=True)); w = z / z.sum(axis=1, keepdims=True)
    ref = np.zeros((T, H))
    for t in range(T):
        for j in range(k):
            e = order[t, j]
            g = w13[e, :I] @ x[t]; u = w13[e, I:] @ x[t]
            ref[t] += w[t, j] * (w2[e] @ (g / (1 + np.exp(-g)) * u))
    got = moe_oracle.get(prec).forward_fp8w(bf16_bits(inp["x"]), l, inp["w13_q"].numpy(), inp["w13_scale"].numpy(),
                                            inp["w2_q"].numpy(), inp["w2_scale"].numpy(), k)
    assert (np.abs(got - ref) <= (1e-4 if prec == "f32" else 1e-11) * (1 + np.abs(ref))).all()
    assert np.abs(ref).max() > 0.02


def test_unit_scales_and_representable_weights_reduce_to_the_bf16_layer_bit_for_bit():
    """Every E4M3 value is a bf16 value: with all scales 1 the FP8 path must equal the bf16 path exactly."""
    rng = np.random.default_rng(0)
    T, H, I, E, k = 4, 128, 128, 2, 1
    table = all_codes_as_float()
    finite = np.flatnonzero(~np.isnan(table) & (np.abs(table) <= 2.0))
    c13 = rng.choice(finite, size=(E, 2 * I, H)).astype(np.uint8)
    c2 = rng.choice(finite, size=(E, H, I)).astype(np.uint8)
    ones13, ones2 = np.ones((E, 2 * I // 128, H // 128), np.float32), np.ones((E, H // 128, I // 128), np.float32)
    x = f32_to_bf16_bits(rng.standard_normal((T, H)) * 0.1)
    l = rng.standard_normal((T, E)).astype(np.float32)
    o = moe_oracle.get("f32")
    a = o.forward_fp8w(x, l, c13, ones13, c2, ones2, k)
    b = o.forward(x, l, f32_to_bf16_bits(table[c13]), f32_to_bf16_bits(table[c2]), k)
    assert np.array_equal(a, b)
    # and a block scale of 4 on every w2 block multiplies the output by exactly 4
    assert np.array_equal(o.forward_fp8w(x, l, c13, ones13, c2, ones2 * 4, k), a * np.float32(4))


def test_quantisation_of_the_synthetic_weights_is_within_half_an_e4m3_step():
    inp = make_fp8w_inputs(dict(T=2, H=256, I=128, E=2, top_k=1, skew=False), seed=2)
    w = inp["w13"].double().numpy()
    deq = dequant(inp["w13_q"].numpy(), inp["w13_scale"].numpy())
    amax = np.abs(w).reshape(2, 2, 128, 2, 128).max(axis=(2, 4))
    bound = np.repeat(np.repeat(amax, 128, axis=1), 128, axis=2) / 448.0 * 16.0   # half a step at the top binade = 16 * scale
    assert (np.abs(deq - w) <= bound + 1e-12).all()
    assert np.abs(deq - w).max() > 0
