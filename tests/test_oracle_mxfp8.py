"""Pins for the oracle's MX FP8 path (E4M3 codes, one E8M0 scale byte per 32 elements): the encoder against
a brute-force nearest-code search and torch's float8 conversion, the block quantiser against the properties
the MX rule fixes and against the library-built weight quantiser, and the whole layer against a NumPy float64
evaluation made of library routines only."""
import numpy as np
import pytest
import torch

from oracle import moe_oracle
from paper_2602_19128_b200.inputs import bf16_bits
from tests.weight_quantizers import make_mxfp8_inputs, quantize_mxfp8
from tests.helpers import bits_to_f64

# every E4M3 code's value, from torch's own float8 type (independent of the oracle's decoder)
TABLE = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)
FINITE = np.array([c for c in range(256) if not np.isnan(TABLE[c])])


def nearest_code(v: float) -> int:
    """Brute force over all finite codes: smallest distance, ties to the even code, sign of v kept for zero."""
    cands = FINITE[(FINITE >= 128) == bool(np.signbit(v))]
    d = np.abs(TABLE[cands] - v)
    best = cands[d == d.min()]
    if len(best) > 1:
        best = best[best % 2 == 0]
    assert len(best) == 1
    return int(best[0])


def test_decoder_matches_torch_table():
    o = moe_oracle.get("f32")
    for c in FINITE:
        assert o.e4m3_decode(int(c)) == TABLE[c]
    assert np.isnan(o.e4m3_decode(0x7F)) and np.isnan(o.e4m3_decode(0xFF))


def test_encoder_round_trips_every_code_and_saturates():
    o = moe_oracle.get("f32")
    for c in FINITE:
        assert o.e4m3_encode(float(TABLE[c])) == c
    assert o.e4m3_encode(1e9) == 0x7E and o.e4m3_encode(-1e9) == 0xFE
    assert o.e4m3_encode(464.0) == 0x7E and o.e4m3_encode(480.0) == 0x7E  # beyond the largest code: saturate
    assert o.e4m3_encode(float("nan")) & 0x7F == 0x7F


def test_encoder_is_nearest_even_by_brute_force():
    o = moe_oracle.get("f32")
    rng = np.random.default_rng(0)
    vals = np.concatenate([
        rng.normal(0, 1, 3000), rng.normal(0, 100, 3000), rng.uniform(-0.02, 0.02, 3000),
        (TABLE[FINITE][:-1] + TABLE[FINITE][1:]) / 2,          # every midpoint between neighbours (within a sign)
        [2.0 ** -10, 3 * 2.0 ** -10, -2.0 ** -10, 2.0 ** -11, 447.9, 448.0, -448.0],
    ]).astype(np.float32)
    vals = vals[np.abs(vals) <= 448]
    for v in vals:
        assert o.e4m3_encode(float(v)) == nearest_code(float(v)), v


def test_encoder_matches_torch_conversion():
    o = moe_oracle.get("f32")
    g = torch.Generator().manual_seed(1)
    v = torch.cat([torch.randn(5000, generator=g) * s for s in (0.01, 1.0, 30.0, 150.0)]).clamp(-448, 448)
    want = v.to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = np.array([o.e4m3_encode(float(a)) for a in v.numpy()], dtype=np.uint8)
    assert np.array_equal(got, want)


def _random_rows(R, K, seed):
    g = torch.Generator().manual_seed(seed)
    scale = torch.exp2(torch.randint(-20, 20, (R, K // 32, 1), generator=g).float())
    return (torch.randn((R, K // 32, 32), generator=g) * scale).view(R, K).numpy()


def test_block_scale_puts_the_largest_element_in_the_top_binade():
    """The rule fixes the scale as the power of two with amax / scale in [2^8, 2^9)."""
    v = _random_rows(16, 256, 2)
    codes, sb = moe_oracle.get("f32").mx_quantize(v)
    amax = np.abs(v.reshape(16, 8, 32)).max(axis=2).astype(np.float64)
    ratio = amax / np.exp2(sb.astype(np.float64) - 127)
    assert np.all((ratio >= 256) & (ratio < 512))
    top = np.abs(TABLE[codes.reshape(16, 8, 32)]).max(axis=2)
    assert np.all((top >= 256) & (top <= 448))


def test_block_codes_are_the_nearest_codes_of_the_scaled_values():
    v = _random_rows(4, 128, 3)
    codes, sb = moe_oracle.get("f32").mx_quantize(v)
    scaled = v.astype(np.float64).reshape(4, 4, 32) / np.exp2(sb.astype(np.float64) - 127)[:, :, None]
    for r in range(4):
        for b in range(4):
            for i in range(32):
                s = float(np.clip(scaled[r, b, i], -448, 448))
                assert codes[r, 32 * b + i] == nearest_code(s)


def test_block_quantiser_matches_the_library_built_one():
    v = _random_rows(64, 512, 4)
    codes, sb = moe_oracle.get("f32").mx_quantize(v)
    c2, s2 = quantize_mxfp8(torch.from_numpy(v))
    assert np.array_equal(sb, s2.numpy()) and np.array_equal(codes, c2.numpy())


def test_power_of_two_scaling_moves_only_the_scale_byte():
    v = _random_rows(8, 128, 5)
    o = moe_oracle.get("f32")
    c0, s0 = o.mx_quantize(v)
    c1, s1 = o.mx_quantize(v * np.float32(2.0 ** 7))
    assert np.array_equal(c0, c1) and np.array_equal(s1.astype(int), s0.astype(int) + 7)


def test_zero_and_non_finite_blocks():
    v = np.zeros((1, 96), np.float32)
    v[0, 40] = np.inf
    v[0, 70] = 3.0
    codes, sb = moe_oracle.get("f32").mx_quantize(v)
    assert sb[0, 0] == 0 and np.all(codes[0, :32] == 0)
    assert sb[0, 1] == 255 and np.all(codes[0, 32:64] == 0x7F)
    assert sb[0, 2] == 127 + 1 - 8 and codes[0, 70] == nearest_code(3.0 * 2.0 ** 7) == 0x7C


def dequant(codes, sb):
    return TABLE[codes] * np.repeat(np.exp2(sb.astype(np.float64) - 127), 32, axis=-1)


def bruteforce_mx_layer(x_bits, logits, w13_q, w13_s, w2_q, w2_s, top_k):
    """Float64, library routines only: torch's float8 conversion (through the weight quantiser) for the
    activations, the torch-derived code table for every stored value, dense NumPy products over EVERY expert,
    a dense [T,E] routing-weight matrix that is zero outside the top-k."""
    x = bits_to_f64(x_bits)
    xq, xs = quantize_mxfp8(torch.from_numpy(x.astype(np.float32)))
    xd = dequant(xq.numpy(), xs.numpy())
    w13, w2 = dequant(w13_q, w13_s), dequant(w2_q, w2_s)
    l = np.asarray(logits, dtype=np.float64)
    T, E = l.shape
    I = w13.shape[1] // 2
    order = np.argsort(-l, axis=1, kind="stable")[:, :top_k]
    sel = np.take_along_axis(l, order, axis=1)
    z = np.exp(sel - sel.max(axis=1, keepdims=True))
    dense_w = np.zeros((T, E))
    np.put_along_axis(dense_w, order, z / z.sum(axis=1, keepdims=True), axis=1)
    out = np.zeros_like(x)
    for e in range(E):
        g = xd @ w13[e, :I].T
        u = xd @ w13[e, I:].T
        h = g / (1.0 + np.exp(-g)) * u
        hq, hs = quantize_mxfp8(torch.from_numpy(h))   # float64 in, so the decision is taken in float64
        out += dense_w[:, e:e + 1] * (dequant(hq.numpy(), hs.numpy()) @ w2[e].T)
    return out


@pytest.mark.parametrize("T,H,I,E,k", [(5, 64, 32, 4, 2), (9, 128, 96, 6, 3), (3, 256, 128, 3, 3)])
def test_layer_matches_float64_brute_force(T, H, I, E, k):
    inp = make_mxfp8_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=False), seed=T)
    args = (bf16_bits(inp["x"]), inp["router_logits"].numpy(), inp["w13_q"].numpy(), inp["w13_s"].numpy(),
            inp["w2_q"].numpy(), inp["w2_s"].numpy())
    want = bruteforce_mx_layer(*args, k)
    got = moe_oracle.get("f64").forward_mxfp8(*args, k)
    assert np.allclose(got, want, rtol=1e-9, atol=1e-9)
    got32 = moe_oracle.get("f32").forward_mxfp8(*args, k)
    # float: the rare h code that flips at a rounding boundary moves one of I terms by one E4M3 step
    assert np.abs(got32 - want).max() <= 2e-2 * (1 + np.abs(want).max())
    assert np.median(np.abs(got32 - want)) <= 1e-4


def test_layer_is_close_to_the_unquantised_layer():
    """Each stored value is within 2^-4 of the value it stands for, relatively; the layer's error stays a
    small fraction of its output's scale."""
    inp = make_mxfp8_inputs(dict(T=16, H=256, I=128, E=4, top_k=2, skew=False), seed=7)
    o = moe_oracle.get("f64")
    q = o.forward_mxfp8(bf16_bits(inp["x"]), inp["router_logits"].numpy(), inp["w13_q"].numpy(), inp["w13_s"].numpy(),
                        inp["w2_q"].numpy(), inp["w2_s"].numpy(), 2)
    full = o.forward(bf16_bits(inp["x"]), inp["router_logits"].numpy(), bf16_bits(inp["w13"]), bf16_bits(inp["w2"]), 2)
    rms = np.sqrt(np.mean(full ** 2))
    assert np.sqrt(np.mean((q - full) ** 2)) < 0.08 * rms
    assert np.sqrt(np.mean((q - full) ** 2)) > 1e-4 * rms  # and it IS a quantised computation


def test_intermediates_are_consistent():
    inp = make_mxfp8_inputs(dict(T=6, H=128, I=64, E=4, top_k=2, skew=False), seed=9)
    o = moe_oracle.get("f32")
    out, h_pre, h_q, h_s = o.forward_mxfp8(bf16_bits(inp["x"]), inp["router_logits"].numpy(), inp["w13_q"].numpy(),
                                           inp["w13_s"].numpy(), inp["w2_q"].numpy(), inp["w2_s"].numpy(), 2,
                                           intermediates=True)
    c, s = o.mx_quantize(h_pre)
    assert np.array_equal(c, h_q) and np.array_equal(s, h_s)
    # quantisation error of a stored value: at most half a step of its binade, 2^-4 relative for normal codes
    err = np.abs(dequant(h_q, h_s) - h_pre)
    bound = np.maximum(np.abs(h_pre) * 2.0 ** -4, np.repeat(np.exp2(h_s.astype(np.float64) - 127), 32, axis=1) * 2.0 ** -10)
    sat = np.abs(dequant(h_q, h_s)) >= 448 * np.repeat(np.exp2(h_s.astype(np.float64) - 127), 32, axis=1)
    assert np.all((err <= bound) | sat)


def test_non_finite_token_poisons_only_itself():
    inp = make_mxfp8_inputs(dict(T=4, H=64, I=32, E=2, top_k=1, skew=False), seed=11)
    x = inp["x"].clone()
    x[2, 5] = float("inf")
    out = moe_oracle.get("f32").forward_mxfp8(bf16_bits(x), inp["router_logits"].numpy(), inp["w13_q"].numpy(),
                                              inp["w13_s"].numpy(), inp["w2_q"].numpy(), inp["w2_s"].numpy(), 1)
    assert np.all(np.isnan(out[2])) and np.all(np.isfinite(out[[0, 1, 3]]))


def test_sampled_form_equals_the_whole_layer_on_those_tokens():
    inp = make_mxfp8_inputs(dict(T=12, H=64, I=64, E=6, top_k=2, skew=False), seed=13)
    o = moe_oracle.get("f32")
    args = (bf16_bits(inp["x"]), inp["router_logits"].numpy())
    w = [inp[n].numpy() for n in ("w13_q", "w13_s", "w2_q", "w2_s")]
    full = o.forward_mxfp8(*args, *w, 2)
    tokens = np.array([11, 0, 5], dtype=np.int32)
    ids, _ = o.route(args[1], 2)
    need = {int(e) for t in tokens for e in ids[t]}
    experts = {e: tuple(a[e] for a in w) for e in need}
    got = o.forward_mxfp8_sampled(*args, experts, 64, 2, tokens)
    assert np.array_equal(got, full[tokens])
    missing = {e: v for e, v in experts.items() if e != int(ids[11][0])}
    with pytest.raises(RuntimeError):
        o.forward_mxfp8_sampled(*args, missing, 64, 2, tokens)
