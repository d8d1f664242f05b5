"""GPU parity at the full workload sizes, in the launch configuration bench.py times.

The CPU oracle cannot evaluate these layers in full, so each workload is checked three ways:
routing and permutation bit-exactly on all tokens (cheap on the CPU); the layer output on a
sample of tokens the oracle computes one by one; and every intermediate and output element
against the CUDA-core validation kernels, which share no code with the tcgen05 path.
"""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
from paper_2602_19128_b200.inputs import CONFIGS, bf16_bits
from tests.weight_quantizers import quantize_mxfp8
from tests.gpu_common import (OUT_TOL, Guarded, assert_close_out, assert_routing_exact, bf16_to_f64, check_guards,
                              gpu_inputs, guarded_out, mx_regions, run_forward)

pytestmark = pytest.mark.gpu


def edge_tokens(off: np.ndarray, s2f: np.ndarray, T: int, E: int, k: int, tile_bound: int) -> np.ndarray:
    """Tokens the oracle evaluates one by one, chosen from ITS permutation so that they sit where an indexing
    mistake would show: the first and last row of the heaviest expert, the rows on both sides of that expert's
    segment, the last row of its first token tile and the first row of the next (when it has several), a token of
    an expert with exactly one row (when there is one), one routed to the highest-indexed active expert (the
    largest weight offsets), the first and last token, and six drawn at random.  At most 16."""
    counts = np.diff(off)
    rows = []
    heavy = int(np.argmax(counts))
    b, c = int(off[heavy]), int(counts[heavy])
    rows += [b, b + c - 1, max(b - 1, 0), min(b + c, len(s2f) - 1)]
    n_tiles = 1 if c <= tile_bound else -(-c // min(tile_bound, 256))
    if n_tiles > 1:
        per = -(-(-(-c // n_tiles)) // 16) * 16
        rows += [b + per - 1, b + per]
    single = np.flatnonzero(counts == 1)
    if len(single):
        rows.append(int(off[single[-1]]))
    last_active = int(np.flatnonzero(counts > 0)[-1])
    rows.append(int(off[last_active + 1]) - 1)
    rng = np.random.default_rng(0)
    tokens = [int(s2f[r]) // k for r in rows] + [0, T - 1] + list(rng.choice(T, size=6, replace=False))
    return np.unique(np.asarray(tokens)).astype(np.int32)


def close_on_device(a: torch.Tensor, b: torch.Tensor, what: str):
    a, b = a.float(), b.float()
    assert torch.isfinite(a).all(), what
    bad = (a - b).abs() > OUT_TOL * (1 + b.abs())
    assert not bad.any(), f"{what}: {int(bad.sum())} elements differ beyond tolerance"


@pytest.mark.parametrize("name", ["mixtral", "dsv3_decode", "skewed", "dsv3_prefill"])
def test_full_size_workload(name):
    cfg = CONFIGS[name]
    T, H, I, E, k = (cfg[n] for n in ("T", "H", "I", "E", "top_k"))
    inp = gpu_inputs(name, seed=0)
    out, views, ws = run_forward(inp)

    # 1. routing and permutation, all tokens, bit-exact
    o = moe_oracle.get("f32")
    logits = inp["router_logits"].cpu().numpy()
    ids, w = o.route(logits, k)
    off, s2f, f2s = o.permute(ids, E)
    assert_routing_exact(views, ids, w, off, s2f, f2s)
    assert torch.equal(views["x_perm"].view(torch.int16),
                       inp["x"][views["sorted_to_flat"].long() // k].view(torch.int16))

    # 2. sampled tokens against the oracle: tile and segment edges, 64-bit weight offsets, and a seeded draw
    tokens = edge_tokens(off, s2f, T, E, k, moe.moe_token_tile_rows(T, H, I, E, k))
    assert 8 <= len(tokens) <= 16
    need = sorted({int(e) for t in tokens for e in ids[t]})
    experts = {e: (bf16_bits(inp["w13"][e]), bf16_bits(inp["w2"][e])) for e in need}
    ref = o.forward_sampled(bf16_bits(inp["x"]), logits, experts, I, k, tokens)
    assert_close_out(bf16_to_f64(out[torch.from_numpy(tokens).long().cuda()]), ref, f"{name} sampled out")

    # 3. run-to-run determinism
    out_again, _, ws2 = run_forward(inp)
    assert torch.equal(out.view(torch.int16), out_again.view(torch.int16))
    del ws2, out_again

    # 4. every element of h, y and out against the CUDA-core validation kernels
    h, y = views["h"].clone(), views["y"].clone()
    del ws, views
    out_v, views_v, _ = run_forward(inp, flags=moe.MOE_FLAG_VALIDATION_GEMM)
    close_on_device(h, views_v["h"], f"{name} h")
    close_on_device(y, views_v["y"], f"{name} y")
    close_on_device(out, out_v, f"{name} out")


@pytest.mark.parametrize("name", ["mixtral", "dsv3_decode", "skewed", "dsv3_prefill"])
def test_full_size_workload_mxfp8(name):
    """The MX FP8 layer at full size (wide-tile CTA-pair kernel for the prefill-sized batches, 160-row pair tiles
    for the Mixtral shape, one-CTA kernel for the decode-sized one): routing bit-exact on all tokens, quantised token rows bit-exact on a sample,
    the output of sampled tokens against the oracle, and run-to-run determinism."""
    cfg = CONFIGS[name]
    T, H, I, E, k = (cfg[n] for n in ("T", "H", "I", "E", "top_k"))
    inp = gpu_inputs(name, seed=0)
    w13_q, w13_s = quantize_mxfp8(inp["w13"])
    inp["w13"] = None
    w2_q, w2_s = quantize_mxfp8(inp["w2"])
    inp["w2"] = None
    sf13, sf2 = moe.moe_mxfp8_pack_scales(w13_s, True), moe.moe_mxfp8_pack_scales(w2_s, False)

    def run():
        wg = Guarded(moe.moe_mxfp8_workspace_bytes(T, H, I, E, k), "cuda")
        ws = wg.inner
        og, out = guarded_out(T, H, "cuda")
        moe.moe_forward_mxfp8(inp["x"], inp["router_logits"], w13_q, sf13, w2_q, sf2, k, out, ws)
        assert moe.moe_last_status(ws) == moe.MOE_OK
        check_guards(wg, og, moe.moe_mxfp8_workspace_layout(T, H, I, E, k), mx_regions(T, H, I, E, k), f"{name} mxfp8")
        return out, ws

    out, ws = run()
    views = moe.mx_workspace_views(ws, T, H, I, E, k)
    o = moe_oracle.get("f32")
    logits = inp["router_logits"].cpu().numpy()
    ids, w = o.route(logits, k)
    off, s2f, f2s = o.permute(ids, E)
    assert_routing_exact(views, ids, w, off, s2f, f2s)

    tokens = edge_tokens(off, s2f, T, E, k, int(views["tile_rows"]))
    assert 8 <= len(tokens) <= 16
    xc, _ = o.mx_quantize(inp["x"][torch.from_numpy(tokens).long().cuda()].float().cpu().numpy())
    for n_i, t in enumerate(tokens):  # every sorted row of a sampled token holds that token's codes
        rows = f2s[t * k:(t + 1) * k]
        got = views["x_q"][torch.from_numpy(rows).long().cuda()].cpu().numpy()
        assert np.array_equal(got, np.broadcast_to(xc[n_i], got.shape))

    need = sorted({int(e) for t in tokens for e in ids[t]})
    experts = {e: (w13_q[e].cpu().numpy(), w13_s[e].cpu().numpy(), w2_q[e].cpu().numpy(), w2_s[e].cpu().numpy()) for e in need}
    ref = o.forward_mxfp8_sampled(bf16_bits(inp["x"]), logits, experts, I, k, tokens)
    assert_close_out(bf16_to_f64(out[torch.from_numpy(tokens).long().cuda()]), ref, f"{name} mxfp8 sampled out")

    del views, ws
    out_again, _ = run()
    assert torch.equal(out.view(torch.int16), out_again.view(torch.int16))
