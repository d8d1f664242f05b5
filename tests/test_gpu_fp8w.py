"""GPU parity of moe_forward_fp8w (FP8 E4M3 block-scaled expert weights) against the oracle."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
from paper_2602_19128_b200.inputs import bf16_bits
from tests.weight_quantizers import make_fp8w_inputs
from tests.gpu_common import (Guarded, assert_close_out, assert_routing_exact, bf16_to_f64, check_guards, guarded_out,
                              layer_regions)

pytestmark = pytest.mark.gpu


def run_fp8w(inp):
    T, H = inp["x"].shape
    E, I2, _ = inp["w13_q"].shape
    I, k = I2 // 2, inp["top_k"]
    wg = Guarded(moe.moe_workspace_bytes(T, H, I, E, k), "cuda")
    ws = wg.inner
    og, out = guarded_out(T, H, "cuda")
    moe.moe_forward_fp8w(inp["x"], inp["router_logits"], inp["w13_q"], inp["w13_scale"], inp["w2_q"], inp["w2_scale"], k,
                         out, ws)
    assert moe.moe_last_status(ws) == moe.MOE_OK
    check_guards(wg, og, moe.moe_workspace_layout(T, H, I, E, k), layer_regions(T, H, I, E, k), "moe_forward_fp8w")
    return out, moe.workspace_views(ws, T, H, I, E, k)


def oracle_out(inp):
    o = moe_oracle.get("f32")
    return o.forward_fp8w(bf16_bits(inp["x"]), inp["router_logits"].cpu().numpy(), inp["w13_q"].cpu().numpy(),
                          inp["w13_scale"].cpu().numpy(), inp["w2_q"].cpu().numpy(), inp["w2_scale"].cpu().numpy(),
                          inp["top_k"])


# T, H, I, E, k, skew: every token-tile bound (32..256), several K blocks, gate/up rows in different scale blocks
CASES = [
    (16, 256, 512, 8, 2, False),
    (1, 128, 128, 4, 1, False),
    (128, 384, 128, 256, 8, False),   # decode-like, N = 16
    (200, 256, 384, 8, 2, False),     # ~50 rows per expert
    (300, 128, 128, 64, 4, True),     # skewed, empty experts
    (700, 256, 256, 4, 2, False),     # two token tiles per expert, N up to 256
    (96, 128, 256, 8, 8, False),
]


@pytest.mark.parametrize("T,H,I,E,k,skew", CASES)
def test_fp8w_forward_matches_oracle(T, H, I, E, k, skew):
    inp = make_fp8w_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=skew), seed=0, device="cuda")
    out, views = run_fp8w(inp)
    o = moe_oracle.get("f32")
    ids, w = o.route(inp["router_logits"].cpu().numpy(), k)
    off, s2f, f2s = o.permute(ids, E)
    assert_routing_exact(views, ids, w, off, s2f, f2s)
    assert_close_out(bf16_to_f64(out), oracle_out(inp), "fp8w out")


def test_fp8w_with_unit_scales_equals_the_bf16_layer_bit_for_bit():
    """All E4M3 values are bf16 values, and a scale of 1 is exact in bf16: both paths see the same operands."""
    g = torch.Generator().manual_seed(0)
    T, H, I, E, k = 64, 256, 128, 4, 2
    table = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float()
    finite = torch.nonzero(~torch.isnan(table) & (table.abs() <= 1.0)).flatten()
    c13 = finite[torch.randint(len(finite), (E, 2 * I, H), generator=g)].to(torch.uint8).cuda()
    c2 = finite[torch.randint(len(finite), (E, H, I), generator=g)].to(torch.uint8).cuda()
    inp = dict(x=(torch.randn(T, H, generator=g) * 0.05).to(torch.bfloat16).cuda(),
               router_logits=torch.randn(T, E, generator=g).cuda(), top_k=k, w13_q=c13, w2_q=c2,
               w13_scale=torch.ones(E, 2 * I // 128, H // 128, device="cuda"),
               w2_scale=torch.ones(E, H // 128, I // 128, device="cuda"))
    out, _ = run_fp8w(inp)
    w13 = table.cuda()[c13.long()].to(torch.bfloat16)
    w2 = table.cuda()[c2.long()].to(torch.bfloat16)
    ref = torch.empty_like(out)
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), "cuda")
    moe.moe_forward(inp["x"], inp["router_logits"], w13, w2, k, ref, ws, flags=moe.MOE_FLAG_SINGLE_CTA_GEMM)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_fp8w_rejects_shapes_outside_its_envelope():
    inp = make_fp8w_inputs(dict(T=8, H=128, I=128, E=2, top_k=1, skew=False), seed=1, device="cuda")
    out = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda")
    ws = moe.alloc_workspace(1 << 20, "cuda")
    bad_q = torch.zeros((2, 2 * 192, 128), dtype=torch.uint8, device="cuda")     # I = 192 is not a multiple of 128
    bad_s = torch.ones((2, 3, 1), device="cuda")
    bad_q2 = torch.zeros((2, 128, 192), dtype=torch.uint8, device="cuda")
    assert moe.moe_forward_fp8w(inp["x"], inp["router_logits"], bad_q, bad_s, bad_q2, bad_s, 1, out, ws, check=False) == -3
