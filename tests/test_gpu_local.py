"""GPU parity of moe_forward_local (only the experts resident on this device are computed)."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
from paper_2602_19128_b200.inputs import bf16_bits
from tests.gpu_common import (WEIGHT_TOL, Guarded, assert_close_out, bf16_to_f64, check_guards, gpu_inputs, guarded_out,
                              layer_regions)

pytestmark = pytest.mark.gpu


def run_local(inp, lo, n, flags=0):
    x, logits, k = inp["x"], inp["router_logits"], inp["top_k"]
    T, H = x.shape
    E = logits.shape[1]
    w13 = inp["w13"][lo:lo + n].contiguous()
    w2 = inp["w2"][lo:lo + n].contiguous()
    I = w13.shape[1] // 2
    wg = Guarded(moe.moe_workspace_bytes(T, H, I, E, k), x.device)
    ws = wg.inner
    og, out = guarded_out(T, H, x.device)
    moe.moe_forward_local(x, logits, w13, w2, k, lo, out, ws, flags=flags)
    assert moe.moe_last_status(ws) == moe.MOE_OK
    check_guards(wg, og, moe.moe_workspace_layout(T, H, I, E, k), layer_regions(T, H, I, E, k, n), "moe_forward_local")
    return out, moe.workspace_views(ws, T, H, I, E, k), ws


# T, H, I, E, k, local offset, local count
CASES = [
    (64, 128, 128, 8, 2, 2, 3),
    (200, 256, 256, 16, 4, 0, 4),        # first quarter
    (200, 256, 256, 16, 4, 12, 4),       # last quarter
    (256, 512, 256, 256, 8, 64, 32),     # the paper's setting: 32 resident experts of 256, top-8
    (700, 256, 256, 4, 2, 1, 2),         # ~350 rows per resident expert: CTA-pair kernel, two token tiles
    (40, 128, 64, 8, 1, 7, 1),           # a single resident expert
]


@pytest.mark.parametrize("flags", [moe.MOE_FLAG_VALIDATION_GEMM, moe.MOE_FLAG_NONE], ids=["cuda_core", "tcgen05"])
@pytest.mark.parametrize("T,H,I,E,k,lo,n", CASES)
def test_local_subset_matches_oracle(T, H, I, E, k, lo, n, flags):
    inp = gpu_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=False), seed=1)
    out, views, _ = run_local(inp, lo, n, flags)
    o = moe_oracle.get("f32")
    logits = inp["router_logits"].cpu().numpy()
    ids, w = o.route(logits, k)
    off, s2f, f2s = o.permute_local(ids, lo, n)
    assert np.array_equal(views["topk_ids"].cpu().numpy(), ids)
    np.testing.assert_allclose(views["topk_weights"].cpu().numpy(), w, rtol=0, atol=WEIGHT_TOL)
    assert np.array_equal(views["expert_offsets"].cpu().numpy()[:n + 1], off)
    assert np.array_equal(views["flat_to_sorted"].cpu().numpy(), f2s)
    assert np.array_equal(views["sorted_to_flat"].cpu().numpy()[:off[-1]], s2f[:off[-1]])
    ref = o.forward_local(bf16_bits(inp["x"]), logits, bf16_bits(inp["w13"][lo:lo + n]), bf16_bits(inp["w2"][lo:lo + n]),
                          E, k, lo)
    assert_close_out(bf16_to_f64(out), ref, "local out")


def test_all_experts_local_equals_moe_forward_bit_for_bit():
    inp = gpu_inputs(dict(T=100, H=128, I=128, E=8, top_k=2, skew=False), seed=2)
    out_local, _, _ = run_local(inp, 0, 8)
    out = torch.empty_like(out_local)
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(100, 128, 128, 8, 2), "cuda")
    moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], 2, out, ws)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), out_local.view(torch.int16))


def test_partial_outputs_of_a_partition_add_up_to_the_full_layer():
    inp = gpu_inputs(dict(T=128, H=256, I=128, E=16, top_k=4, skew=False), seed=3)
    full = moe_oracle.get("f32").forward(bf16_bits(inp["x"]), inp["router_logits"].cpu().numpy(), bf16_bits(inp["w13"]),
                                         bf16_bits(inp["w2"]), 4)
    total = np.zeros_like(full, dtype=np.float64)
    for lo in (0, 4, 8, 12):
        part, _, _ = run_local(inp, lo, 4)
        total += bf16_to_f64(part)
    assert_close_out(total, full, "sum of partial outputs")


def test_no_token_routed_to_the_resident_experts_gives_zeros_and_bad_ranges_are_rejected():
    inp = gpu_inputs(dict(T=32, H=128, I=64, E=8, top_k=2, skew=False), seed=4)
    inp["router_logits"][:, 6:] = -50.0       # nobody picks experts 6, 7
    out, views, ws = run_local(inp, 6, 2)
    assert (out == 0).all() and int(views["expert_offsets"][2]) == 0 and (views["flat_to_sorted"] == -1).all()
    w13, w2 = inp["w13"][:2].contiguous(), inp["w2"][:2].contiguous()
    assert moe.moe_forward_local(inp["x"], inp["router_logits"], w13, w2, 2, 7, out, ws, check=False) == -2  # 7 + 2 > 8
    assert moe.moe_forward_local(inp["x"], inp["router_logits"], w13, w2, 2, -1, out, ws, check=False) == -2
