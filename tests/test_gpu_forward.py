"""GPU parity: the whole layer through moe_forward against the CPU oracle (element by element)."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
from tests.gpu_common import (assert_close_out, assert_routing_exact, bf16_to_f64, gpu_inputs, run_forward,
                              to_host_case)

pytestmark = pytest.mark.gpu

# (T, H, I, E, k, skew): sizes the oracle finishes in seconds, chosen to span several feature tiles,
# several token tiles per expert, ragged tails, empty experts and every token-tile bound (32..256).
SMALL = [
    (16, 256, 512, 8, 2, False),      # the tiny workload
    (1, 128, 64, 4, 1, False),        # one token, one feature tile, three empty experts
    (7, 128, 192, 3, 3, False),       # k = E
    (200, 256, 384, 8, 2, False),     # ~50 rows per expert: N = 64 tiles with a ragged tail
    (700, 128, 128, 4, 2, False),     # ~350 rows per expert: two token tiles per expert
    (300, 128, 64, 64, 4, True),      # skewed: hot experts over 256 rows, most experts empty
    (128, 384, 128, 256, 8, False),   # decode-like: ~4 rows per expert, N = 16
    (96, 128, 256, 8, 8, False),      # k = E = 8: every expert sees every token
    (700, 256, 256, 4, 2, False),     # CTA-pair kernel for both GEMMs, two token tiles per expert
    (300, 512, 384, 2, 2, False),     # CTA-pair kernel, 300 rows per expert: two ragged tiles of N = 160
    (130, 256, 128, 1, 1, False),     # one expert, 130 rows: pair tile with a nearly empty second half
    (700, 256, 256, 2, 1, False),     # ~350 rows per expert: two weight slabs per CTA in the gate/up GEMM
    (600, 512, 512, 2, 2, False),     # 600 rows per expert: three token tiles of 208, two 512-row pair tiles
    (520, 256, 256, 4, 2, False),     # ~260 rows per expert: wide-tile kernel, one tile of up to 320 rows per expert
    (900, 256, 128, 8, 2, True),      # skewed, 225 rows on average: bound 320, hot experts cut into 256-row tiles
    (1200, 512, 384, 8, 2, False),    # 300 rows per expert: bound 384, consecutive tiles overlap in tensor memory
    (2600, 256, 128, 16, 2, False),   # 325 rows per expert: bound 384 with the three-kernel router
]


def oracle_everything(case):
    o = moe_oracle.get("f32")
    ids, w = o.route(case["logits"], case["k"])
    E = case["w13"].shape[0]
    off, s2f, f2s = o.permute(ids, E)
    h, y = o.sorted_intermediates(case["x"], case["w13"], case["w2"], ids, s2f)
    out = o.forward(case["x"], case["logits"], case["w13"], case["w2"], case["k"])
    return ids, w, off, s2f, f2s, h, y, out


@pytest.mark.parametrize("flags", [moe.MOE_FLAG_VALIDATION_GEMM, moe.MOE_FLAG_SINGLE_CTA_GEMM,
                                   moe.MOE_FLAG_TWO_SLAB_GEMM, moe.MOE_FLAG_NARROW_TILES, moe.MOE_FLAG_NONE],
                         ids=["cuda_core", "tcgen05_single", "tcgen05_two_slab", "tcgen05_narrow", "tcgen05"])
@pytest.mark.parametrize("T,H,I,E,k,skew", SMALL)
def test_forward_matches_oracle(T, H, I, E, k, skew, flags):
    inp = gpu_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=skew), seed=0)
    out, views, _ = run_forward(inp, flags=flags)
    ids, w, off, s2f, f2s, h, y, ref = oracle_everything(to_host_case(inp))
    assert_routing_exact(views, ids, w, off, s2f, f2s)
    x_perm = views["x_perm"].cpu().view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(x_perm, to_host_case(inp)["x"][s2f // k]), "gathered rows"
    assert_close_out(bf16_to_f64(views["h"]), h, "h")
    assert_close_out(bf16_to_f64(views["y"]), y, "y")
    assert_close_out(bf16_to_f64(out), ref, "out")


@pytest.mark.parametrize("T,H,I,E,k,skew", [(520, 256, 256, 4, 2, False), (900, 256, 128, 8, 2, True),
                                            (1200, 512, 384, 8, 2, False), (700, 256, 256, 2, 1, False)])
def test_gather_in_load_matches_oracle(T, H, I, E, k, skew):
    """The wide-tile gate/up GEMM fetching token rows from x by index (no expert-contiguous copy): h, y and out
    against the oracle, and bit-identical to the path that reads the copy (same operands, same order)."""
    assert moe.moe_token_tile_rows(T, H, I, E, k) in (320, 384)
    inp = gpu_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=skew), seed=0)
    out, views, _ = run_forward(inp, flags=moe.MOE_FLAG_GATHER_IN_LOAD, x_perm_written=False)
    ids, w, off, s2f, f2s, h, y, ref = oracle_everything(to_host_case(inp))
    assert_routing_exact(views, ids, w, off, s2f, f2s)
    assert_close_out(bf16_to_f64(views["h"]), h, "h")
    assert_close_out(bf16_to_f64(views["y"]), y, "y")
    assert_close_out(bf16_to_f64(out), ref, "out")
    plain, _, _ = run_forward(inp)
    assert torch.equal(out.view(torch.int16), plain.view(torch.int16))


def test_forward_is_deterministic_and_leaves_inputs_alone():
    inp = gpu_inputs(dict(T=200, H=256, I=384, E=8, top_k=2), seed=3)
    before = {n: inp[n].clone() for n in ("x", "router_logits", "w13", "w2")}
    a, _, _ = run_forward(inp)
    b, _, _ = run_forward(inp)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    for n, t in before.items():
        assert torch.equal(t.view(torch.int16) if t.dtype == torch.bfloat16 else t,
                           inp[n].view(torch.int16) if t.dtype == torch.bfloat16 else inp[n])


def test_token_permutation_equivariance():
    inp = gpu_inputs(dict(T=64, H=128, I=128, E=8, top_k=2), seed=4)
    out, views, _ = run_forward(inp)
    perm = torch.randperm(64, generator=torch.Generator().manual_seed(0)).cuda()
    inp2 = dict(inp, x=inp["x"][perm].contiguous(), router_logits=inp["router_logits"][perm].contiguous())
    out2, views2, _ = run_forward(inp2)
    assert torch.equal(views["topk_ids"][perm], views2["topk_ids"])
    a, b = bf16_to_f64(out[perm]), bf16_to_f64(out2)
    assert (np.abs(a - b) <= 2e-2 * (1 + np.abs(a))).all()


def test_identical_experts_with_k_equal_E_is_one_dense_mlp():
    inp = gpu_inputs(dict(T=40, H=128, I=192, E=8, top_k=8), seed=6)
    inp["w13"] = inp["w13"][:1].repeat(8, 1, 1).contiguous()
    inp["w2"] = inp["w2"][:1].repeat(8, 1, 1).contiguous()
    out, views, _ = run_forward(inp)
    np.testing.assert_allclose(views["topk_weights"].sum(dim=1).cpu().numpy(), 1.0, atol=1e-5)
    x = inp["x"].double().cpu(); a = inp["w13"][0].double().cpu(); b = inp["w2"][0].double().cpu()
    ref = (torch.nn.functional.silu(x @ a[:192].T) * (x @ a[192:].T)) @ b.T
    assert_close_out(bf16_to_f64(out), ref.numpy(), "dense MLP")


def test_argument_validation_happens_before_any_launch():
    dev = "cuda"
    T, H, I, E, k = 16, 256, 512, 8, 2
    inp = gpu_inputs(dict(T=T, H=H, I=I, E=E, top_k=k))
    out = torch.zeros((T, H), dtype=torch.bfloat16, device=dev)
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), dev)
    small = moe.alloc_workspace(1024, dev)
    assert moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], k, out, small, check=False) == -5
    assert moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], E + 1, out, ws, check=False) == -2
    bad_h = torch.zeros((T, 200), dtype=torch.bfloat16, device=dev)
    bad_w13 = torch.zeros((E, 2 * I, 200), dtype=torch.bfloat16, device=dev)
    assert moe.moe_forward(bad_h, inp["router_logits"], bad_w13, inp["w2"], k, out, ws, check=False) == -3
    misaligned = ws[8:]
    assert moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], k, out, misaligned, check=False) == -4
    # T = 0 succeeds without touching anything
    empty = torch.empty((0, H), dtype=torch.bfloat16, device=dev)
    assert moe.moe_forward(empty, torch.empty((0, E), device=dev), inp["w13"], inp["w2"], k, empty, ws) == 0
    torch.cuda.synchronize()
    assert (out == 0).all()


def test_forward_host_buffers_match_device_buffers():
    inp = gpu_inputs(dict(T=200, H=256, I=384, E=8, top_k=2), seed=7)
    ref, _, _ = run_forward(inp)
    T, H = inp["x"].shape
    xh = inp["x"].cpu().pin_memory()
    lh = inp["router_logits"].cpu().pin_memory()
    oh = torch.zeros((T, H), dtype=torch.bfloat16).pin_memory()
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, 384, 8, 2), "cuda")
    moe.moe_forward_host(xh, lh, inp["w13"], inp["w2"], 2, oh, ws)
    assert moe.moe_last_status(ws) == 0
    assert torch.equal(oh.view(torch.int16), ref.cpu().view(torch.int16))


def test_forward_with_the_largest_top_k():
    inp = gpu_inputs(dict(T=24, H=128, I=64, E=64, top_k=32), seed=8)
    out, views, _ = run_forward(inp)
    ids, w, off, s2f, f2s, h, y, ref = oracle_everything(to_host_case(inp))
    assert_routing_exact(views, ids, w, off, s2f, f2s)
    assert_close_out(bf16_to_f64(out), ref, "out")
