"""GPU parity of the grouped sigmoid router (sigmoid scores, selection bias, group-limited top-k, scaled weights):
ids, offsets and the permutation bit for bit against the oracle (both evaluate the selection in binary32 with the
same sequence of correctly rounded operations), weights to fp32 rounding, and the layer output through it."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
from paper_2602_19128_b200.inputs import bf16_bits, make_inputs
from tests.gpu_common import assert_close_out, bf16_to_f64

pytestmark = pytest.mark.gpu


def run_route(logits, k, n_group, topk_group, bias, scale):
    T, E = logits.shape
    dev = logits.device
    ids = torch.full((T, k), -1, dtype=torch.int32, device=dev)
    w = torch.full((T, k), float("nan"), dtype=torch.float32, device=dev)
    off = torch.full((E + 1,), -1, dtype=torch.int32, device=dev)
    s2f = torch.full((T * k,), -1, dtype=torch.int32, device=dev)
    f2s = torch.full((T * k,), -1, dtype=torch.int32, device=dev)
    ws = moe.alloc_workspace(moe.moe_route_workspace_bytes(T, E, k), dev)
    ws.fill_(0xFF)
    router = moe.grouped_router(n_group, topk_group, bias, scale)
    moe.moe_route_grouped(logits, k, router, ids, w, off, s2f, f2s, ws)
    torch.cuda.synchronize()
    return [t.cpu().numpy() for t in (ids, w, off, s2f, f2s)]


# T, E, k, n_group, topk_group: groups inside a register (G < 32), exactly a register (G = 32), several registers
# (G > 32), groups of one, a single group, E below 32, both router launch forms (fused up to 1024 tokens)
CASES = [
    (257, 256, 8, 8, 4),      # the published setting: 8 groups of 32, 4 eligible
    (100, 64, 6, 8, 3),       # G = 8
    (64, 32, 4, 32, 5),       # groups of one
    (50, 16, 16, 1, 1),       # one group, every expert chosen
    (300, 256, 8, 2, 1),      # G = 128: four registers per group
    (200, 128, 8, 2, 2),      # G = 64
    (1500, 256, 8, 8, 4),     # three-kernel router
    (77, 48, 5, 3, 2),        # E not a multiple of 32, G = 16
    (1, 8, 2, 4, 2),
    (90, 64, 5, 64, 9),       # more groups than lanes (groups of one): the per-register ranking path
    (60, 256, 8, 128, 6),     # 128 groups of two
    (40, 256, 32, 8, 4),      # top_k = 32
]


@pytest.mark.parametrize("T,E,k,n_group,topk_group", CASES)
def test_grouped_route_matches_oracle(T, E, k, n_group, topk_group):
    g = torch.Generator().manual_seed(T + E)
    logits = (torch.randn((T, E), generator=g) * 1.5).cuda()
    bias = (torch.randn(E, generator=g) * 0.2).cuda()
    ids, w, off, s2f, f2s = run_route(logits, k, n_group, topk_group, bias, 2.5)
    o = moe_oracle.get("f32")
    want_ids, want_w = o.route_grouped(logits.cpu().numpy(), k, n_group, topk_group, bias=bias.cpu().numpy(), scale=2.5)
    assert np.array_equal(ids, want_ids)
    assert np.array_equal(w, want_w)          # the same binary32 operations in the same order
    want_off, want_s2f, want_f2s = o.permute(want_ids, E)
    assert np.array_equal(off, want_off) and np.array_equal(s2f, want_s2f) and np.array_equal(f2s, want_f2s)


def test_grouped_route_without_bias_and_with_ties():
    logits = torch.zeros((40, 64), device="cuda")
    logits[:, 37] = 1.0
    ids, w, *_ = run_route(logits, 4, 8, 2, None, 1.0)
    want_ids, want_w = moe_oracle.get("f32").route_grouped(logits.cpu().numpy(), 4, 8, 2)
    assert np.array_equal(ids, want_ids) and np.array_equal(w, want_w)
    assert ids[0].tolist() == [37, 0, 1, 2]   # group 4 wins, then group 0 on the tie; experts in index order


def test_grouped_route_rejects_settings_outside_the_envelope():
    logits = torch.zeros((4, 48), device="cuda")
    ids = torch.empty((4, 2), dtype=torch.int32, device="cuda")
    w = torch.empty((4, 2), dtype=torch.float32, device="cuda")
    off = torch.empty(49, dtype=torch.int32, device="cuda")
    s2f, f2s = torch.empty(8, dtype=torch.int32, device="cuda"), torch.empty(8, dtype=torch.int32, device="cuda")
    ws = moe.alloc_workspace(moe.moe_route_workspace_bytes(4, 48, 2), "cuda")
    for n_group, topk_group, want in ((5, 1, -3), (4, 1, -3), (3, 4, -3), (0, 1, -2), (48, 1, -3)):
        st = moe.moe_route_grouped(logits, 2, moe.grouped_router(n_group, topk_group), ids, w, off, s2f, f2s, ws, check=False)
        assert st == want, (n_group, topk_group, st)   # -3 unsupported (48/4 = 12 is not a power of two; 1 group of 1 < k), -2 shape


@pytest.mark.parametrize("flags", [0, moe.MOE_FLAG_SINGLE_CTA_GEMM])
def test_layer_with_the_grouped_router(flags):
    cfg = dict(T=200, H=256, I=128, E=64, top_k=6, skew=False)
    inp = make_inputs(cfg, seed=5, device="cuda")
    bias = torch.linspace(-0.3, 0.3, 64).cuda()
    T, H, I, E, k = 200, 256, 128, 64, 6
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), "cuda")
    ws.fill_(0xFF)
    out = torch.full((T, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    moe.moe_forward_grouped(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], k, moe.grouped_router(8, 3, bias, 2.5),
                            out, ws, flags=flags)
    assert moe.moe_last_status(ws) == moe.MOE_OK
    o = moe_oracle.get("f32")
    logits = inp["router_logits"].cpu().numpy()
    ids, _ = o.route_grouped(logits, k, 8, 3, bias=bias.cpu().numpy(), scale=2.5)
    views = moe.workspace_views(ws, T, H, I, E, k)
    assert np.array_equal(views["topk_ids"].cpu().numpy(), ids)
    experts = {e: (bf16_bits(inp["w13"][e]), bf16_bits(inp["w2"][e])) for e in range(E)}
    ref = o.forward_sampled_grouped(bf16_bits(inp["x"]), logits, experts, I, k, np.arange(T), 8, 3, bias=bias.cpu().numpy(),
                                    scale=2.5)
    # the weights sum to 2.5 instead of 1, and the tolerance scales with them
    err = np.abs(bf16_to_f64(out) - ref)
    assert np.all(err <= 2e-2 * (2.5 + np.abs(ref)))
