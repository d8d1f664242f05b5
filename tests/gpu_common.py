"""Helpers for the GPU parity tests: run the CUDA path through the C ABI and fetch its results."""
from __future__ import annotations

import numpy as np
import torch

import paper_2602_19128_b200 as moe
from paper_2602_19128_b200.inputs import bf16_bits, make_inputs

OUT_TOL = 2e-2      # |gpu - oracle| <= OUT_TOL * (1 + |oracle|), every element (workload definition)
WEIGHT_TOL = 1e-5   # routing weights: fp32 exp/div differ between host libm and the GPU


def run_forward(inp: dict, flags: int = 0, poison: bool = True):
    """moe_forward on device tensors.  Returns (out bf16 [T,H] on device, workspace views)."""
    x, logits, w13, w2, k = inp["x"], inp["router_logits"], inp["w13"], inp["w2"], inp["top_k"]
    T, H = x.shape
    E, I2, _ = w13.shape
    I = I2 // 2
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), x.device)
    if poison:
        ws.fill_(0xFF)  # bf16 0xFFFF is a NaN: anything read before it is written shows up
    out = torch.full((T, H), float("nan"), dtype=torch.bfloat16, device=x.device)
    moe.moe_forward(x, logits, w13, w2, k, out, ws, flags=flags)
    status = moe.moe_last_status(ws)
    assert status == moe.MOE_OK, moe.moe_status_string(status)
    return out, moe.workspace_views(ws, T, H, I, E, k), ws


def to_host_case(inp: dict) -> dict:
    return dict(x=bf16_bits(inp["x"]), logits=inp["router_logits"].cpu().numpy(), w13=bf16_bits(inp["w13"]),
                w2=bf16_bits(inp["w2"]), k=inp["top_k"])


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def assert_close_out(gpu: np.ndarray, ref: np.ndarray, what: str = "out"):
    assert np.isfinite(gpu).all(), f"{what}: non-finite values"
    err = np.abs(gpu - ref)
    bound = OUT_TOL * (1.0 + np.abs(ref))
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), f"{what}: worst at {worst}: gpu={gpu[worst]} ref={ref[worst]}"


def assert_routing_exact(views: dict, ids, w, off, s2f, f2s):
    assert np.array_equal(views["topk_ids"].cpu().numpy(), ids), "topk_ids"
    assert np.array_equal(views["expert_offsets"].cpu().numpy(), off), "expert_offsets"
    assert np.array_equal(views["sorted_to_flat"].cpu().numpy(), s2f), "sorted_to_flat"
    assert np.array_equal(views["flat_to_sorted"].cpu().numpy(), f2s), "flat_to_sorted"
    np.testing.assert_allclose(views["topk_weights"].cpu().numpy(), w, rtol=0, atol=WEIGHT_TOL)


def gpu_inputs(cfg, seed=0):
    return make_inputs(cfg, seed=seed, device="cuda")
