"""Helpers for the GPU parity tests: run the CUDA path through the C ABI and fetch its results."""
from __future__ import annotations

import numpy as np
import torch

import paper_2602_19128_b200 as moe
from paper_2602_19128_b200.inputs import bf16_bits, make_inputs

OUT_TOL = 2e-2      # |gpu - oracle| <= OUT_TOL * (1 + |oracle|), every element (workload definition)
WEIGHT_TOL = 1e-5   # routing weights: fp32 exp/div differ between host libm and the GPU


# ---- guard bands -------------------------------------------------------------------------------------------
# No memory checker runs on the GPU here, so the parity tests carry their own evidence that the kernels stay
# inside their buffers: the workspace and the result tensor of every call live inside larger allocations with a
# sentinel band on both sides, the workspace itself is pre-filled with a poison byte, and after the call the bands
# and the alignment gaps between the workspace's regions (and its staging area, which only the host-buffer entry
# points use) must be untouched.  An out-of-bounds WRITE of up to a band's width shows up as a changed byte.
GUARD_BYTES = 4096
SENTINEL = 0xA5
POISON = 0xFF   # bf16 0xFFFF is a NaN: anything read before it is written shows up as well


class Guarded:
    """`nbytes` of device memory (256-byte aligned) between two sentinel bands of GUARD_BYTES each."""

    def __init__(self, nbytes: int, device="cuda", fill: int = POISON):
        self.n = max(int(nbytes), 256)
        self.base = torch.empty(2 * GUARD_BYTES + self.n, dtype=torch.uint8, device=device)
        self.base[:GUARD_BYTES].fill_(SENTINEL)
        self.base[GUARD_BYTES + self.n:].fill_(SENTINEL)
        self.inner = self.base[GUARD_BYTES:GUARD_BYTES + self.n]
        assert self.inner.data_ptr() % 256 == 0
        self.inner.fill_(fill)

    def assert_bands_intact(self, what: str):
        lo, hi = self.base[:GUARD_BYTES], self.base[GUARD_BYTES + self.n:]
        assert bool((lo == SENTINEL).all()), f"{what}: bytes below the buffer were overwritten"
        assert bool((hi == SENTINEL).all()), f"{what}: bytes above the buffer were overwritten"


def guarded_out(T: int, H: int, device="cuda"):
    """A bf16 [T,H] result tensor filled with NaN between two sentinel bands; returns (guard, tensor)."""
    g = Guarded(T * H * 2, device)
    out = g.inner[:T * H * 2].view(torch.bfloat16).view(T, H)
    return g, out


def assert_gaps_untouched(ws: torch.Tensor, layout, used: dict, what: str):
    """`layout` is a ctypes layout struct of byte offsets, `used` maps a region's field name to the bytes the call may
    write there (regions not named are skipped).  Everything between the end of a region's used bytes and the start
    of the next region must still hold the poison byte the workspace was filled with."""
    skip = ("total_bytes", "sf_atoms", "tile_rows")
    offs = sorted((getattr(layout, n), n) for n, _ in layout._fields_ if n not in skip)
    ends = [o for o, _ in offs[1:]] + [int(layout.total_bytes)]
    for (off, name), end in zip(offs, ends):
        if name not in used:
            continue
        gap = ws[off + used[name]:end]
        assert bool((gap == POISON).all()), f"{what}: the gap after workspace region '{name}' was written"


def layer_regions(T: int, H: int, I: int, E: int, k: int, n_local=None) -> dict:
    """Bytes a moe_forward-family call may write in each region of its workspace (the staging area: none)."""
    n_local = E if n_local is None else n_local
    A = T * k
    n_chunks = (T + 31) // 32
    return dict(topk_ids=A * 4, topk_weights=A * 4, expert_offsets=(n_local + 1) * 4, sorted_to_flat=A * 4,
                flat_to_sorted=A * 4, route_scratch=(n_chunks * n_local + 3 * n_local + 1) * 4, x_perm=A * H * 2,
                h=A * I * 2, y=A * H * 2, staging=0)


def mx_regions(T: int, H: int, I: int, E: int, k: int, n_local=None) -> dict:
    """The same for the MX FP8 layer's workspace (its scale-atom regions are whole multiples of 512 bytes)."""
    n_local = E if n_local is None else n_local
    A = T * k
    n_chunks = (T + 31) // 32
    return dict(topk_ids=A * 4, topk_weights=A * 4, expert_offsets=(n_local + 1) * 4, sorted_to_flat=A * 4,
                flat_to_sorted=A * 4, route_scratch=(n_chunks * n_local + 3 * n_local + 1) * 4, x_q=A * H, h_q=A * I,
                y=A * H * 2, staging=0)


def check_guards(ws_guard: Guarded, out_guard: Guarded, layout, used: dict, what: str):
    torch.cuda.synchronize()
    ws_guard.assert_bands_intact(f"{what} workspace")
    out_guard.assert_bands_intact(f"{what} out")
    assert_gaps_untouched(ws_guard.inner, layout, used, what)


def run_forward(inp: dict, flags: int = 0, poison: bool = True, x_perm_written: bool = True):
    """moe_forward on device tensors, workspace and result between guard bands.  Returns (out bf16 [T,H] on device,
    workspace views, workspace)."""
    x, logits, w13, w2, k = inp["x"], inp["router_logits"], inp["w13"], inp["w2"], inp["top_k"]
    T, H = x.shape
    E, I2, _ = w13.shape
    I = I2 // 2
    wg = Guarded(moe.moe_workspace_bytes(T, H, I, E, k), x.device, POISON if poison else 0)
    ws = wg.inner
    og, out = guarded_out(T, H, x.device)
    moe.moe_forward(x, logits, w13, w2, k, out, ws, flags=flags)
    status = moe.moe_last_status(ws)
    assert status == moe.MOE_OK, moe.moe_status_string(status)
    if poison:
        regions = layer_regions(T, H, I, E, k)
        if not x_perm_written:  # gather-in-load: the region must stay untouched as a whole
            regions["x_perm"] = 0
        check_guards(wg, og, moe.moe_workspace_layout(T, H, I, E, k), regions, "moe_forward")
    else:
        wg.assert_bands_intact("moe_forward workspace")
        og.assert_bands_intact("moe_forward out")
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
