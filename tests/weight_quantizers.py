"""Offline weight quantisers for the FP8 / MX FP8 variants of the layer: harness code for the tests and the
benchmark, which prepare quantised weights as INPUTS of the library and of the oracle.  They are built from
torch's own float8 conversion and frexp / ldexp, independently of both the CUDA kernels and the C oracle (for
which they also serve as a library-built pin), and are deliberately kept out of the product package.
"""
from __future__ import annotations

import torch

from paper_2602_19128_b200.inputs import make_inputs

FP8_BLOCK = 128
E4M3_MAX = 448.0


def quantize_fp8_blocks(w: torch.Tensor):
    """Offline weight quantisation for the FP8 workloads: every 128 x 128 block of each expert's matrix
    [E, rows, cols] gets the fp32 scale amax / 448 (1 for an all-zero block) and its entries are rounded to
    E4M3 after division by it (torch's float8_e4m3fn conversion).  Returns (codes uint8 [E,rows,cols],
    scales f32 [E, rows/128, cols/128]).  This prepares inputs; the layer's own arithmetic starts from them."""
    E, R, C = w.shape
    assert R % FP8_BLOCK == 0 and C % FP8_BLOCK == 0
    codes = torch.empty((E, R, C), dtype=torch.uint8, device=w.device)
    scales = torch.empty((E, R // FP8_BLOCK, C // FP8_BLOCK), dtype=torch.float32, device=w.device)
    for e in range(E):  # one expert at a time keeps the fp32 temporaries small
        blocks = w[e].float().view(R // FP8_BLOCK, FP8_BLOCK, C // FP8_BLOCK, FP8_BLOCK)
        amax = blocks.abs().amax(dim=(1, 3))
        scale = torch.where(amax > 0, amax / E4M3_MAX, torch.ones_like(amax))
        q = (blocks / scale[:, None, :, None]).to(torch.float8_e4m3fn)
        codes[e] = q.view(torch.uint8).view(R, C)
        scales[e] = scale
    return codes, scales


def make_fp8w_inputs(cfg, seed: int = 0, device="cpu") -> dict:
    """make_inputs plus the FP8 block-scaled form of the expert weights (w13_q, w13_scale, w2_q, w2_scale)."""
    inp = make_inputs(cfg, seed=seed, device=device)
    inp["w13_q"], inp["w13_scale"] = quantize_fp8_blocks(inp["w13"])
    inp["w2_q"], inp["w2_scale"] = quantize_fp8_blocks(inp["w2"])
    return inp


MX_BLOCK = 32


def quantize_mxfp8(w: torch.Tensor):
    """Offline MX FP8 quantisation of a weight tensor [..., K] along K (OCP Microscaling, MXFP8 E4M3): every 32
    consecutive elements share the scale 2^(floor(log2(amax)) - 8), stored as the byte exponent + 127 (0 for an
    all-zero block), and are rounded to E4M3 after division by it (torch's float8_e4m3fn conversion after
    clamping to +-448).  Returns (codes uint8 [..., K], scale bytes uint8 [..., K/32]).  This prepares inputs;
    the layer's own arithmetic starts from them."""
    K = w.shape[-1]
    assert K % MX_BLOCK == 0
    lead = w.shape[:-1]
    codes = torch.empty(w.shape, dtype=torch.uint8, device=w.device)
    scales = torch.empty((*lead, K // MX_BLOCK), dtype=torch.uint8, device=w.device)
    flat_w, flat_c, flat_s = w.reshape(-1, K), codes.view(-1, K), scales.view(-1, K // MX_BLOCK)
    step = max(1, (1 << 24) // K)  # bound the fp32 temporaries
    for r0 in range(0, flat_w.shape[0], step):
        blocks = flat_w[r0:r0 + step].float().view(-1, K // MX_BLOCK, MX_BLOCK)
        amax = blocks.abs().amax(dim=2)
        _, ex = torch.frexp(amax)  # amax = m * 2^ex with m in [0.5, 1): floor(log2 amax) = ex - 1
        b = torch.where(amax > 0, (ex - 1 - 8 + 127).clamp(0, 254), torch.zeros_like(ex))
        scaled = torch.ldexp(blocks, (127 - b)[:, :, None].expand_as(blocks)).clamp(-E4M3_MAX, E4M3_MAX)
        flat_c[r0:r0 + step] = scaled.to(torch.float8_e4m3fn).view(torch.uint8).view(-1, K)
        flat_s[r0:r0 + step] = b.to(torch.uint8)
    return codes, scales


def make_mxfp8_inputs(cfg, seed: int = 0, device="cpu") -> dict:
    """make_inputs plus the MX FP8 form of the expert weights: w13_q [E,2I,H] / w13_s [E,2I,H/32] and
    w2_q [E,H,I] / w2_s [E,H,I/32] (codes and scale bytes, blocks of 32 along the contraction dimension)."""
    inp = make_inputs(cfg, seed=seed, device=device)
    inp["w13_q"], inp["w13_s"] = quantize_mxfp8(inp["w13"])
    inp["w2_q"], inp["w2_s"] = quantize_mxfp8(inp["w2"])
    return inp
