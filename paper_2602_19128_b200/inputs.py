"""Seeded synthetic inputs for the MoE layer (shapes, dtypes and distributions of the
benchmark workloads).  This module only draws random numbers and reshapes them: it holds
none of the layer's arithmetic, and it is the one module that both the CUDA path's callers
and the CPU oracle's callers share.

Recipe (all draws from one ``torch.Generator`` seeded per workload, in the order
x, router_logits, w13, w2):
  x              [T,H]     N(0,1)            drawn in fp32, rounded to bf16
  router_logits  [T,E]     N(0,1) fp32       (+ a per-expert bias for the skewed workload)
  w13            [E,2I,H]  N(0,1/H)          std H**-0.5, drawn in fp32, rounded to bf16
  w2             [E,H,I]   N(0,1/I)          std I**-0.5, drawn in fp32, rounded to bf16
The skewed workload adds bias_e = 2*ln(1/(e+1)**1.1) = -2.2*ln(e+1) to every token's logit of
expert e, so a few low-index experts receive most tokens and most experts receive none.
The bytes produced are what both sides consume; a CPU generator and a CUDA generator give
different streams, so a test draws once and hands the same tensors to both sides.
"""
from __future__ import annotations

import math

import numpy as np
import torch

CONFIGS = {
    # name: T tokens, H hidden, I intermediate, E experts, top_k, zipf-biased router
    "tiny": dict(T=16, H=256, I=512, E=8, top_k=2, skew=False),
    "mixtral": dict(T=512, H=4096, I=14336, E=8, top_k=2, skew=False),
    "dsv3_decode": dict(T=128, H=7168, I=2048, E=256, top_k=8, skew=False),
    "dsv3_prefill": dict(T=8192, H=7168, I=2048, E=256, top_k=8, skew=False),
    "skewed": dict(T=4096, H=4096, I=1536, E=128, top_k=8, skew=True),
}

# The paper's own deployment shape (Sec. 4.5: top-8 of 256 experts, 32 of them resident, hidden 7168), in
# bf16: the router sees 256 experts, weights exist only for experts [local_offset, local_offset + local).
LOCAL_CONFIGS = {
    "dsv3_local32_prefill": dict(T=8192, H=7168, I=2048, E=256, top_k=8, skew=False, local_offset=64, local=32),
    "dsv3_local32_decode": dict(T=128, H=7168, I=2048, E=256, top_k=8, skew=False, local_offset=64, local=32),
}


def zipf_bias(E: int) -> torch.Tensor:
    rank = torch.arange(1, E + 1, dtype=torch.float32)
    return (-2.2 * torch.log(rank)).to(torch.float32)


def _normal_bf16(shape, std: float, gen: torch.Generator, device, chunk_elems: int = 1 << 28) -> torch.Tensor:
    """N(0, std^2) in bf16, drawn in fp32 slabs along dim 0 so the fp32 temporary stays small."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    rows = shape[0]
    per_row = int(np.prod(shape[1:])) if len(shape) > 1 else 1
    step = max(1, chunk_elems // max(per_row, 1))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        slab = torch.randn((r1 - r0, *shape[1:]), generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            slab.mul_(std)
        out[r0:r1] = slab.to(torch.bfloat16)
    return out


def make_inputs(cfg, seed: int = 0, device="cpu") -> dict:
    """Draw one workload.  ``cfg`` is a name in CONFIGS or a dict with T,H,I,E,top_k[,skew]."""
    if isinstance(cfg, str):
        cfg = CONFIGS[cfg] if cfg in CONFIGS else LOCAL_CONFIGS[cfg]
    T, H, I, E = cfg["T"], cfg["H"], cfg["I"], cfg["E"]
    device = torch.device(device)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    x = _normal_bf16((T, H), 1.0, gen, device)
    logits = torch.randn((T, E), generator=gen, device=device, dtype=torch.float32)
    if cfg.get("skew", False):
        logits = logits + zipf_bias(E).to(device)
    n_experts = cfg.get("local", E)  # weights are drawn only for the resident experts
    w13 = _normal_bf16((n_experts, 2 * I, H), 1.0 / math.sqrt(H), gen, device)
    w2 = _normal_bf16((n_experts, H, I), 1.0 / math.sqrt(I), gen, device)
    return dict(x=x, router_logits=logits.contiguous(), w13=w13, w2=w2, T=T, H=H, I=I, E=E, top_k=cfg["top_k"],
                local_offset=cfg.get("local_offset", 0), local=n_experts)


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


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The uint16 bit pattern of a bf16 tensor, on the host, as a numpy array."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
