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


def make_inputs(cfg, seed: int = 0, device="cpu", weights=None) -> dict:
    """Draw one workload.  ``cfg`` is a name in CONFIGS or a dict with T,H,I,E,top_k[,skew].  ``weights`` =
    (w13, w2) of a workload with the same H, I and expert count reuses those tensors instead of drawing new
    ones (two batch sizes of one model share its parameters); x and the logits are drawn as usual."""
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
    if weights is not None:
        w13, w2 = weights
        assert tuple(w13.shape) == (n_experts, 2 * I, H) and tuple(w2.shape) == (n_experts, H, I)
    else:
        w13 = _normal_bf16((n_experts, 2 * I, H), 1.0 / math.sqrt(H), gen, device)
        w2 = _normal_bf16((n_experts, H, I), 1.0 / math.sqrt(I), gen, device)
    return dict(x=x, router_logits=logits.contiguous(), w13=w13, w2=w2, T=T, H=H, I=I, E=E, top_k=cfg["top_k"],
                local_offset=cfg.get("local_offset", 0), local=n_experts)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The uint16 bit pattern of a bf16 tensor, on the host, as a numpy array."""
    assert t.dtype == torch.bfloat16
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# ---- second workload: one decode step of grouped-query attention over a paged key-value cache -----------------
# (paper, Table 2 and Sec. 4.6: "GQA Paged Decode", model context Qwen3-30B-A3B: 32 query heads, 4 key-value heads,
# head dimension 128.)  Seeded stand-ins for the serving traces the paper measured on: a batch of sequences whose
# cached lengths are drawn uniformly from [len_lo, len_hi], their pages scattered over the physical cache by a random
# permutation, queries and cache contents N(0,1) rounded to bf16.
GQA_CONFIGS = {
    # name: batch, query heads, kv heads, head dim, page size, cached-length range
    "gqa_tiny": dict(B=3, Hq=8, Hkv=2, D=128, page_size=4, len_lo=1, len_hi=70),
    "gqa_decode_b64": dict(B=64, Hq=32, Hkv=4, D=128, page_size=16, len_lo=1024, len_hi=8192),
    "gqa_decode_b1_long": dict(B=1, Hq=32, Hkv=4, D=128, page_size=16, len_lo=65536, len_hi=65536),
    "gqa_decode_b256": dict(B=256, Hq=32, Hkv=4, D=128, page_size=16, len_lo=256, len_hi=2048),
    # long enough that launch, pipeline fill and the merge are small beside the stream: the kernel's steady state
    "gqa_decode_b64_16k": dict(B=64, Hq=32, Hkv=4, D=128, page_size=16, len_lo=16384, len_hi=16384),
}


def make_gqa_inputs(cfg, seed: int = 0, device="cpu", spare_pages: int = 7) -> dict:
    """Draw one paged-decode workload.  ``cfg`` is a name in GQA_CONFIGS or a dict with the same keys (an explicit
    ``lengths`` list overrides the drawn lengths).  Returns q [B,Hq,D] bf16, k_cache / v_cache [num_pages,P,Hkv,D]
    bf16, kv_indptr [B+1] / kv_indices / kv_last_page_len [B] int32 (all on ``device``), kv_len (a host list) and
    sm_scale = D ** -0.5."""
    if isinstance(cfg, str):
        cfg = GQA_CONFIGS[cfg]
    B, Hq, Hkv, D, P = cfg["B"], cfg["Hq"], cfg["Hkv"], cfg["D"], cfg["page_size"]
    device = torch.device(device)
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    if "lengths" in cfg:
        lengths = [int(v) for v in cfg["lengths"]]
    else:
        lengths = torch.randint(cfg["len_lo"], cfg["len_hi"] + 1, (B,), generator=gen).tolist()
    pages = [(n + P - 1) // P for n in lengths]
    num_pages = sum(pages) + spare_pages
    perm = torch.randperm(num_pages, generator=gen)[:sum(pages)].to(torch.int32)
    indptr = torch.zeros(B + 1, dtype=torch.int32)
    indptr[1:] = torch.cumsum(torch.tensor(pages, dtype=torch.int64), 0).to(torch.int32)
    last = torch.tensor([(n - 1) % P + 1 if n > 0 else 0 for n in lengths], dtype=torch.int32)
    dgen = torch.Generator(device=device)
    dgen.manual_seed(seed + 1)
    q = _normal_bf16((B, Hq, D), 1.0, dgen, device)
    k_cache = _normal_bf16((num_pages, P, Hkv, D), 1.0, dgen, device)
    v_cache = _normal_bf16((num_pages, P, Hkv, D), 1.0, dgen, device)
    return dict(q=q, k_cache=k_cache, v_cache=v_cache, kv_indptr=indptr.to(device), kv_indices=perm.to(device),
                kv_last_page_len=last.to(device), kv_len=lengths, sm_scale=float(D) ** -0.5, B=B, Hq=Hq, Hkv=Hkv, D=D,
                page_size=P, num_pages=num_pages)
