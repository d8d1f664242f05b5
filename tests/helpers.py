"""Shared test helpers: fixture parsing, bf16 helpers, and an independent float64 brute force."""
from __future__ import annotations

import os

import numpy as np
import torch

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name: str) -> dict:
    cases, cur = {}, None
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("case "):
                cur = cases.setdefault(line.split()[1], {})
                continue
            key, vals = line.split(":", 1)
            cur[key.strip()] = [float(v) for v in vals.split()]
    return cases


def f32_to_bf16_bits(a) -> np.ndarray:
    """Round float values to bf16 (nearest even, via torch) and return the uint16 bit patterns."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bruteforce_dense_moe(x_bits, logits, w13_bits, w2_bits, top_k: int) -> np.ndarray:
    """Float64 evaluation that shares nothing with the oracle's structure: EVERY expert is applied
    to EVERY token with dense matrix products, and the result is contracted with a dense [T,E]
    matrix of routing weights that is zero outside the top-k.  Selection uses a stable argsort of
    the negated logits (ties -> lower index), weights are softmax over the selected logits."""
    x = bits_to_f64(x_bits)
    w13 = bits_to_f64(w13_bits)
    w2 = bits_to_f64(w2_bits)
    l = np.asarray(logits, dtype=np.float32)
    T, E = l.shape
    I = w13.shape[1] // 2
    order = np.argsort(-l.astype(np.float64), axis=1, kind="stable")[:, :top_k]
    sel = np.take_along_axis(l.astype(np.float64), order, axis=1)
    z = np.exp(sel - sel.max(axis=1, keepdims=True))
    wsel = z / z.sum(axis=1, keepdims=True)
    dense_w = np.zeros((T, E))
    np.put_along_axis(dense_w, order, wsel, axis=1)
    out = np.zeros_like(x)
    for e in range(E):
        g = x @ w13[e, :I].T
        u = x @ w13[e, I:].T
        s = g / (1.0 + np.exp(-g)) * u
        out += dense_w[:, e:e + 1] * (s @ w2[e].T)
    return out


def small_case(T, H, I, E, k, seed=0, skew=False):
    from paper_2602_19128_b200.inputs import bf16_bits, make_inputs
    inp = make_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=skew), seed=seed, device="cpu")
    return dict(x=bf16_bits(inp["x"]), logits=inp["router_logits"].numpy(), w13=bf16_bits(inp["w13"]),
                w2=bf16_bits(inp["w2"]), k=k, T=T, H=H, I=I, E=E)
