"""Seeded random shapes through the tensor-core path and through the CUDA-core validation GEMMs (which share no
code with it): routing identical, every element of h, y and out within the workload tolerance.  Shapes are drawn
across the token-tile bounds (32 / 64 / 128 / 256), both GEMM kernels (one CTA, CTA pairs) and both router
forms (fused up to 1024 tokens, three kernels beyond)."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from tests.gpu_common import OUT_TOL, gpu_inputs, run_forward

pytestmark = pytest.mark.gpu


def draw_shapes(n, seed):
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < n:
        E = int(rng.choice([1, 2, 3, 5, 8, 16, 24, 64, 128, 256]))
        k = int(rng.integers(1, min(E, 8) + 1))
        H = 128 * int(rng.integers(1, 5))
        I = 64 * int(rng.integers(1, 9))
        T = int(rng.choice([1, 2, 7, 31, 33, 100, 257, 600, 1025, 1500]))
        if T * k * (H + I) > 3_000_000:   # keep the validation GEMMs quick
            continue
        shapes.append((T, H, I, E, k, bool(rng.integers(0, 2))))
    return shapes


@pytest.mark.parametrize("T,H,I,E,k,skew", draw_shapes(36, seed=2024))
def test_random_shape_against_validation_gemms(T, H, I, E, k, skew):
    inp = gpu_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=skew), seed=T + E)
    out, views, _ = run_forward(inp)
    out_v, views_v, _ = run_forward(inp, flags=moe.MOE_FLAG_VALIDATION_GEMM)
    for name in ("topk_ids", "expert_offsets", "sorted_to_flat", "flat_to_sorted"):
        assert torch.equal(views[name], views_v[name]), name
    for name, a, b in (("h", views["h"], views_v["h"]), ("y", views["y"], views_v["y"]), ("out", out, out_v)):
        a, b = a.float(), b.float()
        assert torch.isfinite(a).all(), name
        bad = (a - b).abs() > OUT_TOL * (1 + b.abs())
        assert not bad.any(), f"{name}: {int(bad.sum())} elements beyond tolerance"
