"""GPU test of moe_route_static, the router + sort-scatter entry point that allocates nothing.

Some callers cannot call cudaMalloc and have no workspace to lend: code running inside a serving loop
whose memory plan is frozen, or a plugin that is handed tensors but no allocator.  For them the
library keeps the router's scratch in a fixed 512 KiB device array of its own.  This file checks that
the entry point, called through the C ABI, returns exactly what moe_route returns with a caller
workspace, on two calls in a row that share (and therefore reuse) that array -- the second with a
different shape, so anything left over from the first would show -- and that problems beyond the
array's size are refused.  It is collected last on purpose (the name sorts after the other tests).
"""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from tests.gpu_common import WEIGHT_TOL

pytestmark = pytest.mark.gpu


def outputs(T, E, k, dev):
    A = T * k
    return dict(ids=torch.full((T, k), -7, dtype=torch.int32, device=dev),
                w=torch.full((T, k), float("nan"), dtype=torch.float32, device=dev),
                off=torch.full((E + 1,), -7, dtype=torch.int32, device=dev),
                s2f=torch.full((A,), -7, dtype=torch.int32, device=dev),
                f2s=torch.full((A,), -7, dtype=torch.int32, device=dev))


def route_both_ways(logits, k):
    T, E = logits.shape
    dev = logits.device
    ref = outputs(T, E, k, dev)
    ws = moe.alloc_workspace(moe.moe_route_workspace_bytes(T, E, k), dev)
    moe.moe_route(logits, k, ref["ids"], ref["w"], ref["off"], ref["s2f"], ref["f2s"], ws)
    got = outputs(T, E, k, dev)  # allocated by the test, before the call: the call itself allocates nothing
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    moe.moe_route_static(logits, k, got["ids"], got["w"], got["off"], got["s2f"], got["f2s"])
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    for name in ("ids", "off", "s2f", "f2s"):
        assert torch.equal(got[name], ref[name]), name
    np.testing.assert_allclose(got["w"].cpu().numpy(), ref["w"].cpu().numpy(), rtol=0, atol=WEIGHT_TOL)
    assert int(got["off"][-1]) == T * k


def test_static_scratch_route_matches_workspace_route_on_two_calls_in_a_row():
    g = torch.Generator().manual_seed(11)
    first = torch.randn(2048, 256, generator=g).cuda()          # fills a large part of the static array
    route_both_ways(first, 8)
    second = (torch.randn(333, 40, generator=g) - 2.2 * torch.log(torch.arange(1, 41).float())).cuda()
    route_both_ways(second, 5)                                   # smaller, skewed: stale contents would show
    route_both_ways(first, 8)                                    # and back again


def test_static_scratch_limit_and_argument_errors():
    dev = "cuda"
    E, k = 256, 8
    T = 16256                                                    # the largest T that fits at E = 256
    logits = torch.randn(T, E, generator=torch.Generator().manual_seed(3)).cuda()
    route_both_ways(logits, k)
    too_big = torch.zeros(T + 32, E, device=dev)
    o = outputs(T + 32, E, k, dev)
    st = moe.moe_route_static(too_big, k, o["ids"], o["w"], o["off"], o["s2f"], o["f2s"], check=False)
    assert st == -9 and "512 KiB" in moe.moe_status_string(st)
    torch.cuda.synchronize()
    assert (o["off"] == -7).all()                                # nothing was launched
    small = torch.zeros(4, 8, device=dev)
    o = outputs(4, 8, 2, dev)
    assert moe.moe_route_static(small, 9, o["ids"], o["w"], o["off"], o["s2f"], o["f2s"], check=False) == -2
