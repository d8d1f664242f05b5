"""GPU test of moe_route_static, the router + sort-scatter entry point that allocates nothing.

Some callers cannot call cudaMalloc and have no workspace to lend: code running inside a serving loop
whose memory plan is frozen, or a plugin that is handed tensors but no allocator.  For them the
library keeps the router's scratch in a fixed 512 KiB device array of its own.  This file checks that
the entry point, called through the C ABI, returns exactly what moe_route returns with a caller
workspace, on two calls in a row that share (and therefore reuse) that array -- the second with a
different shape, so anything left over from the first would show -- that both agree with the CPU oracle,
that the device's free memory does not move across the calls, and that problems beyond the array's size
are refused.  The file name sorts after the other test files on purpose: pytest collects it last, so a run
that stops at the first failure (-x) has already run every parity test of the method before it reaches
this packaging variant; it passes alone in a fresh process as well as after the others.
"""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
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
    # One call first, so that what a first call may set up (the lazily loaded kernels, the address look-up of
    # the array) is done; then the driver's own count of free device memory must not move across further
    # calls.  cudaMemGetInfo sees every allocation on the device, whoever made it; torch's counter, which
    # only sees torch's allocator, is kept as a second check.
    moe.moe_route_static(logits, k, got["ids"], got["w"], got["off"], got["s2f"], got["f2s"])
    torch.cuda.synchronize()
    for name, fill in (("ids", -7), ("off", -7), ("s2f", -7), ("f2s", -7)):
        got[name].fill_(fill)
    got["w"].fill_(float("nan"))
    torch.cuda.synchronize()
    free_before, torch_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    for _ in range(3):
        moe.moe_route_static(logits, k, got["ids"], got["w"], got["off"], got["s2f"], got["f2s"])
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "free device memory changed across moe_route_static calls"
    assert torch.cuda.memory_allocated() == torch_before
    for name in ("ids", "off", "s2f", "f2s"):
        assert torch.equal(got[name], ref[name]), name
    np.testing.assert_allclose(got["w"].cpu().numpy(), ref["w"].cpu().numpy(), rtol=0, atol=WEIGHT_TOL)
    assert int(got["off"][-1]) == T * k
    # and against the CPU oracle directly, so that this entry point's parity does not lean on moe_route's
    o = moe_oracle.get("f32")
    ids, w = o.route(logits.cpu().numpy(), k)
    off, s2f, f2s = o.permute(ids, E)
    assert np.array_equal(got["ids"].cpu().numpy(), ids) and np.array_equal(got["off"].cpu().numpy(), off)
    assert np.array_equal(got["s2f"].cpu().numpy(), s2f) and np.array_equal(got["f2s"].cpu().numpy(), f2s)
    np.testing.assert_allclose(got["w"].cpu().numpy(), w, rtol=0, atol=WEIGHT_TOL)


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
    # an array that is not 4-byte aligned is refused on the host (-4) and nothing is launched
    import ctypes
    raw = [ctypes.c_void_p(t.data_ptr()) for t in (small, o["ids"], o["w"], o["off"], o["s2f"], o["f2s"])]
    raw[1] = ctypes.c_void_p(o["ids"].data_ptr() + 2)
    st = moe.lib().moe_route_static(raw[0], 4, 8, 2, *raw[1:], ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
    assert st == -4
    torch.cuda.synchronize()
    assert (o["off"] == -7).all() and (o["ids"] == -7).all()
