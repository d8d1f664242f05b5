"""The layer captured into a CUDA graph: the library never synchronises, allocates or reads device memory on the
host, so its launch sequence can be recorded once and replayed; a replay on new inputs must equal a plain call."""
import pytest
import torch

import paper_2602_19128_b200 as moe
from paper_2602_19128_b200.inputs import make_inputs
from tests.weight_quantizers import make_mxfp8_inputs

pytestmark = pytest.mark.gpu


def _capture(call):
    """Runs `call(stream)` once eagerly on a side stream, then records it into a graph on that stream."""
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        call(s)
        s.synchronize()
        with torch.cuda.graph(g, stream=s):
            call(torch.cuda.current_stream())
    torch.cuda.synchronize()
    return g


@pytest.mark.parametrize("cfg", [dict(T=16, H=256, I=512, E=8, top_k=2, skew=False),
                                 dict(T=1500, H=256, I=128, E=32, top_k=4, skew=True)])  # fused and three-kernel router
def test_bf16_layer_replays_from_a_graph(cfg):
    a, b = make_inputs(cfg, seed=1, device="cuda"), make_inputs(cfg, seed=2, device="cuda")
    T, H, I, E, k = cfg["T"], cfg["H"], cfg["I"], cfg["E"], cfg["top_k"]
    x, logits = a["x"].clone(), a["router_logits"].clone()
    out = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), "cuda")
    g = _capture(lambda s: moe.moe_forward(x, logits, a["w13"], a["w2"], k, out, ws, stream=s))
    for inp in (b, a):  # the graph reads whatever the captured buffers hold at replay time
        x.copy_(inp["x"])
        logits.copy_(inp["router_logits"])
        g.replay()
        torch.cuda.synchronize()
        assert moe.moe_last_status(ws) == moe.MOE_OK
        ref = torch.empty_like(out)
        ws2 = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), "cuda")
        moe.moe_forward(inp["x"], inp["router_logits"], a["w13"], a["w2"], k, ref, ws2)
        torch.cuda.synchronize()
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_mxfp8_layer_replays_from_a_graph():
    cfg = dict(T=300, H=256, I=256, E=16, top_k=4, skew=True)
    a, b = make_mxfp8_inputs(cfg, seed=1, device="cuda"), make_inputs(cfg, seed=2, device="cuda")
    T, H, I, E, k = cfg["T"], cfg["H"], cfg["I"], cfg["E"], cfg["top_k"]
    sf13, sf2 = moe.moe_mxfp8_pack_scales(a["w13_s"], True), moe.moe_mxfp8_pack_scales(a["w2_s"], False)
    x, logits = a["x"].clone(), a["router_logits"].clone()
    out = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
    ws = moe.alloc_workspace(moe.moe_mxfp8_workspace_bytes(T, H, I, E, k), "cuda")
    g = _capture(lambda s: moe.moe_forward_mxfp8(x, logits, a["w13_q"], sf13, a["w2_q"], sf2, k, out, ws, stream=s))
    x.copy_(b["x"])
    logits.copy_(b["router_logits"])
    g.replay()
    torch.cuda.synchronize()
    assert moe.moe_last_status(ws) == moe.MOE_OK
    ref = torch.empty_like(out)
    ws2 = moe.alloc_workspace(moe.moe_mxfp8_workspace_bytes(T, H, I, E, k), "cuda")
    moe.moe_forward_mxfp8(b["x"], b["router_logits"], a["w13_q"], sf13, a["w2_q"], sf2, k, ref, ws2)
    torch.cuda.synchronize()
    assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_two_streams_with_their_own_workspaces_do_not_interfere():
    """The library keeps no state between calls except what lives in the caller's workspace, so calls on different
    streams with different workspaces may run concurrently."""
    cfg = dict(T=700, H=256, I=256, E=16, top_k=4, skew=True)
    a, b = make_inputs(cfg, seed=11, device="cuda"), make_inputs(cfg, seed=12, device="cuda")
    T, H, I, E, k = cfg["T"], cfg["H"], cfg["I"], cfg["E"], cfg["top_k"]
    refs = []
    for inp in (a, b):
        ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), "cuda")
        ref = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
        moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], k, ref, ws)
        torch.cuda.synchronize()
        refs.append(ref)
    lanes = []
    for inp in (a, b):
        lanes.append((torch.cuda.Stream(), inp, moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), "cuda"),
                      torch.empty((T, H), dtype=torch.bfloat16, device="cuda")))
    torch.cuda.synchronize()
    for _ in range(20):  # interleave the two lanes' launches
        for st, inp, ws, out in lanes:
            moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], k, out, ws, stream=st)
    torch.cuda.synchronize()
    for (st, inp, ws, out), ref in zip(lanes, refs):
        assert moe.moe_last_status(ws, stream=st) == moe.MOE_OK
        assert torch.equal(out.view(torch.int16), ref.view(torch.int16))


def test_alternating_problems_on_one_workspace_stay_bit_identical():
    """The hand-over between the two GEMMs lives in the workspace's status region and is reset by every call:
    back-to-back calls of different problems on the same workspace must not see each other's counters."""
    cfgs = [dict(T=600, H=256, I=256, E=8, top_k=2, skew=False), dict(T=90, H=256, I=128, E=64, top_k=6, skew=True),
            dict(T=1300, H=128, I=64, E=16, top_k=4, skew=False)]
    inps = [make_inputs(c, seed=30 + i, device="cuda") for i, c in enumerate(cfgs)]
    need = max(moe.moe_workspace_bytes(c["T"], c["H"], c["I"], c["E"], c["top_k"]) for c in cfgs)
    ws = moe.alloc_workspace(need, "cuda")
    ws.fill_(0xFF)
    outs = [torch.empty((c["T"], c["H"]), dtype=torch.bfloat16, device="cuda") for c in cfgs]
    refs = None
    for it in range(40):
        for inp, c, out in zip(inps, cfgs, outs):
            moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], c["top_k"], out, ws)
        if it == 0:
            torch.cuda.synchronize()
            assert moe.moe_last_status(ws) == moe.MOE_OK
            refs = []
            for inp, c in zip(inps, cfgs):  # the reference: each problem alone, on a fresh workspace
                w2 = moe.alloc_workspace(need, "cuda")
                r = torch.empty((c["T"], c["H"]), dtype=torch.bfloat16, device="cuda")
                moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], c["top_k"], r, w2)
                torch.cuda.synchronize()
                refs.append(r)
            for out, r in zip(outs, refs):
                assert torch.equal(out.view(torch.int16), r.view(torch.int16))
    torch.cuda.synchronize()
    assert moe.moe_last_status(ws) == moe.MOE_OK
    for out, r in zip(outs, refs):
        assert torch.equal(out.view(torch.int16), r.view(torch.int16))


def test_an_expired_device_wait_is_reported_and_leaves_the_device_usable():
    """Every device-side wait is bounded.  The self-test kernel waits about 0.1 s for a flag nothing raises: it must
    return with MOE_ERR_DEVICE_TIMEOUT in the status word, and the next call on the same workspace must work."""
    cfg = dict(T=64, H=256, I=128, E=8, top_k=2, skew=False)
    inp = make_inputs(cfg, seed=40, device="cuda")
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(64, 256, 128, 8, 2), "cuda")
    moe.moe_selftest_wait_timeout(ws)
    assert moe.moe_last_status(ws) == -7
    views = moe.workspace_views(ws, 64, 256, 128, 8, 2)
    assert views["status"][1].item() == 11          # the site recorded next to the status
    out = torch.empty((64, 256), dtype=torch.bfloat16, device="cuda")
    moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], 2, out, ws)
    assert moe.moe_last_status(ws) == moe.MOE_OK
    assert torch.isfinite(out.float()).all()


_FRESH = r"""
import sys, torch
sys.path.insert(0, {root!r})
import paper_2602_19128_b200 as moe
from paper_2602_19128_b200.inputs import make_inputs
cfg = dict(T={T}, H={H}, I={I}, E={E}, top_k={k}, skew=False)
inp = make_inputs(cfg, seed={seed}, device="cuda")
out = torch.empty(({T}, {H}), dtype=torch.bfloat16, device="cuda")
ws = moe.alloc_workspace(moe.moe_workspace_bytes({T}, {H}, {I}, {E}, {k}), "cuda")
moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], {k}, out, ws)
assert moe.moe_last_status(ws) == 0
torch.save(out.cpu(), {path!r})
"""


def test_tensor_map_cache_alternating_weight_sets_and_shapes_match_fresh_processes(tmp_path):
    """The library caches encoded tensor maps keyed by every argument of the encoding.  One process alternates two
    weight sets and two shapes, frees a weight set and allocates another where it was, and every result must be
    bit-identical to the result of a process that has never run anything else (so no entry can be stale)."""
    import subprocess
    import sys
    from pathlib import Path
    root = str(Path(__file__).resolve().parent.parent)
    cases = [(dict(T=300, H=256, I=256, E=8, top_k=2, skew=False), 51), (dict(T=300, H=256, I=256, E=8, top_k=2, skew=False), 52),
             (dict(T=700, H=128, I=192, E=4, top_k=2, skew=False), 53)]
    fresh = []
    for i, (c, seed) in enumerate(cases):
        path = str(tmp_path / f"fresh{i}.pt")
        src = _FRESH.format(root=root, T=c["T"], H=c["H"], I=c["I"], E=c["E"], k=c["top_k"], seed=seed, path=path)
        r = subprocess.run([sys.executable, "-c", src], capture_output=True, text=True, timeout=600)
        assert r.returncode == 0, r.stderr
        fresh.append(torch.load(path).cuda())
    inps = [make_inputs(c, seed=s, device="cuda") for c, s in cases]
    wss = [moe.alloc_workspace(moe.moe_workspace_bytes(c["T"], c["H"], c["I"], c["E"], c["top_k"]), "cuda") for c, _ in cases]
    for it in range(6):
        for i in (0, 1, 2, 1, 0):
            c = cases[i][0]
            out = torch.empty((c["T"], c["H"]), dtype=torch.bfloat16, device="cuda")
            moe.moe_forward(inps[i]["x"], inps[i]["router_logits"], inps[i]["w13"], inps[i]["w2"], c["top_k"], out, wss[i])
            torch.cuda.synchronize()
            assert torch.equal(out.view(torch.int16), fresh[i].view(torch.int16)), (it, i)
        if it == 2:  # drop weight set 0 and draw it again: torch's allocator hands back the same addresses
            ptr = inps[0]["w13"].data_ptr()
            inps[0] = None
            inps[0] = make_inputs(cases[0][0], seed=cases[0][1], device="cuda")
            assert isinstance(ptr, int)


def test_two_host_threads_calling_concurrently_with_their_own_workspaces():
    """The tensor-map cache is the library's only shared mutable state; it is guarded by a mutex, so two host threads
    may call at the same time (each on its own stream, with its own workspace)."""
    import threading
    cfgs = [dict(T=500, H=256, I=256, E=16, top_k=4, skew=True), dict(T=200, H=384, I=128, E=8, top_k=2, skew=False)]
    inps = [make_inputs(c, seed=60 + i, device="cuda") for i, c in enumerate(cfgs)]
    refs = []
    for inp, c in zip(inps, cfgs):
        ws = moe.alloc_workspace(moe.moe_workspace_bytes(c["T"], c["H"], c["I"], c["E"], c["top_k"]), "cuda")
        r = torch.empty((c["T"], c["H"]), dtype=torch.bfloat16, device="cuda")
        moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], c["top_k"], r, ws)
        torch.cuda.synchronize()
        refs.append(r)
    errors, outs = [], [None, None]

    def worker(i):
        try:
            torch.cuda.set_device(0)
            c, inp = cfgs[i], inps[i]
            st = torch.cuda.Stream()
            ws = moe.alloc_workspace(moe.moe_workspace_bytes(c["T"], c["H"], c["I"], c["E"], c["top_k"]), "cuda")
            out = torch.empty((c["T"], c["H"]), dtype=torch.bfloat16, device="cuda")
            for _ in range(200):
                moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], c["top_k"], out, ws, stream=st)
            st.synchronize()
            assert moe.moe_last_status(ws, stream=st) == moe.MOE_OK
            outs[i] = out
        except Exception as exc:  # surfaced in the main thread
            errors.append(exc)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for out, r in zip(outs, refs):
        assert torch.equal(out.view(torch.int16), r.view(torch.int16))


_OVERLAP = r"""
import sys, torch
sys.path.insert(0, {root!r})
import paper_2602_19128_b200 as moe
from paper_2602_19128_b200.inputs import make_inputs
cfg = dict(T={T}, H={H}, I={I}, E={E}, top_k={k}, skew=False)
inp = make_inputs(cfg, seed=70, device="cuda")
ws = [moe.alloc_workspace(moe.moe_workspace_bytes({T}, {H}, {I}, {E}, {k}), "cuda") for _ in range(2)]
outs = [torch.empty(({T}, {H}), dtype=torch.bfloat16, device="cuda") for _ in range(3)]
moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], {k}, outs[2], ws[0])
torch.cuda.synchronize()
streams = [torch.cuda.Stream(), torch.cuda.Stream()]
for it in range({groups}):
    for i in range(20):   # deep queues on both streams: the calls' kernels overlap in every phase combination
        moe.moe_forward(inp["x"], inp["router_logits"], inp["w13"], inp["w2"], {k}, outs[i % 2], ws[i % 2], stream=streams[i % 2])
    torch.cuda.synchronize()
for i in range(2):
    assert moe.moe_last_status(ws[i], stream=streams[i]) == 0
    assert torch.equal(outs[i].view(torch.int16), outs[2].view(torch.int16))
print("overlap ok")
"""


@pytest.mark.parametrize("T,H,I,E,k", [(2048, 512, 256, 256, 8),    # 128-row CTA-pair kernel, three-kernel router
                                       (2048, 512, 256, 64, 8)])    # wide-tile kernel, three-kernel router
def test_many_overlapping_calls_on_two_streams_complete(T, H, I, E, k):
    """Thousands of calls queued twenty deep on two streams, so that every kernel of one call meets every kernel of
    the other on the SMs.  CTA-pair kernels take a whole SM's shared memory for themselves; before they did, small
    blocks of the other stream's sort-scatter shared their SMs and, about once per thousand calls, a later pair waited
    for tensor memory for ever.  Run in a child process with a time limit so that a regression ends as a failure."""
    import subprocess
    import sys
    from pathlib import Path
    src = _OVERLAP.format(root=str(Path(__file__).resolve().parent.parent), T=T, H=H, I=I, E=E, k=k, groups=150)
    r = subprocess.run([sys.executable, "-c", src], capture_output=True, text=True, timeout=240)
    assert r.returncode == 0 and "overlap ok" in r.stdout, r.stderr[-2000:]


_OVERLAP_MX = r"""
import sys, torch
sys.path.insert(0, {root!r})
import paper_2602_19128_b200 as moe
from tests.weight_quantizers import make_mxfp8_inputs
cfg = dict(T={T}, H={H}, I={I}, E={E}, top_k={k}, skew=False)
inp = make_mxfp8_inputs(cfg, seed=71, device="cuda")
sf13, sf2 = moe.moe_mxfp8_pack_scales(inp["w13_s"], True), moe.moe_mxfp8_pack_scales(inp["w2_s"], False)
ws = [moe.alloc_workspace(moe.moe_mxfp8_workspace_bytes({T}, {H}, {I}, {E}, {k}), "cuda") for _ in range(2)]
outs = [torch.empty(({T}, {H}), dtype=torch.bfloat16, device="cuda") for _ in range(3)]
def call(o, w, stream=None):
    moe.moe_forward_mxfp8(inp["x"], inp["router_logits"], inp["w13_q"], sf13, inp["w2_q"], sf2, {k}, o, w, stream=stream)
call(outs[2], ws[0])
torch.cuda.synchronize()
streams = [torch.cuda.Stream(), torch.cuda.Stream()]
for it in range({groups}):
    for i in range(20):
        call(outs[i % 2], ws[i % 2], streams[i % 2])
    torch.cuda.synchronize()
for i in range(2):
    assert moe.moe_last_status(ws[i], stream=streams[i]) == 0
    assert torch.equal(outs[i].view(torch.int16), outs[2].view(torch.int16))
print("overlap ok")
"""


def test_many_overlapping_mxfp8_calls_on_two_streams_complete():
    """The same stress for the MX FP8 layer on its wide-tile kernel (304-row bound), which also takes a whole SM's
    shared memory: a child process with a time limit."""
    import subprocess
    import sys
    from pathlib import Path
    T, H, I, E, k = 2048, 512, 256, 64, 8
    assert moe.moe_mxfp8_workspace_layout(T, H, I, E, k).tile_rows == 304
    src = _OVERLAP_MX.format(root=str(Path(__file__).resolve().parent.parent), T=T, H=H, I=I, E=E, k=k, groups=100)
    r = subprocess.run([sys.executable, "-c", src], capture_output=True, text=True, timeout=240)
    assert r.returncode == 0 and "overlap ok" in r.stdout, r.stderr[-2000:]
