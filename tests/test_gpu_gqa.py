"""GPU parity of the second workload, paged grouped-query decode attention (include/gqa_decode.h), against the
double-precision CPU oracle, element by element, through the C ABI.

Tolerance: |gpu - oracle| <= 1e-2 * (1 + |oracle|) for every output element and 2e-3 for lse.  The kernel rounds the
probabilities to bf16 for the P V product (relative 2^-9 each, averaging out over the tokens) and the result to bf16
(relative 2^-9); scores and sums are fp32.  Outputs are O(1), so the bound is several times the expected error."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import gqa_oracle
from paper_2602_19128_b200.inputs import GQA_CONFIGS, bf16_bits, make_gqa_inputs
from tests.gpu_common import Guarded

pytestmark = pytest.mark.gpu

OUT_TOL, LSE_TOL = 1e-2, 2e-3


def run_gpu(inp, max_kv_len=None, want_lse=True):
    B, Hq, Hkv, D = inp["B"], inp["Hq"], inp["Hkv"], inp["D"]
    max_kv_len = max(inp["kv_len"] + [0]) if max_kv_len is None else max_kv_len
    wg = Guarded(moe.gqa_decode_workspace_bytes(B, Hq, Hkv, D, max_kv_len), "cuda")
    og = Guarded(B * Hq * D * 2, "cuda")
    out = og.inner[:B * Hq * D * 2].view(torch.bfloat16).view(B, Hq, D)
    lg = Guarded(B * Hq * 4, "cuda")
    lse = lg.inner[:B * Hq * 4].view(torch.float32).view(B, Hq) if want_lse else None
    moe.gqa_paged_decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["kv_indptr"], inp["kv_indices"],
                         inp["kv_last_page_len"], max_kv_len, inp["sm_scale"], out, wg.inner, lse=lse)
    torch.cuda.synchronize()
    for g, name in ((wg, "workspace"), (og, "out"), (lg, "lse")):
        g.assert_bands_intact(f"gqa_paged_decode {name}")
    return out, lse


def oracle(inp):
    return gqa_oracle.get("f64").paged_decode(bf16_bits(inp["q"]), bf16_bits(inp["k_cache"]), bf16_bits(inp["v_cache"]),
                                              inp["kv_indptr"].cpu().numpy(), inp["kv_indices"].cpu().numpy(),
                                              inp["kv_last_page_len"].cpu().numpy(), inp["sm_scale"])


def check(inp, max_kv_len=None):
    out, lse = run_gpu(inp, max_kv_len)
    ref, ref_lse = oracle(inp)
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    err, bound = np.abs(got - ref), OUT_TOL * (1 + np.abs(ref))
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    assert (err <= bound).all(), f"out worst at {worst}: gpu={got[worst]} ref={ref[worst]}"
    got_lse = lse.cpu().numpy().astype(np.float64)
    empty = np.isneginf(ref_lse)
    assert np.array_equal(np.isneginf(got_lse), empty)
    assert np.abs(got_lse[~empty] - ref_lse[~empty]).max(initial=0) <= LSE_TOL
    return out


# B, Hq, Hkv, page size, lengths: chunk and split edges, ragged last pages, empty items, every group size
CASES = [
    (3, 8, 2, 4, [5, 60, 64]),
    (4, 32, 4, 16, [1, 63, 65, 129]),                 # the paper's head geometry; 64-token chunk edges
    (2, 4, 4, 1, [17, 300]),                          # one token per page; groups of one head
    (3, 16, 1, 8, [0, 5, 700]),                       # an item with nothing cached; a group of 16 heads
    (2, 6, 2, 16, [1024, 2047]),                      # groups of three; several splits per sequence
    (1, 32, 4, 16, [20000]),                          # one long sequence: many splits merged by the last block
    (5, 32, 4, 32, [16, 32, 33, 4096, 257]),          # mixed lengths: some sequences use one split, some many
    (40, 8, 4, 16, [100 + 37 * i for i in range(40)]),  # enough items that every sequence is a single split
    (2, 2, 1, 64, [64, 6000]),                        # groups of two, large pages
    (3, 32, 4, 8, [7, 1000, 5000]),                   # the smallest page the tiled gather takes: 32 boxes per chunk
    (2, 32, 4, 128, [100, 7000]),                     # pages larger than a chunk: boxes start inside a page
    (2, 8, 1, 256, [255, 9000]),
    (3, 32, 4, 12, [11, 1000, 5000]),                 # page sizes that are no power of two: the row gather
    (2, 16, 2, 3, [2, 4100]),
    (2, 32, 4, 24, [24, 6001]),
    (2, 32, 4, 2, [3000, 1]),
]


@pytest.mark.parametrize("B,Hq,Hkv,P,lengths", CASES, ids=[f"B{c[0]}h{c[1]}kv{c[2]}p{c[3]}" for c in CASES])
def test_decode_matches_oracle(B, Hq, Hkv, P, lengths):
    inp = make_gqa_inputs(dict(B=B, Hq=Hq, Hkv=Hkv, D=128, page_size=P, lengths=lengths), seed=B + Hq, device="cuda")
    check(inp)


@pytest.mark.parametrize("P", [16, 12, 64, 128])
def test_slots_past_the_end_of_a_sequence_are_never_used(P):
    """The cache behind the last token of a sequence, and every page no sequence owns, holds NaN: the tiled gather
    copies whole pages into shared memory and must still keep those values out of the result."""
    lengths = [1, P + 1, 5 * P - 1, 3000 + P // 2, 64 * 7 + 5]
    inp = make_gqa_inputs(dict(B=len(lengths), Hq=32, Hkv=4, D=128, page_size=P, lengths=lengths), seed=P, device="cuda")
    owned = torch.zeros((inp["num_pages"], P), dtype=torch.bool, device="cuda")
    indptr, indices = inp["kv_indptr"].tolist(), inp["kv_indices"]
    for b, n in enumerate(lengths):
        pages = indices[indptr[b]:indptr[b + 1]].long()
        flat = torch.zeros(len(pages) * P, dtype=torch.bool, device="cuda")
        flat[:n] = True
        owned[pages] = flat.view(len(pages), P)
    for cache in (inp["k_cache"], inp["v_cache"]):
        cache[~owned] = float("nan")
    check(inp)


def test_the_workspace_status_word_reports_success():
    inp = make_gqa_inputs(dict(B=2, Hq=32, Hkv=4, D=128, page_size=16, lengths=[5000, 300]), seed=3, device="cuda")
    ws = moe.alloc_workspace(moe.gqa_decode_workspace_bytes(2, 32, 4, 128, 5000), "cuda")
    ws.fill_(0x5A)
    out = torch.empty((2, 32, 128), dtype=torch.bfloat16, device="cuda")
    moe.gqa_paged_decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["kv_indptr"], inp["kv_indices"],
                         inp["kv_last_page_len"], 5000, inp["sm_scale"], out, ws)
    assert moe.moe_last_status(ws) == 0


def test_an_expired_barrier_wait_is_reported_and_leaves_the_device_usable():
    """Every wait of the kernel is bounded.  The self-test waits a few milliseconds on a barrier at which nothing
    arrives: it must come back with MOE_ERR_DEVICE_TIMEOUT in the status word, and the next call must work."""
    inp = make_gqa_inputs(dict(B=2, Hq=32, Hkv=4, D=128, page_size=16, lengths=[5000, 300]), seed=3, device="cuda")
    ws = moe.alloc_workspace(moe.gqa_decode_workspace_bytes(2, 32, 4, 128, 5000), "cuda")
    moe.gqa_selftest_wait_timeout(ws)
    assert moe.moe_last_status(ws) == -7
    assert ws[:12].view(torch.int32)[1].item() == 12          # the site recorded next to the status
    check(inp)
    out = torch.empty((2, 32, 128), dtype=torch.bfloat16, device="cuda")
    moe.gqa_paged_decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["kv_indptr"], inp["kv_indices"],
                         inp["kv_last_page_len"], 5000, inp["sm_scale"], out, ws)
    assert moe.moe_last_status(ws) == 0


def test_a_sequence_longer_than_the_hint_is_still_computed_in_full():
    inp = make_gqa_inputs(dict(B=2, Hq=32, Hkv=4, D=128, page_size=16, lengths=[3000, 500]), seed=2, device="cuda")
    check(inp, max_kv_len=1024)     # the last split runs to the end of the sequence


def test_results_do_not_depend_on_which_block_finishes_last():
    inp = make_gqa_inputs(dict(B=3, Hq=32, Hkv=4, D=128, page_size=16, lengths=[9000, 4000, 12345]), seed=4, device="cuda")
    first, lse0 = run_gpu(inp)
    for _ in range(5):
        again, lse1 = run_gpu(inp)
        assert torch.equal(first.view(torch.int16), again.view(torch.int16)) and torch.equal(lse0, lse1)


def test_lse_is_optional_and_arguments_are_checked_before_any_launch():
    inp = make_gqa_inputs("gqa_tiny", seed=0, device="cuda")
    out, _ = run_gpu(inp, want_lse=False)
    ref, _ = oracle(inp)
    assert (np.abs(out.float().cpu().numpy() - ref) <= OUT_TOL * (1 + np.abs(ref))).all()
    B, Hq, Hkv, D = inp["B"], inp["Hq"], inp["Hkv"], inp["D"]
    ws = moe.alloc_workspace(moe.gqa_decode_workspace_bytes(B, Hq, Hkv, D, 70), "cuda")
    o = torch.zeros((B, Hq, D), dtype=torch.bfloat16, device="cuda")
    args = (inp["q"], inp["k_cache"], inp["v_cache"], inp["kv_indptr"], inp["kv_indices"], inp["kv_last_page_len"])
    assert moe.gqa_paged_decode(*args, 70, 0.1, o, ws[:256], check=False) == -5            # workspace too small
    assert moe.gqa_paged_decode(*args, 70, 0.1, o, ws[8:], check=False) == -4              # workspace misaligned
    bad_q = torch.zeros((B, 7, D), dtype=torch.bfloat16, device="cuda")                     # 7 heads over 2 kv heads
    assert moe.gqa_paged_decode(bad_q, *args[1:], 70, 0.1, o, ws, check=False) == -3
    assert moe.gqa_decode_workspace_bytes(B, Hq, Hkv, 64, 70) == 0                          # D must be 128
    torch.cuda.synchronize()
    assert (o == 0).all()


@pytest.mark.parametrize("name", ["gqa_decode_b64", "gqa_decode_b256", "gqa_decode_b1_long", "gqa_decode_b64_16k"])
def test_full_size_workload(name):
    """The benchmark's workloads in its launch configuration: every element against the oracle."""
    inp = make_gqa_inputs(GQA_CONFIGS[name], seed=0, device="cuda")
    out = check(inp)
    again, _ = run_gpu(inp)
    assert torch.equal(out.view(torch.int16), again.view(torch.int16))
