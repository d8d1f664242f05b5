"""Pins of the paged grouped-query decode oracle (oracle/gqa_oracle.c) against what the definition and the
mathematics fix: hand-derived closed forms, a library routine (torch's scaled_dot_product_attention on the gathered
dense cache), a NumPy float64 evaluation written with matrix products, and invariants chosen so that a plausible
mistake -- a wrong page or slot index, a head mapped to the wrong key-value head, a dropped scale, a softmax over the
wrong axis, a last page read in full -- fails at least one of them."""
from pathlib import Path

import numpy as np
import pytest
import torch

from oracle import gqa_oracle
from paper_2602_19128_b200.inputs import bf16_bits, make_gqa_inputs
from tests.helpers import bits_to_f64, f32_to_bf16_bits

GOLDEN = {}
for line in (Path(__file__).parent / "golden" / "gqa_closed_forms.txt").read_text().splitlines():
    if line and not line.startswith("#"):
        name, *vals = line.split()
        GOLDEN[name] = np.array([float(v) for v in vals])


def bits(a):
    return f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def run(q, k, v, indptr, indices, last, scale, prec="f64"):
    return gqa_oracle.get(prec).paged_decode(bits(q), bits(k), bits(v), np.asarray(indptr, np.int32),
                                             np.asarray(indices, np.int32), np.asarray(last, np.int32), scale)


def test_one_token_gives_its_value_and_its_score():
    q = np.array([[[1, 2, 0, -1]]], np.float32)
    k = np.zeros((3, 2, 1, 4), np.float32); v = np.zeros((3, 2, 1, 4), np.float32)
    k[2, 0, 0] = [0.5, 0.25, 3, 1]; v[2, 0, 0] = [2, -4, 0.5, 8]
    k[2, 1, 0] = 9; v[2, 1, 0] = 9                      # the unused slot of the last page must not be read
    out, lse = run(q, k, v, [0, 1], [2], [1], 0.5)
    np.testing.assert_allclose(out[0, 0], GOLDEN["one_token_o"], atol=1e-12)
    np.testing.assert_allclose(lse[0, 0], GOLDEN["one_token_lse"], atol=1e-12)


def test_equal_scores_give_the_mean_of_the_values_across_pages():
    q = np.zeros((1, 1, 2), np.float32)
    k = np.ones((5, 2, 1, 2), np.float32); v = np.full((5, 2, 1, 2), 77, np.float32)
    pages = [3, 1]                                      # token t sits in page pages[t // 2], slot t % 2
    for t in range(4):
        v[pages[t // 2], t % 2, 0] = [t, 2 * t]
    out, lse = run(q, k, v, [0, 2], pages, [2], 1.0)
    np.testing.assert_allclose(out[0, 0], GOLDEN["equal_scores_o"], atol=1e-12)
    np.testing.assert_allclose(lse[0, 0], GOLDEN["equal_scores_lse"], atol=1e-12)


def test_two_tokens_with_a_known_score_gap():
    scale = float(np.log(3.0) / 2)
    q = np.array([[[2.0]]], np.float32)
    k = np.zeros((1, 2, 1, 1), np.float32); v = np.zeros((1, 2, 1, 1), np.float32)
    k[0, 0, 0, 0], k[0, 1, 0, 0] = 1, 0
    v[0, 0, 0, 0], v[0, 1, 0, 0] = 8, -4
    out, lse = run(q, k, v, [0, 1], [0], [2], scale)
    np.testing.assert_allclose(out[0, 0], GOLDEN["two_tokens_o"], atol=1e-12)
    np.testing.assert_allclose(lse[0, 0], GOLDEN["two_tokens_lse"], atol=1e-12)


def dense_kv(inp, b):
    """The cached keys and values of item b gathered into [L, Hkv, D] float64 (index bookkeeping only)."""
    P, L = inp["page_size"], inp["kv_len"][b]
    ip = inp["kv_indptr"].numpy(); idx = inp["kv_indices"].numpy()
    rows = [(int(idx[ip[b] + t // P]), t % P) for t in range(L)]
    k = bits_to_f64(bf16_bits(inp["k_cache"])); v = bits_to_f64(bf16_bits(inp["v_cache"]))
    pg = np.array([r[0] for r in rows], dtype=np.int64); sl = np.array([r[1] for r in rows], dtype=np.int64)
    return k[pg, sl], v[pg, sl]


CASES = [dict(B=3, Hq=8, Hkv=2, D=128, page_size=4, len_lo=1, len_hi=70),
         dict(B=4, Hq=6, Hkv=3, D=32, page_size=1, len_lo=1, len_hi=40),        # one token per page
         dict(B=2, Hq=4, Hkv=4, D=64, page_size=16, lengths=[16, 33]),          # a full last page; group of one
         dict(B=3, Hq=16, Hkv=1, D=16, page_size=8, lengths=[0, 5, 64])]        # an item with nothing cached


@pytest.mark.parametrize("cfg", CASES, ids=lambda c: f"B{c['B']}h{c['Hq']}kv{c['Hkv']}d{c['D']}p{c['page_size']}")
def test_against_torch_sdpa_and_numpy_matmul(cfg):
    inp = make_gqa_inputs(cfg, seed=3)
    out, lse = gqa_oracle.get("f64").paged_decode(bf16_bits(inp["q"]), bf16_bits(inp["k_cache"]), bf16_bits(inp["v_cache"]),
                                                  inp["kv_indptr"].numpy(), inp["kv_indices"].numpy(),
                                                  inp["kv_last_page_len"].numpy(), inp["sm_scale"])
    q = bits_to_f64(bf16_bits(inp["q"]))
    G = cfg["Hq"] // cfg["Hkv"]
    for b in range(cfg["B"]):
        if inp["kv_len"][b] == 0:
            assert np.all(out[b] == 0) and np.all(np.isneginf(lse[b]))
            continue
        k, v = dense_kv(inp, b)                                               # [L, Hkv, D]
        kk = np.repeat(k, G, axis=1).transpose(1, 0, 2); vv = np.repeat(v, G, axis=1).transpose(1, 0, 2)  # [Hq, L, D]
        # library routine
        ref = torch.nn.functional.scaled_dot_product_attention(torch.from_numpy(q[b])[:, None, :], torch.from_numpy(kk),
                                                               torch.from_numpy(vv), scale=inp["sm_scale"])[:, 0].numpy()
        np.testing.assert_allclose(out[b], ref, rtol=0, atol=1e-12)
        # the definition with matrix products
        s = inp["sm_scale"] * np.einsum("hd,hld->hl", q[b], kk)
        p = np.exp(s - s.max(axis=1, keepdims=True)); p /= p.sum(axis=1, keepdims=True)
        np.testing.assert_allclose(out[b], np.einsum("hl,hld->hd", p, vv), rtol=0, atol=1e-12)
        np.testing.assert_allclose(lse[b], np.log(np.exp(s - s.max(axis=1, keepdims=True)).sum(axis=1)) + s.max(axis=1),
                                   rtol=0, atol=1e-12)


def test_physical_page_order_does_not_matter():
    cfg = dict(B=3, Hq=8, Hkv=2, D=64, page_size=4, len_lo=5, len_hi=50)
    inp = make_gqa_inputs(cfg, seed=5)
    o = gqa_oracle.get("f64")
    args = lambda i: (bf16_bits(i["q"]), bf16_bits(i["k_cache"]), bf16_bits(i["v_cache"]), i["kv_indptr"].numpy(),
                      i["kv_indices"].numpy(), i["kv_last_page_len"].numpy(), i["sm_scale"])
    base, base_lse = o.paged_decode(*args(inp))
    perm = torch.randperm(inp["num_pages"], generator=torch.Generator().manual_seed(1))
    moved = dict(inp)
    inv = torch.empty_like(perm); inv[perm] = torch.arange(len(perm))
    moved["k_cache"] = inp["k_cache"][perm].contiguous(); moved["v_cache"] = inp["v_cache"][perm].contiguous()
    moved["kv_indices"] = inv[inp["kv_indices"].long()].to(torch.int32)      # old page i now lives at inv[i]
    again, again_lse = o.paged_decode(*args(moved))
    assert np.array_equal(base, again) and np.array_equal(base_lse, again_lse)


def test_heads_of_one_group_share_their_key_value_head():
    cfg = dict(B=2, Hq=8, Hkv=2, D=32, page_size=4, len_lo=9, len_hi=30)
    inp = make_gqa_inputs(cfg, seed=7)
    inp["q"][:, 1] = inp["q"][:, 0]; inp["q"][:, 4] = inp["q"][:, 0]        # head 1: same group as head 0; head 4: the other
    out, _ = gqa_oracle.get("f64").paged_decode(bf16_bits(inp["q"]), bf16_bits(inp["k_cache"]), bf16_bits(inp["v_cache"]),
                                                inp["kv_indptr"].numpy(), inp["kv_indices"].numpy(),
                                                inp["kv_last_page_len"].numpy(), inp["sm_scale"])
    assert np.array_equal(out[:, 0], out[:, 1]) and not np.allclose(out[:, 0], out[:, 4])


def test_float_build_is_close_to_the_double_build():
    inp = make_gqa_inputs("gqa_tiny", seed=0)
    a = [bf16_bits(inp["q"]), bf16_bits(inp["k_cache"]), bf16_bits(inp["v_cache"]), inp["kv_indptr"].numpy(),
         inp["kv_indices"].numpy(), inp["kv_last_page_len"].numpy(), inp["sm_scale"]]
    o64, l64 = gqa_oracle.get("f64").paged_decode(*a)
    o32, l32 = gqa_oracle.get("f32").paged_decode(*a)
    assert np.abs(o32 - o64).max() < 2e-5 and np.abs(l32 - l64).max() < 2e-5
