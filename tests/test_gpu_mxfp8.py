"""GPU parity of the MX FP8 path (E4M3 codes, E8M0 scale bytes, block-scaled tensor-core MMA) against the oracle:
the row quantiser and the scale repacking bit for bit, the quantised token rows bit for bit, the codes of h up to
the few decisions that sit on a rounding boundary, and the layer output within the workload's tolerance."""
import numpy as np
import pytest
import torch

import paper_2602_19128_b200 as moe
from oracle import moe_oracle
from paper_2602_19128_b200.inputs import bf16_bits
from tests.weight_quantizers import make_mxfp8_inputs
from tests.gpu_common import (Guarded, assert_close_out, assert_routing_exact, bf16_to_f64, check_guards, guarded_out,
                              mx_regions)

pytestmark = pytest.mark.gpu

TABLE = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).float().numpy().astype(np.float64)


def atom_byte(r, sf):
    return (r % 32) * 16 + (r // 32) * 4 + sf


def expert_tile_rows(count: int, tile: int) -> int:
    """Rows of every token tile of an expert with ``count`` rows (include/moe.h, the MX workspace layout): the bound
    itself up to 256; for the wide bounds one tile of round16(count) rows, or evenly sized tiles of at most 256."""
    if tile <= 256:
        return tile
    n = 1 if count <= tile else -(-count // 256)
    return (-(-count // n) + 15) // 16 * 16


def unpack_act_scales(atoms: np.ndarray, offsets: np.ndarray, n_blocks: int, tile: int) -> np.ndarray:
    """Scale atoms [K/128, n_atoms, 512] -> plain [rows, K/32] for the rows of every expert segment."""
    E = len(offsets) - 1
    rows = offsets[E]
    plain = np.zeros((rows, n_blocks), np.uint8)
    apt, stride = (tile + 127) // 128, min(tile, 256)
    for e in range(E):
        begin = offsets[e]
        count = offsets[e + 1] - begin
        per_tile = expert_tile_rows(int(count), tile) if count else tile
        for i in range(count):
            r = i % per_tile
            a = (begin // stride + e + i // per_tile) * apt + r // 128
            for b in range(n_blocks):
                plain[begin + i, b] = atoms[b // 4, a, atom_byte(r % 128, b % 4)]
    return plain


def run_mx(inp, local_offset=0):
    T, H = inp["x"].shape
    n_local, I2, _ = inp["w13_q"].shape
    E = inp["router_logits"].shape[1]
    I, k = I2 // 2, inp["top_k"]
    w13_sf = moe.moe_mxfp8_pack_scales(inp["w13_s"], gate_up=True)
    w2_sf = moe.moe_mxfp8_pack_scales(inp["w2_s"], gate_up=False)
    wg = Guarded(moe.moe_mxfp8_workspace_bytes(T, H, I, E, k), "cuda")
    ws = wg.inner
    og, out = guarded_out(T, H, "cuda")
    moe.moe_forward_mxfp8(inp["x"], inp["router_logits"], inp["w13_q"], w13_sf, inp["w2_q"], w2_sf, k, out, ws,
                          local_expert_offset=local_offset)
    status = moe.moe_last_status(ws)
    assert status == moe.MOE_OK, moe.moe_status_string(status)
    check_guards(wg, og, moe.moe_mxfp8_workspace_layout(T, H, I, E, k), mx_regions(T, H, I, E, k, n_local), "moe_forward_mxfp8")
    return out, moe.mx_workspace_views(ws, T, H, I, E, k)


def oracle_mx(inp, intermediates=False, prec="f32"):
    return moe_oracle.get(prec).forward_mxfp8(bf16_bits(inp["x"]), inp["router_logits"].cpu().numpy(),
                                             inp["w13_q"].cpu().numpy(), inp["w13_s"].cpu().numpy(),
                                             inp["w2_q"].cpu().numpy(), inp["w2_s"].cpu().numpy(), inp["top_k"],
                                             intermediates=intermediates)


@pytest.mark.parametrize("R,K,scale", [(1, 128, 1.0), (37, 384, 1.0), (300, 7168, 3.0), (64, 256, 1e-30), (9, 128, 1e30),
                                       (17, 128, 1e-38)])
def test_row_quantiser_is_bit_exact(R, K, scale):
    g = torch.Generator().manual_seed(R)
    x = (torch.randn((R, K), generator=g) * torch.exp2(torch.randint(-6, 6, (R, K // 32, 1), generator=g).float())
         .expand(R, K // 32, 32).reshape(R, K) * scale).to(torch.bfloat16)
    x[0, :32] = 0                                    # an all-zero block
    if R > 2:
        x[1, 5] = float("inf")                       # non-finite blocks
        x[2, 40] = float("nan")
        x[2, 100] = -0.0
    codes, scales = moe.moe_mxfp8_quantize_rows(x.cuda())
    torch.cuda.synchronize()
    want_c, want_s = moe_oracle.get("f32").mx_quantize(x.float().numpy())
    assert np.array_equal(scales.cpu().numpy(), want_s)
    assert np.array_equal(codes.cpu().numpy(), want_c)


@pytest.mark.parametrize("E,rows,K,gate_up", [(2, 256, 128, True), (3, 512, 384, True), (2, 128, 256, False), (4, 384, 512, False)])
def test_scale_repacking_is_the_documented_permutation(E, rows, K, gate_up):
    g = torch.Generator().manual_seed(0)
    plain = torch.randint(0, 255, (E, rows, K // 32), dtype=torch.uint8, generator=g)
    packed = moe.moe_mxfp8_pack_scales(plain.cuda(), gate_up=gate_up).cpu().numpy()
    p = plain.numpy()
    slots = K // 128
    tiles = rows // 128
    got = packed.reshape(E, tiles, slots, 512)
    I = rows // 2
    for e in range(E):
        for t in range(tiles):
            for m in range(128):
                if gate_up:
                    q, half, j = m // 32, (m // 16) % 2, m % 16
                    row = half * I + 64 * t + 16 * q + j
                else:
                    row = 128 * t + m
                for s in range(slots):
                    for sf in range(4):
                        assert got[e, t, s, atom_byte(m, sf)] == p[e, row, 4 * s + sf]


# T, H, I, E, k, skew: token-tile bounds 32 / 64 / 128, several tiles per expert
CASES = [
    (16, 256, 512, 8, 2, False),
    (1, 128, 128, 4, 1, False),
    (128, 384, 128, 256, 8, False),   # decode-like
    (200, 256, 384, 8, 2, False),     # ~50 rows per expert
    (300, 128, 128, 64, 4, True),     # skewed, empty experts, several tiles for the popular ones
    (700, 256, 256, 4, 2, False),     # ~350 rows per expert: one wide tile each (bound 384: two MMA parts, three atoms)
    (96, 128, 256, 8, 8, False),
    (513, 128, 128, 2, 1, False),     # ~256 rows per expert; H not a multiple of 256: one-CTA kernel, 128-row tiles
    (513, 256, 128, 2, 1, False),     # the same on CTA pairs: wide tiles, bound 320
    (1000, 512, 384, 4, 2, False),    # ~500 rows per expert: three pair tiles each, several feature tiles
    (130, 256, 256, 4, 2, False),     # 128-row pair tiles (one atom each)
    (300, 256, 128, 16, 4, True),     # the same, skewed: popular experts spill into a second tile
    (64, 128, 128, 64, 32, False),    # top_k = 32
    (2000, 128, 128, 1, 1, False),    # one expert, sixteen 128-row tiles: gate/up on pairs, down (H % 256 != 0) on one CTA
    (2000, 256, 128, 1, 1, False),    # one expert, nine 240-row tiles on pairs
    (33, 640, 384, 5, 3, False),      # H, I multiples of 128 only; E not a power of two
    (1200, 512, 384, 8, 2, False),    # ~300 rows per expert, bound 384: tiles of 257..384 rows, several feature tiles
    (1100, 256, 256, 8, 2, True),     # the same bound, skewed: popular experts take several 384-row tiles, others a few rows
    (2600, 256, 128, 16, 2, False),   # ~325 rows per expert: consecutive wide tiles overlap in the accumulator ring
    (1030, 256, 128, 8, 2, False),    # ~257 rows per expert, bound 320: tiles just above and below 256 rows
]


def draw_shapes(n, seed):
    """Seeded random shapes inside the MX envelope, small enough for the oracle."""
    rng = np.random.default_rng(seed)
    shapes = []
    while len(shapes) < n:
        E = int(rng.choice([1, 2, 3, 6, 8, 16, 32, 128]))
        k = int(rng.integers(1, min(E, 6) + 1))
        H, I = 128 * int(rng.integers(1, 5)), 128 * int(rng.integers(1, 4))
        T = int(rng.choice([1, 5, 32, 70, 150, 400, 1030]))
        if T * k * H * I > 120_000_000:
            continue
        shapes.append((T, H, I, E, k, bool(rng.integers(0, 2))))
    return shapes


@pytest.mark.parametrize("T,H,I,E,k,skew", CASES + draw_shapes(16, seed=77))
def test_mxfp8_forward_matches_oracle(T, H, I, E, k, skew):
    inp = make_mxfp8_inputs(dict(T=T, H=H, I=I, E=E, top_k=k, skew=skew), seed=0, device="cuda")
    out, views = run_mx(inp)
    o = moe_oracle.get("f32")
    ids, w = o.route(inp["router_logits"].cpu().numpy(), k)
    off, s2f, f2s = o.permute(ids, E)
    assert_routing_exact(views, ids, w, off, s2f, f2s)

    # token rows: gathered and quantised exactly as the oracle quantises x
    xc, xs = o.mx_quantize(inp["x"].float().cpu().numpy())
    tok = s2f // k
    assert np.array_equal(views["x_q"].cpu().numpy(), xc[tok])
    assert np.array_equal(unpack_act_scales(views["x_sf"].cpu().numpy(), off, H // 32, views["tile_rows"]), xs[tok])

    ref, h_pre, h_q, h_s = oracle_mx(inp, intermediates=True)
    # h: the same codes and scale bytes except where fp32 summation order moves a value across a rounding
    # boundary; a differing code must still be a valid quantisation of the oracle's h (within one step)
    got_q = views["h_q"].cpu().numpy()
    got_s = unpack_act_scales(views["h_sf"].cpu().numpy(), off, I // 32, views["tile_rows"])
    same = (got_q == h_q[s2f]) & (np.repeat(got_s, 32, axis=1) == np.repeat(h_s[s2f], 32, axis=1))
    assert same.mean() > 0.98, same.mean()
    got_h = TABLE[got_q] * np.repeat(np.exp2(got_s.astype(np.float64) - 127), 32, axis=1)
    scale = np.repeat(np.exp2(got_s.astype(np.float64) - 127), 32, axis=1)
    step = scale * np.maximum(np.abs(TABLE[got_q]), 2.0 ** -6) * 2.0 ** -3
    step = np.where(np.abs(TABLE[got_q]) == 448, 64 * scale, step)   # the top binade saturates: [448, 512) -> 448
    assert np.all(np.abs(got_h - h_pre[s2f]) <= 1.01 * step + 1e-30)

    assert_close_out(bf16_to_f64(out), ref, "mxfp8 out")


@pytest.mark.parametrize("cfg,lo,n", [(dict(T=160, H=256, I=128, E=16, top_k=4, skew=False), 4, 8),
                                      # wide token tiles (bound 384) with resident experts in the middle of the range
                                      (dict(T=1200, H=256, I=128, E=8, top_k=2, skew=False), 2, 4),
                                      (dict(T=1100, H=256, I=128, E=8, top_k=2, skew=True), 0, 3)])
def test_mxfp8_local_experts(cfg, lo, n):
    full = make_mxfp8_inputs(cfg, seed=3, device="cuda")
    inp = dict(full)
    for key in ("w13_q", "w13_s", "w2_q", "w2_s"):
        inp[key] = full[key][lo:lo + n].contiguous()
    out, views = run_mx(inp, local_offset=lo)
    # the oracle with the other experts' weights zeroed: their assignments contribute nothing
    z = dict(full)
    for key in ("w2_q",):
        z[key] = full[key].clone()
        z[key][:lo] = 0
        z[key][lo + n:] = 0
    ref = oracle_mx(z)
    assert_close_out(bf16_to_f64(out), ref, "mxfp8 local out")
    assert views["expert_offsets"][n].item() == int(((views["topk_ids"] >= lo) & (views["topk_ids"] < lo + n)).sum())


def test_mxfp8_non_finite_token_poisons_only_itself():
    inp = make_mxfp8_inputs(dict(T=8, H=128, I=128, E=2, top_k=1, skew=False), seed=5, device="cuda")
    inp["x"][3, 17] = float("inf")
    out, _ = run_mx(inp)
    got = out.float().cpu().numpy()
    assert np.all(np.isnan(got[3]))
    assert np.all(np.isfinite(np.delete(got, 3, axis=0)))


def test_mxfp8_rejects_shapes_outside_its_envelope():
    assert moe.moe_mxfp8_workspace_bytes(8, 128, 64, 2, 1) == 0   # I must be a multiple of 128
    inp = make_mxfp8_inputs(dict(T=8, H=128, I=128, E=2, top_k=1, skew=False), seed=1, device="cuda")
    ws = moe.alloc_workspace(1 << 20, "cuda")
    out = torch.empty((8, 128), dtype=torch.bfloat16, device="cuda")
    sf13 = moe.moe_mxfp8_pack_scales(inp["w13_s"], True)
    sf2 = moe.moe_mxfp8_pack_scales(inp["w2_s"], False)
    st = moe.moe_forward_mxfp8(inp["x"], inp["router_logits"], inp["w13_q"], sf13, inp["w2_q"], sf2, 1, out, ws[:1024],
                               check=False)
    assert st == -5  # MOE_ERR_WORKSPACE
    st = moe.moe_forward_mxfp8(inp["x"], inp["router_logits"], inp["w13_q"], None, inp["w2_q"], sf2, 1, out, ws, check=False)
    assert st == -1  # MOE_ERR_NULL


def test_mxfp8_repeated_calls_are_deterministic():
    inp = make_mxfp8_inputs(dict(T=300, H=256, I=256, E=16, top_k=4, skew=True), seed=2, device="cuda")
    a, _ = run_mx(inp)
    b, _ = run_mx(inp)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16))


def test_mxfp8_host_entry_point_equals_the_device_one():
    inp = make_mxfp8_inputs(dict(T=200, H=256, I=128, E=8, top_k=2, skew=False), seed=4, device="cuda")
    out, _ = run_mx(inp)
    T, H = inp["x"].shape
    ws = moe.alloc_workspace(moe.moe_mxfp8_workspace_bytes(T, H, 128, 8, 2), "cuda")
    xh, lh = inp["x"].cpu().pin_memory(), inp["router_logits"].cpu().pin_memory()
    oh = torch.empty((T, H), dtype=torch.bfloat16).pin_memory()
    moe.moe_forward_mxfp8_host(xh, lh, inp["w13_q"], moe.moe_mxfp8_pack_scales(inp["w13_s"], True), inp["w2_q"],
                               moe.moe_mxfp8_pack_scales(inp["w2_s"], False), 2, oh, ws)
    torch.cuda.synchronize()
    assert moe.moe_last_status(ws) == moe.MOE_OK
    assert torch.equal(oh.view(torch.int16), out.cpu().view(torch.int16))


def test_mxfp8_with_grouped_router_and_local_experts():
    """The configuration the paper's kernel serves, scaled down: FP8 operands, grouped sigmoid routing, a resident
    subset of the experts."""
    cfg = dict(T=180, H=256, I=128, E=32, top_k=4, skew=False)
    full = make_mxfp8_inputs(cfg, seed=8, device="cuda")
    lo, n = 8, 16
    inp = dict(full)
    for key in ("w13_q", "w13_s", "w2_q", "w2_s"):
        inp[key] = full[key][lo:lo + n].contiguous()
    bias = torch.linspace(-0.2, 0.2, 32).cuda()
    T, H, I, E, k = 180, 256, 128, 32, 4
    ws = moe.alloc_workspace(moe.moe_mxfp8_workspace_bytes(T, H, I, E, k), "cuda")
    ws.fill_(0xFF)
    out = torch.full((T, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    moe.moe_forward_mxfp8(inp["x"], inp["router_logits"], inp["w13_q"], moe.moe_mxfp8_pack_scales(inp["w13_s"], True),
                          inp["w2_q"], moe.moe_mxfp8_pack_scales(inp["w2_s"], False), k, out, ws, local_expert_offset=lo,
                          router=moe.grouped_router(4, 2, bias, 2.5))
    assert moe.moe_last_status(ws) == moe.MOE_OK
    o = moe_oracle.get("f32")
    logits = full["router_logits"].cpu().numpy()
    ids, w = o.route_grouped(logits, k, 4, 2, bias=bias.cpu().numpy(), scale=2.5)
    views = moe.mx_workspace_views(ws, T, H, I, E, k)
    assert np.array_equal(views["topk_ids"].cpu().numpy(), ids)
    assert np.array_equal(views["topk_weights"].cpu().numpy(), w)
    # reference: every expert applied to its tokens by the oracle's sampled MX form, combined with the grouped
    # weights here, assignments to experts that are not resident dropped
    tokens = np.arange(T, dtype=np.int32)
    ref = np.zeros((T, H))
    host = {key: full[key].cpu().numpy() for key in ("w13_q", "w13_s", "w2_q", "w2_s")}
    xb = bf16_bits(full["x"])
    for e in range(lo, lo + n):
        sel = np.nonzero((ids == e).any(axis=1))[0].astype(np.int32)
        if len(sel) == 0:
            continue
        # a one-expert layer (k = 1, every logit column but e irrelevant): its output is expert e applied to the token
        one = o.forward_mxfp8(xb[sel], np.zeros((len(sel), 1), np.float32), host["w13_q"][e:e + 1], host["w13_s"][e:e + 1],
                              host["w2_q"][e:e + 1], host["w2_s"][e:e + 1], 1)
        wsel = np.array([w[t][list(ids[t]).index(e)] for t in sel])
        ref[sel] += wsel[:, None] * one
    err = np.abs(bf16_to_f64(out) - ref)
    assert np.all(err <= 2e-2 * (2.5 + np.abs(ref)))


def test_mxfp8_large_batch_codes_and_scale_bytes():
    """A batch of 16384 assignments: the scattered codes and every scale byte must equal the oracle's, and sampled
    outputs its layer."""
    cfg = dict(T=2048, H=4096, I=128, E=16, top_k=8, skew=False)
    inp = make_mxfp8_inputs(cfg, seed=21, device="cuda")
    out, views = run_mx(inp)
    T, H, I, E, k = (cfg[n] for n in ("T", "H", "I", "E", "top_k"))
    o = moe_oracle.get("f32")
    logits = inp["router_logits"].cpu().numpy()
    ids, w = o.route(logits, k)
    off, s2f, f2s = o.permute(ids, E)
    assert_routing_exact(views, ids, w, off, s2f, f2s)
    xc, xs = o.mx_quantize(inp["x"].float().cpu().numpy())
    tok = s2f // k
    assert np.array_equal(views["x_q"].cpu().numpy(), xc[tok])
    # scale bytes: vectorised form of unpack_act_scales
    tile = views["tile_rows"]
    apt, stride = (tile + 127) // 128, min(tile, 256)
    per_tile = np.array([expert_tile_rows(int(off[e + 1] - off[e]), tile) if off[e + 1] > off[e] else tile for e in range(E)])
    e_of_row = np.searchsorted(off, np.arange(off[E]), side="right") - 1
    i = np.arange(off[E]) - off[e_of_row]
    r = i % per_tile[e_of_row]
    atom = (off[e_of_row] // stride + e_of_row + i // per_tile[e_of_row]) * apt + r // 128
    base = (r % 128 % 32) * 16 + (r % 128 // 32) * 4
    atoms = views["x_sf"].cpu().numpy()
    got = np.stack([atoms[b // 4, atom, base + b % 4] for b in range(H // 32)], axis=1)
    assert np.array_equal(got, xs[tok])
    tokens = np.array([0, 1, 777, T - 1], dtype=np.int32)
    need = sorted({int(e) for t in tokens for e in ids[t]})
    experts = {e: tuple(inp[n][e].cpu().numpy() for n in ("w13_q", "w13_s", "w2_q", "w2_s")) for e in need}
    ref = o.forward_mxfp8_sampled(bf16_bits(inp["x"]), logits, experts, I, k, tokens)
    assert_close_out(bf16_to_f64(out[torch.from_numpy(tokens).long().cuda()]), ref, "two-step sampled out")
