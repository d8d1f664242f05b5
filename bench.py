#!/usr/bin/env python
"""Benchmark of the MoE layer forward pass (one step = one whole pass: router, sort-scatter, row
gather, gate/up GEMM + SwiGLU, down GEMM, combine) on seeded synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

Prints ONE JSON line.  With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank
runs an independent replica on its own tokens -- the layer has no exchange step on one node, so
there is no data-path collective -- and the line reports the aggregate (weak scaling).
`--impl reference` times the CPU oracle (test infrastructure under oracle/) on the host cores for
the same workload and metric; it is a deliberately plain program, reported as a baseline.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2602_19128_b200.inputs import (CONFIGS, LOCAL_CONFIGS, bf16_bits, make_inputs,  # noqa: E402
                                          quantize_fp8_blocks, quantize_mxfp8)

CONFIGS = dict(CONFIGS, **LOCAL_CONFIGS)  # the five workloads plus the local-expert-subset shapes

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024
# Which roofline bounds the dominant kernel (gate/up GEMM) of each workload: weight bytes per useful
# flop put mixtral / dsv3_decode (and tiny) below the ridge point and the prefill-sized ones above it.
BOUND = {"tiny": "hbm", "mixtral": "hbm", "dsv3_decode": "hbm", "dsv3_prefill": "tensor", "skewed": "tensor",
         "dsv3_local32_prefill": "hbm", "dsv3_local32_decode": "hbm"}
# DRAM bytes (read + write) of one gate/up GEMM launch, from the ncu capture summarised under profiles/.
NCU_TRAFFIC_BYTES = {"mixtral": 1928438528}


def load_peaks() -> dict:
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), tflops_burst=float(d["bf16_tflops"]),
                    tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi (clocks, power, throttle reasons) for one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            uuid = str(torch.cuda.get_device_properties(device).uuid)
            ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            self.proc = subprocess.Popen(["nvidia-smi", "-i", ident, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "25"], stdout=self.tmp,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unavailable"])
        time.sleep(0.03)  # let the last sample under load be written
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        rows = [r.split(",") for r in Path(self.tmp.name).read_text().strip().splitlines() if r.count(",") >= 7]
        os.unlink(self.tmp.name)
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); smax.append(float(r[1])); power.append(float(r[2]))
            except ValueError:
                continue
            for n, v in zip(names, r[4:8]):
                if v.strip().lower() == "active":
                    reasons.add(n)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no_samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), power_w=round(statistics.median(power), 1),
                    samples=len(sm), reasons=sorted(reasons), window="timed steps and the instrumented pass after them")


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        return dist, rank, world, local
    if n_gpus != 1:
        raise SystemExit("--gpus N > 1 must be launched with torch.distributed.run (one rank per GPU)")
    torch.cuda.set_device(0)
    return None, 0, 1, 0


def max_over_ranks(dist, value: float, device) -> float:
    """The slowest rank's time: the whole job is as slow as that rank."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_tokens_per_s(world: int, tokens_per_rank_step: int, steps: int, total_ms: float) -> float:
    """Whole-job throughput of `world` independent replicas (weak scaling): all tokens / slowest time."""
    return world * tokens_per_rank_step * steps / (total_ms * 1e-3)


def flush_l2(buf: torch.Tensor):
    buf.add_(1)


def oracle_sample(cfg_name: str, inp: dict, n_tokens: int, seed: int = 0):
    """Host-side arguments for the oracle on a bounded sample of tokens: only the experts those tokens
    route to are copied to the host."""
    from oracle import moe_oracle
    o = moe_oracle.get("f32")
    T, k, I = inp["T"], inp["top_k"], inp["I"]
    rng = np.random.default_rng(seed)
    tokens = np.sort(rng.choice(T, size=min(n_tokens, T), replace=False)).astype(np.int32)
    logits = inp["router_logits"].cpu().numpy()
    ids, _ = o.route(logits, k)
    need = sorted({int(e) for t in tokens for e in ids[t]})
    experts = {e: (bf16_bits(inp["w13"][e]), bf16_bits(inp["w2"][e])) for e in need}
    return o, bf16_bits(inp["x"]), logits, experts, I, k, tokens


def token_tile_bound(T: int, E: int, k: int) -> int:
    """The library's token-tile bound for the bf16 layer: the smallest of 32, 64, 128 holding 1.5 x the mean rows
    per expert, else 256 (reporting only; mirrors the rule stated in the design notes)."""
    avg = T * k / E
    for nt in (32, 64, 128):
        if 1.5 * avg <= nt:
            return nt
    return 256


def computed_rows(counts, tile_bound: int, even: bool) -> int:
    """Rows the GEMMs multiply (MMA N summed over token tiles): an expert's rows are cut into as few tiles as fit
    under the bound, evenly sized (bf16) or of exactly the bound (MX), and each tile is rounded up to 16 rows."""
    total = 0
    for c in (int(v) for v in counts):
        if c == 0:
            continue
        n_tiles = -(-c // tile_bound)
        rows = -(-(-(-c // n_tiles)) // 16) * 16 if even else tile_bound
        for j in range(n_tiles):
            total += -(-min(rows, c - j * rows) // 16) * 16
    return total


def time_oracle(cfg_name: str, inp: dict, budget_s: float):
    """Times the oracle, as it stands, on a token sample sized to take roughly budget_s seconds."""
    from oracle import moe_oracle
    cores = moe_oracle.get("f32").num_threads
    o, x, logits, experts, I, k, tokens = oracle_sample(cfg_name, inp, cores)
    t0 = time.perf_counter()
    o.forward_sampled(x, logits, experts, I, k, tokens)
    t_probe = time.perf_counter() - t0
    rounds = max(1, min(64, int(budget_s / max(t_probe, 1e-3))))
    n = min(inp["T"], cores * rounds)
    if n > len(tokens):
        o, x, logits, experts, I, k, tokens = oracle_sample(cfg_name, inp, n)
        t0 = time.perf_counter()
        o.forward_sampled(x, logits, experts, I, k, tokens)
        t_probe = time.perf_counter() - t0
    return dict(value=len(tokens) / t_probe, unit=UNIT, cores=cores, kind="oracle",
                sample=f"{len(tokens)} of {inp['T']} tokens of '{cfg_name}' (all top-k experts of each), float oracle, "
                       f"{t_probe:.2f} s wall")


def time_oracle_mx(cfg_name: str, x, logits, w13_q, s13, w2_q, s2, k: int, budget_s: float):
    """Times the oracle's MX FP8 layer, as it stands, on the first tokens of the workload (all weights on the host)."""
    from oracle import moe_oracle
    o = moe_oracle.get("f32")
    cores = o.num_threads
    host = [t.cpu().numpy() for t in (w13_q, s13, w2_q, s2)]
    xb, lg = bf16_bits(x), logits.cpu().numpy()

    def run(n):
        t0 = time.perf_counter()
        o.forward_mxfp8(xb[:n], lg[:n], *host, k)
        return time.perf_counter() - t0

    n = min(x.shape[0], cores)
    t = run(n)
    rounds = max(1, min(64, int(budget_s / max(t, 1e-3))))
    if min(x.shape[0], cores * rounds) > n:
        n = min(x.shape[0], cores * rounds)
        t = run(n)
    return dict(value=n / t, unit=UNIT, cores=cores, kind="oracle",
                sample=f"first {n} of {x.shape[0]} tokens of '{cfg_name}' (all top-k experts of each), float oracle, "
                       f"MX FP8 layer, {t:.2f} s wall")


def run_reference(args):
    """The reference arm: the CPU oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import moe_oracle
    cfg = CONFIGS[args.config]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    inp = make_inputs(CONFIGS[args.config], seed=args.seed, device=dev)
    cores = moe_oracle.get("f32").num_threads
    o, x, logits, experts, I, k, tokens = oracle_sample(args.config, inp, cores)
    del inp
    t0 = time.perf_counter()
    o.forward_sampled(x, logits, experts, I, k, tokens)
    probe = time.perf_counter() - t0
    # keep the whole run within a few minutes: shrink the per-step sample if K steps would not fit
    total_steps = args.steps + args.warmup
    n = len(tokens)
    if probe * total_steps > 240.0:
        n = max(1, int(n * 240.0 / (probe * total_steps)))
        tokens = tokens[:n]
    for _ in range(args.warmup):
        o.forward_sampled(x, logits, experts, I, k, tokens)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        o.forward_sampled(x, logits, experts, I, k, tokens)
    wall = time.perf_counter() - t0
    value = n * args.steps / wall
    sample = f"{n} tokens of '{args.config}' per step (all top-k experts of each), float oracle"
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * wall / args.steps, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f32", data="synthetic",
                config=dict(workload=args.config, **{k_: cfg[k_] for k_ in ("T", "H", "I", "E", "top_k")},
                            tokens_per_step=n),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line), flush=True)


def run_ours(args):
    import paper_2602_19128_b200 as moe
    dist, rank, world, local = dist_setup(args.gpus)
    dev = torch.device("cuda", local)
    cfg = CONFIGS[args.config]
    T, H, I, E, k = (cfg[n] for n in ("T", "H", "I", "E", "top_k"))
    inp = make_inputs(CONFIGS[args.config], seed=args.seed + rank, device=dev)
    x, logits, w13, w2 = inp["x"], inp["router_logits"], inp["w13"], inp["w2"]
    local_offset, n_local = inp["local_offset"], inp["local"]
    out = torch.empty((T, H), dtype=torch.bfloat16, device=dev)
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), dev)
    fp8 = args.weights == "fp8"
    mx = args.weights == "mxfp8"
    if mx:  # MX FP8: E4M3 codes + one E8M0 scale byte per 32 elements, scale bytes repacked once; bf16 originals dropped
        ws = moe.alloc_workspace(moe.moe_mxfp8_workspace_bytes(T, H, I, E, k), dev)
        w13, s13 = quantize_mxfp8(w13)
        w2, s2 = quantize_mxfp8(w2)
        inp["w13"], inp["w2"] = None, None
        w13_sf, w2_sf = moe.moe_mxfp8_pack_scales(s13, gate_up=True), moe.moe_mxfp8_pack_scales(s2, gate_up=False)
        torch.cuda.synchronize()
        mx_plain_scales = (s13, s2) if (w13.numel() + w2.numel()) <= (4 << 30) else None  # for the CPU baseline leg
        del s13, s2
    if fp8:  # FP8 (E4M3) codes + one fp32 scale per 128 x 128 block; the bf16 originals are dropped
        if n_local != E:
            raise SystemExit("--weights fp8 covers the whole-layer workloads")
        w13, w13_scale = quantize_fp8_blocks(w13)
        w2, w2_scale = quantize_fp8_blocks(w2)
        inp["w13"], inp["w2"] = None, None
    bytes_per_weight = 1 if fp8 else (1 + 1 / 32) if mx else 2
    weight_bytes = int((w13.numel() + w2.numel()) * bytes_per_weight)
    need_flush = weight_bytes < 2 * L2_BYTES

    grouped = None
    if args.router == "grouped":  # the published DeepSeek-V3 setting: 8 groups, 4 eligible, weights scaled by 2.5
        if not mx or E % 8 != 0 or (E // 8) & (E // 8 - 1) or 4 * (E // 8) < k:
            raise SystemExit("--router grouped is wired for --weights mxfp8 and E = 8 groups of a power of two")
        gen = torch.Generator(device=dev)
        gen.manual_seed(args.seed + 1000 + rank)
        router_bias = torch.randn(E, generator=gen, device=dev) * 0.1
        grouped = moe.grouped_router(8, 4, router_bias, 2.5)

    def forward(events=None):
        if mx:
            moe.moe_forward_mxfp8(x, logits, w13, w13_sf, w2, w2_sf, k, out, ws, stage_events=events,
                                  local_expert_offset=local_offset, router=grouped)
        elif fp8:
            moe.moe_forward_fp8w(x, logits, w13, w13_scale, w2, w2_scale, k, out, ws, stage_events=events)
        elif events is None:
            moe.moe_forward_local(x, logits, w13, w2, k, local_offset, out, ws)
        else:
            moe.moe_forward_staged(x, logits, w13, w2, k, out, ws, events, local_expert_offset=local_offset)
    flush_buf = torch.zeros(2 * L2_BYTES // 4, dtype=torch.float32, device=dev) if need_flush else None
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        forward()
    status = moe.moe_last_status(ws)
    if status != moe.MOE_OK:
        raise SystemExit(f"device status {status}: {moe.moe_status_string(status)}")
    # The K timed steps run as a user's would: no event between the kernels of a step (an event record between two
    # launches costs several microseconds of launch pipelining).  With an L2 flush between steps each step gets its
    # own pair of events; otherwise one pair brackets all K.
    step_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(args.steps if need_flush else 1)]
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    if not need_flush:
        step_events[0][0].record()
    for s in range(args.steps):
        if need_flush:
            flush_l2(flush_buf)
            step_events[s][0].record()
        forward()
        if need_flush:
            step_events[s][1].record()
    if not need_flush:
        step_events[0][1].record()
    barrier()
    total_ms = sum(a.elapsed_time(b) for a, b in step_events)
    # Per-kernel times: the same steps again, instrumented with an event between the stages.
    # (at least 0.1 s of it, so that the clock sampler sees the load even when K is small)
    n_staged = min(max(min(args.steps, 100), int(100.0 * args.steps / max(total_ms, 1e-3)) + 1), 2000)
    stage_events = [moe.make_stage_events() for _ in range(n_staged)]
    for s in range(n_staged):
        if need_flush:
            flush_l2(flush_buf)
        forward(stage_events[s])
    barrier()
    # the clock samples cover the timed steps and the instrumented pass over the same steps (the same load), so that
    # a short run still yields samples under load
    clocks = sampler.stop() if sampler else None
    stage_ms = {name: statistics.fmean(ev[i].elapsed_time(ev[i + 1]) for ev in stage_events)
                for i, name in enumerate(moe.STAGE_NAMES)}
    total_ms = max_over_ranks(dist, total_ms, dev)
    status = moe.moe_last_status(ws)
    if status != moe.MOE_OK:
        raise SystemExit(f"device status {status}: {moe.moe_status_string(status)}")
    views = moe.mx_workspace_views(ws, T, H, I, E, k) if mx else moe.workspace_views(ws, T, H, I, E, k)
    counts = torch.diff(views["expert_offsets"][:n_local + 1]).cpu().numpy()
    rows_scheduled = int(counts.sum())  # = T*k unless only a subset of the experts is resident
    n_active = int((counts > 0).sum())

    # ---- end to end through the host-buffer entry point ---------------------------------------------
    xh = x.cpu().pin_memory()
    lh = logits.cpu().pin_memory()
    oh = torch.empty((T, H), dtype=torch.bfloat16).pin_memory()
    x_stage, l_stage = torch.empty_like(x), torch.empty_like(logits)

    def host_step(out_host=None, workspace=None, stream=None):
        out_host = oh if out_host is None else out_host
        workspace = ws if workspace is None else workspace
        if mx:
            moe.moe_forward_mxfp8_host(xh, lh, w13, w13_sf, w2, w2_sf, k, out_host, workspace, stream=stream,
                                       local_expert_offset=local_offset, router=grouped)
        elif fp8:  # no host-buffer entry point for this variant: the same copies, issued here on the same stream
            x_stage.copy_(xh, non_blocking=True)
            l_stage.copy_(lh, non_blocking=True)
            moe.moe_forward_fp8w(x_stage, l_stage, w13, w13_scale, w2, w2_scale, k, out, ws)
            oh.copy_(out, non_blocking=True)
        else:
            moe.moe_forward_host(xh, lh, w13, w2, k, out_host, workspace, stream=stream, local_expert_offset=local_offset)

    for _ in range(3):
        host_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2e_ms = 0.0
    if need_flush:
        for _ in range(args.steps):
            flush_l2(flush_buf)
            e0.record()
            host_step()
            e1.record()
            e1.synchronize()
            e2e_ms += e0.elapsed_time(e1)
    else:
        e0.record()
        for _ in range(args.steps):
            host_step()
        e1.record()
        e1.synchronize()
        e2e_ms = e0.elapsed_time(e1)
    barrier()
    e2e_ms = max_over_ranks(dist, e2e_ms, dev)
    same = bool(torch.equal(oh.view(torch.int16), out.cpu().view(torch.int16)))

    # The same K end-to-end steps as a serving loop would issue them: two streams, each with its own workspace
    # and result buffer, alternating, so that one step's copies overlap the other's kernels.  Every step still
    # copies its inputs in and its result out.
    e2e_overlapped_ms = None
    if not need_flush and not fp8:
        ws_b = moe.alloc_workspace(ws.numel(), dev)
        oh_b = torch.empty_like(oh).pin_memory()
        lanes = [(torch.cuda.Stream(device=dev), oh, ws), (torch.cuda.Stream(device=dev), oh_b, ws_b)]
        main = torch.cuda.current_stream()
        for st, o_h, w_s in lanes:  # warm both lanes
            st.wait_stream(main)
            host_step(o_h, w_s, st)
        for st, _, _ in lanes:
            main.wait_stream(st)
        barrier()
        e0.record()
        for st, _, _ in lanes:
            st.wait_event(e0)
        for i in range(args.steps):
            st, o_h, w_s = lanes[i % 2]
            host_step(o_h, w_s, st)
        for st, _, _ in lanes:
            main.wait_stream(st)
        e1.record()
        e1.synchronize()
        e2e_overlapped_ms = max_over_ranks(dist, e0.elapsed_time(e1), dev)
        barrier()
        same = same and bool(torch.equal(oh_b.view(torch.int16), out.cpu().view(torch.int16)))
        if moe.moe_last_status(ws_b) != moe.MOE_OK:
            raise SystemExit("device status of the second end-to-end lane is not ok")

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (gate/up GEMM + SwiGLU) -----------------------------------
    peaks = load_peaks()
    A = rows_scheduled
    t_gemm1 = stage_ms["gemm1_swiglu"] * 1e-3
    bound = BOUND[args.config]
    if bound == "hbm":
        algorithmic = int(n_active * 2 * I * H * bytes_per_weight)  # bytes of the active experts' w13, read once
        achieved = algorithmic / t_gemm1 / 1e9
        peak, unit = peaks["hbm_gbs"], "GB/s"
    else:
        algorithmic = 4.0 * A * H * I  # useful flops of the gate and up projections
        achieved = algorithmic / t_gemm1 / 1e12
        peak, unit = peaks["tflops_sustained"], "TFLOP/s"
        if mx:  # 8-bit operands: the measured bf16 peak times the nominal fp8 / bf16 ratio
            peak *= 2
    step_s = total_ms * 1e-3 / args.steps
    active_weight_bytes = int(n_active * 3 * I * H * bytes_per_weight)
    roofline = dict(bound=bound, kernel="gate/up GEMM (grouped_gemm_tc*_kernel<swiglu>)", achieved=achieved, peak=peak,
                    unit=unit, frac=achieved / peak, peak_source=f"of {peaks['source']}",
                    traffic=None if (fp8 or mx) else NCU_TRAFFIC_BYTES.get(args.config), algorithmic_per_launch=algorithmic,
                    kernel_ms=stage_ms["gemm1_swiglu"])
    # per-step latencies: from the timed steps when each has its own events, else from the instrumented pass
    per_step_ms = sorted(a.elapsed_time(b) for a, b in step_events) if need_flush else \
        sorted(ev[0].elapsed_time(ev[-1]) for ev in stage_events)
    tile_bound = int(views["tile_rows"]) if mx else token_tile_bound(T, E, k)
    layer = dict(stage_ms={n: round(v, 5) for n, v in stage_ms.items()}, n_active_experts=n_active,
                 latency_ms_median=statistics.median(per_step_ms), latency_ms_min=per_step_ms[0],
                 latency_source="timed steps" if need_flush else "instrumented pass (events between the stages)",
                 stage_ms_source=f"instrumented pass of {n_staged} steps after the timed ones",
                 padding_efficiency=rows_scheduled / max(1, computed_rows(counts, tile_bound, even=not mx)),
                 weight_gbs_frac_nominal=active_weight_bytes / step_s / 1e9 / 8000.0,
                 useful_tflops_frac_nominal=6.0 * A * H * I / step_s / 1e12 / (4500.0 if mx else 2250.0),
                 rows_per_expert_min=int(counts.min()), rows_per_expert_max=int(counts.max()),
                 weight_gbs=active_weight_bytes / step_s / 1e9, weight_gbs_frac=active_weight_bytes / step_s / 1e9 / peaks["hbm_gbs"],
                 useful_tflops=6.0 * A * H * I / step_s / 1e12,
                 useful_tflops_frac_sustained=6.0 * A * H * I / step_s / 1e12 / peaks["tflops_sustained"],
                 useful_tflops_frac_burst=6.0 * A * H * I / step_s / 1e12 / peaks["tflops_burst"])

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline and n_local == E and not fp8 and not mx:
        cpu_baseline = time_oracle(args.config, inp, budget_s=15.0)
    if world == 1 and not args.no_cpu_baseline and n_local == E and mx and mx_plain_scales is not None:
        cpu_baseline = time_oracle_mx(args.config, x, logits, w13, mx_plain_scales[0], w2, mx_plain_scales[1], k, 15.0)

    line = dict(metric=METRIC, value=aggregate_tokens_per_s(world, T, args.steps, total_ms), unit=UNIT, n_gpus=world,
                steps=args.steps, warmup=max(args.warmup, 3), ms_per_step=total_ms / args.steps, higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="mxfp8" if mx else "bf16", data="synthetic",
                config=dict(workload=args.config, T=T, H=H, I=I, E=E, top_k=k, resident_experts=n_local,
                            weights="fp8 e4m3 codes + fp32 scale per 128x128 block" if fp8 else
                            "mxfp8: e4m3 codes + e8m0 scale per 32 elements, activations quantised on the fly" if mx else "bf16",
                            router=args.router, parallelism=f"replicas x{world}",
                            l2="flushed between steps" if need_flush else "weights larger than L2, no flush",
                            seed=args.seed),
                clocks=clocks,
                e2e=dict(value=aggregate_tokens_per_s(world, T, args.steps, e2e_ms), unit=UNIT,
                         h2d_bytes_per_step=T * H * 2 + T * E * 4, d2h_bytes_per_step=T * H * 2,
                         ms_per_step=e2e_ms / args.steps, matches_device_path=same,
                         overlapped=None if e2e_overlapped_ms is None else dict(
                             value=aggregate_tokens_per_s(world, T, args.steps, e2e_overlapped_ms), unit=UNIT,
                             ms_per_step=e2e_overlapped_ms / args.steps,
                             how="two streams with their own workspaces alternate, so copies overlap kernels")),
                gpu_launches=moe.moe_forward_launch_count(T) * args.steps,
                roofline=roofline, layer=layer, cpu_baseline=cpu_baseline)
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=500)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", choices=list(CONFIGS), default="mixtral")
    ap.add_argument("--shape", default=None, help="custom T,H,I,E,top_k instead of a named workload (profiling)")
    ap.add_argument("--weights", choices=["bf16", "fp8", "mxfp8"], default="bf16",
                    help="fp8: expert weights as E4M3 codes with one fp32 scale per 128 x 128 block (moe_forward_fp8w); "
                         "mxfp8: weights and activations in MX FP8 on the block-scaled MMA (moe_forward_mxfp8)")
    ap.add_argument("--router", choices=["softmax", "grouped"], default="softmax",
                    help="grouped: sigmoid scores, selection bias, 8 groups of which 4 eligible, weights x 2.5 (with --weights mxfp8)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.shape:
        T, H, I, E, k = (int(v) for v in args.shape.split(","))
        args.config = f"custom_{T}x{H}x{I}x{E}x{k}"
        CONFIGS[args.config] = dict(T=T, H=H, I=I, E=E, top_k=k, skew=False)
        BOUND[args.config] = "hbm"
    if args.impl == "reference":
        if args.config in LOCAL_CONFIGS:
            raise SystemExit("the reference arm covers the five whole-layer workloads")
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
