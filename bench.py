#!/usr/bin/env python
"""Benchmark of the MoE layer forward pass (one step = one whole pass: router, sort-scatter, token rows
into expert order, gate/up GEMM + SwiGLU, down GEMM, combine) on seeded synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

Prints ONE JSON line.  Without --config the headline is the largest workload that fits one GPU, the
DeepSeek-V3-shaped prefill batch (`dsv3_prefill`), with `roofline`, `cpu_baseline` and `e2e` for it, and a
`sweep` object that holds the other four workloads (tiny, mixtral, skewed, dsv3_decode), each with its own
step time, roofline fractions and clock record.  The two DeepSeek-shaped batches share one draw of the
256 experts' weights.  --config NAME measures that workload alone.

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs an independent replica on
its own tokens -- the layer has no exchange step on one node, so there is no data-path collective -- and
the line reports the aggregate (weak scaling); the sweep is a single-GPU report and is left out.
`--impl reference` times the CPU oracle (test infrastructure under oracle/) on the host cores for the same
workload and metric; it is a deliberately plain program, reported as a baseline.
"""
from __future__ import annotations

import argparse
import faulthandler
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time
from pathlib import Path

import numpy as np
import torch

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

from paper_2602_19128_b200.inputs import (CONFIGS, GQA_CONFIGS, LOCAL_CONFIGS, bf16_bits, make_gqa_inputs,  # noqa: E402
                                          make_inputs)
from tests.weight_quantizers import quantize_fp8_blocks, quantize_mxfp8  # noqa: E402

CONFIGS = dict(CONFIGS, **LOCAL_CONFIGS)  # the five workloads plus the local-expert-subset shapes

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"
HEADLINE = "dsv3_prefill"                      # the largest workload that fits one GPU
SWEEP = ("tiny", "mixtral", "skewed", "dsv3_decode")
L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
SM_COUNT = 148
TENSOR_FLOP_PER_CLK_SM = 8192                  # dense bf16, fp32 accumulation: 2.25 PFLOP/s at 1.86 GHz on 148 SMs
# Which roofline bounds the dominant kernel (gate/up GEMM) of each workload: weight bytes per useful
# flop put mixtral / dsv3_decode (and tiny) below the ridge point and the prefill-sized ones above it.
BOUND = {"tiny": "hbm", "mixtral": "hbm", "dsv3_decode": "hbm", "dsv3_prefill": "tensor", "skewed": "tensor",
         "dsv3_local32_prefill": "hbm", "dsv3_local32_decode": "hbm"}
# DRAM bytes (read + write) of one gate/up GEMM launch, from the ncu captures summarised under profiles/.  Each
# entry names the kernel instance and the commit it was captured on; `scale` multiplies a capture of a smaller
# case of the same per-expert shape up to the units (experts) of a full launch.
NCU_TRAFFIC = {
    "mixtral": dict(bytes=1928651520, scale=1, kernel="grouped_gemm_tc_pair_kernel<256,7,1,swiglu>", commit="b010af5",
                    source="profiles/grouped_gemm_tc_pair_mixtral.md"),
    "dsv3_prefill": dict(bytes=2055034880, scale=8, kernel="grouped_gemm_tc_ring_kernel<320,6,swiglu>", commit="b010af5",
                         source="profiles/grouped_gemm_tc_ring_dsv3_prefill.md",
                         note="captured on T=1024, E=32, top_k=8 (the headline's per-expert shape with an eighth of "
                              "its experts); traffic grows with the number of experts"),
}


def load_peaks() -> dict:
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), tflops_burst=float(d["bf16_tflops"]),
                    tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock, power and throttle reasons of one GPU while a timed region runs: NVML queries from a
    thread of this process, a few milliseconds apart (read-only), or an nvidia-smi child process if NVML cannot
    be loaded."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    REASON_BITS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, device: int, period_s: float = 0.01):
        self.rows, self.proc, self.thread, self.tmp = [], None, None, None
        self.stop_flag = threading.Event()
        uuid = str(torch.cuda.get_device_properties(device).uuid)
        ident = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        try:
            import pynvml
            pynvml.nvmlInit()
            h = pynvml.nvmlDeviceGetHandleByUUID(ident)
            smax = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                pynvml.nvmlDeviceGetCurrentClocksThrottleReasons
            reasons_fn(h)  # an unsupported query raises here, not in the thread

            def loop():
                while not self.stop_flag.is_set():
                    try:
                        self.rows.append((float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)), smax,
                                          pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0, int(reasons_fn(h))))
                    except Exception:
                        pass
                    time.sleep(period_s)
            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            self.how = "NVML thread"
        except Exception:
            self.thread = None
            self.how = "nvidia-smi"
            self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            try:
                self.proc = subprocess.Popen(["nvidia-smi", "-i", ident, f"--query-gpu={self.FIELDS}",
                                              "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.tmp,
                                             stderr=subprocess.DEVNULL)
            except Exception:
                self.proc = None

    def stop(self) -> dict:
        sm, smax, reasons, power = [], [], set(), []
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join(timeout=2)
            for c, m, p, bits in self.rows:
                sm.append(c); smax.append(m); power.append(p)
                reasons.update(n for n in self.NAMES if bits & self.REASON_BITS[n])
        elif self.proc is not None:
            time.sleep(0.03)  # let the last sample under load be written
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.tmp.flush()
            rows = [r.split(",") for r in Path(self.tmp.name).read_text().strip().splitlines() if r.count(",") >= 7]
            os.unlink(self.tmp.name)
            for r in rows:
                try:
                    sm.append(float(r[0])); smax.append(float(r[1])); power.append(float(r[2]))
                except ValueError:
                    continue
                reasons.update(n for n, v in zip(self.NAMES, r[4:8]) if v.strip().lower() == "active")
        else:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unavailable"])
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no_samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), sm_mhz_lowest=min(sm), sm_mhz_highest=max(sm),
                    power_w=round(statistics.median(power), 1), samples=len(sm), reasons=sorted(reasons), how=self.how,
                    window="the timed steps and the instrumented pass after them")


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


def fraction_at_clock(flops: float, seconds: float, sm_mhz):
    """Useful flops of a kernel over what the tensor pipes could do in its time AT THE CLOCK THE SMs RAN AT
    (SMs x 8192 flop/clk x the sampled median clock): separates the kernel from the power state of the box."""
    if not sm_mhz or seconds <= 0:
        return None
    return flops / (seconds * sm_mhz * 1e6 * SM_COUNT * TENSOR_FLOP_PER_CLK_SM)


def tensor_fractions(flops: float, seconds: float, peaks: dict, sm_mhz, scale: float = 1.0) -> dict:
    """A kernel's useful TFLOP/s against every denominator in use: the measured sustained and burst cuBLAS
    rates, the nominal dense peak, and the at-clock pipe peak (scale = 2 for 8-bit operands)."""
    tf = flops / seconds / 1e12
    at_clock = fraction_at_clock(flops, seconds, sm_mhz)
    return dict(achieved=tf, unit="TFLOP/s", frac_sustained=tf / (scale * peaks["tflops_sustained"]),
                frac_burst=tf / (scale * peaks["tflops_burst"]), frac_nominal=tf / (scale * NOMINAL_BF16_TFLOPS),
                frac_at_clock=None if at_clock is None else at_clock / scale)


def hbm_fractions(nbytes: float, seconds: float, peaks: dict) -> dict:
    """Bytes per second against the measured copy bandwidth (a read + write stream: a read-only stream can exceed
    it) and against the nominal 8 TB/s."""
    gbs = nbytes / seconds / 1e9
    return dict(achieved=gbs, unit="GB/s", frac_measured_copy=gbs / peaks["hbm_gbs"], frac_nominal=gbs / NOMINAL_HBM_GBS)


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


def computed_rows(counts, tile_bound: int, even: bool) -> int:
    """Rows the GEMMs multiply (MMA N summed over token tiles): an expert's rows are one tile if they fit under the
    bound, else as few tiles as fit under min(bound, 256), evenly sized (bf16) or of exactly the bound (MX), and each
    tile is rounded up to 16 rows."""
    total = 0
    for c in (int(v) for v in counts):
        if c == 0:
            continue
        n_tiles = 1 if c <= tile_bound else -(-c // min(tile_bound, 256))
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
    name = args.config or HEADLINE
    cfg = CONFIGS[name]
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    inp = make_inputs(cfg, seed=args.seed, device=dev)
    cores = moe_oracle.get("f32").num_threads
    o, x, logits, experts, I, k, tokens = oracle_sample(name, inp, cores)
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
    sample = f"{n} tokens of '{name}' per step (all top-k experts of each), float oracle"
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1e3 * wall / args.steps, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f32", data="synthetic",
                config=dict(workload=name, **{k_: cfg[k_] for k_ in ("T", "H", "I", "E", "top_k")},
                            oracle_tokens_per_step=n),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line), flush=True)


class Ctx:
    """What every workload of one bench run shares: the library binding, the process group, the device."""
    def __init__(self, moe, dist, rank, world, local, args):
        self.moe, self.dist, self.rank, self.world, self.local, self.args = moe, dist, rank, world, local, args
        self.dev = torch.device("cuda", local)
        self.peaks = load_peaks()

    def barrier(self):
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
        torch.cuda.synchronize()


def measure(ctx: Ctx, name: str, inp: dict, steps, warmup: int, with_e2e: bool, with_cpu_baseline: bool,
            min_timed_s: float = 0.0) -> dict:
    """Times one workload.  `steps` = None sizes the timed region to about `min_timed_s` seconds (sweep
    entries); otherwise exactly `steps` steps are timed.  Warm-up runs at least `warmup` steps AND at least
    --warm-seconds of back-to-back steps, so that the timed steps see the clock the GPU settles at under its
    power cap rather than the first milliseconds of a cool, fast-clocked part."""
    moe, args, dist, dev, peaks = ctx.moe, ctx.args, ctx.dist, ctx.dev, ctx.peaks
    cfg = CONFIGS[name]
    T, H, I, E, k = (cfg[n] for n in ("T", "H", "I", "E", "top_k"))
    x, logits, w13, w2 = inp["x"], inp["router_logits"], inp["w13"], inp["w2"]
    local_offset, n_local = inp["local_offset"], inp["local"]
    out = torch.empty((T, H), dtype=torch.bfloat16, device=dev)
    ws = moe.alloc_workspace(moe.moe_workspace_bytes(T, H, I, E, k), dev)
    fp8 = args.weights == "fp8"
    mx = args.weights == "mxfp8"
    mx_plain_scales = None
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
        gen.manual_seed(args.seed + 1000 + ctx.rank)
        router_bias = torch.randn(E, generator=gen, device=dev) * 0.1
        grouped = moe.grouped_router(8, 4, router_bias, 2.5)

    def forward(events=None):
        if mx:
            moe.moe_forward_mxfp8(x, logits, w13, w13_sf, w2, w2_sf, k, out, ws, stage_events=events,
                                  local_expert_offset=local_offset, router=grouped)
        elif fp8:
            moe.moe_forward_fp8w(x, logits, w13, w13_scale, w2, w2_scale, k, out, ws, stage_events=events)
        elif events is None:
            moe.moe_forward_local(x, logits, w13, w2, k, local_offset, out, ws, flags=args.flags)
        else:
            moe.moe_forward_staged(x, logits, w13, w2, k, out, ws, events, local_expert_offset=local_offset, flags=args.flags)
    flush_buf = torch.zeros(2 * L2_BYTES // 4, dtype=torch.float32, device=dev) if need_flush else None

    def check_status(w=None):
        status = moe.moe_last_status(ws if w is None else w)
        if status != moe.MOE_OK:
            raise RuntimeError(f"{name}: device status {status}: {moe.moe_status_string(status)}")

    # ---- warm-up: W steps at least, and long enough to reach the settled power state ---------------------
    for _ in range(3):
        forward()
    check_status()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(3):
        forward()
    e1.record()
    e1.synchronize()
    est_ms = max(e0.elapsed_time(e1) / 3, 1e-3)
    n_warm = int(min(max(warmup, 3, math.ceil(args.warm_seconds * 1e3 / est_ms)), 5000))
    for _ in range(max(0, n_warm - 6)):
        forward()
    n_warm = max(n_warm, 6)
    if steps is None:
        steps = args.steps if args.few_launches else int(min(max(20, math.ceil(min_timed_s * 1e3 / est_ms)), 2000))

    # ---- device-resident timing ----------------------------------------------------------------
    # The K timed steps run as a user's would: no event between the kernels of a step (an event record between two
    # launches costs several microseconds of launch pipelining).  With an L2 flush between steps each step gets its
    # own pair of events; otherwise one pair brackets all K.
    step_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(steps if need_flush else 1)]
    ctx.barrier()
    sampler = ClockSampler(ctx.local) if ctx.rank == 0 else None
    if not need_flush:
        step_events[0][0].record()
    for s in range(steps):
        if need_flush:
            flush_l2(flush_buf)
            step_events[s][0].record()
        forward()
        if need_flush:
            step_events[s][1].record()
    if not need_flush:
        step_events[0][1].record()
    ctx.barrier()
    total_ms = sum(a.elapsed_time(b) for a, b in step_events)
    # Per-kernel times: the same steps again, instrumented with an event between the stages
    # (at least 0.15 s of it, so that the clock sampler sees the load even when K is small).
    n_staged = min(max(min(steps, 100), int(150.0 * steps / max(total_ms, 1e-3)) + 1), 2000)
    if args.few_launches:
        n_staged = min(steps, 3)
    stage_events = [moe.make_stage_events() for _ in range(n_staged)]
    for s in range(n_staged):
        if need_flush:
            flush_l2(flush_buf)
        forward(stage_events[s])
    ctx.barrier()
    clocks = sampler.stop() if sampler else None
    stage_ms = {nm: statistics.fmean(ev[i].elapsed_time(ev[i + 1]) for ev in stage_events)
                for i, nm in enumerate(moe.STAGE_NAMES)}
    total_ms = max_over_ranks(dist, total_ms, dev)
    check_status()

    # Host time of one call: the calling thread's time over a run of un-synchronised calls (argument checks,
    # tensor-map look-ups, the launches), the queue empty at the start and far from full at the end.
    torch.cuda.synchronize()
    n_host = 1 if args.few_launches else int(min(max(steps, 20), 100))
    host_t0 = time.perf_counter()
    for _ in range(n_host):
        forward()
    host_us = (time.perf_counter() - host_t0) / n_host * 1e6
    torch.cuda.synchronize()

    # The GEMM kernels' own clock probes (block 0's SM cycle counter and the global nanosecond timer at its start
    # and end, left in the status region by the last call): the clock each kernel really ran at.
    probe = ws[128:192].view(torch.int64).cpu().tolist()
    probes = []
    for g in range(2):
        cyc, ns = probe[4 * g + 1] - probe[4 * g], probe[4 * g + 3] - probe[4 * g + 2]
        probes.append(dict(cycles=cyc, ns=ns, sm_mhz=1e3 * cyc / ns) if cyc > 0 and ns > 0 else None)

    views = moe.mx_workspace_views(ws, T, H, I, E, k) if mx else moe.workspace_views(ws, T, H, I, E, k)
    counts = torch.diff(views["expert_offsets"][:n_local + 1]).cpu().numpy()
    rows_scheduled = int(counts.sum())  # = T*k unless only a subset of the experts is resident
    n_active = int((counts > 0).sum())

    # ---- end to end through the host-buffer entry point ---------------------------------------------
    e2e = None
    if with_e2e:
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
        ctx.barrier()
        e2e_ms = 0.0
        if need_flush:
            for _ in range(steps):
                flush_l2(flush_buf)
                e0.record()
                host_step()
                e1.record()
                e1.synchronize()
                e2e_ms += e0.elapsed_time(e1)
        else:
            e0.record()
            for _ in range(steps):
                host_step()
            e1.record()
            e1.synchronize()
            e2e_ms = e0.elapsed_time(e1)
        ctx.barrier()
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
            ctx.barrier()
            e0.record()
            for st, _, _ in lanes:
                st.wait_event(e0)
            for i in range(steps):
                st, o_h, w_s = lanes[i % 2]
                host_step(o_h, w_s, st)
            for st, _, _ in lanes:
                main.wait_stream(st)
            e1.record()
            e1.synchronize()
            e2e_overlapped_ms = max_over_ranks(dist, e0.elapsed_time(e1), dev)
            ctx.barrier()
            same = same and bool(torch.equal(oh_b.view(torch.int16), out.cpu().view(torch.int16)))
            check_status(ws_b)
            del ws_b
        e2e = dict(value=aggregate_tokens_per_s(ctx.world, T, steps, e2e_ms), unit=UNIT,
                   h2d_bytes_per_step=T * H * 2 + T * E * 4, d2h_bytes_per_step=T * H * 2,
                   ms_per_step=e2e_ms / steps, matches_device_path=same,
                   overlapped=None if e2e_overlapped_ms is None else dict(
                       value=aggregate_tokens_per_s(ctx.world, T, steps, e2e_overlapped_ms), unit=UNIT,
                       ms_per_step=e2e_overlapped_ms / steps,
                       how="two streams with their own workspaces alternate, so copies overlap kernels"))

    # ---- roofline of the dominant kernel (gate/up GEMM + SwiGLU), and of the down GEMM beside it ----------
    A = rows_scheduled
    sm_mhz = clocks.get("sm_mhz") if clocks else None
    t_gemm1, t_gemm2 = stage_ms["gemm1_swiglu"] * 1e-3, stage_ms["gemm2"] * 1e-3
    bound = BOUND[name]
    scale = 2.0 if mx else 1.0  # 8-bit operands: the measured bf16 peak times the nominal fp8 / bf16 ratio
    g1_flops, g2_flops = 4.0 * A * H * I, 2.0 * A * H * I
    g1_bytes, g2_bytes = int(n_active * 2 * I * H * bytes_per_weight), int(n_active * I * H * bytes_per_weight)
    g1_tensor = tensor_fractions(g1_flops, t_gemm1, peaks, sm_mhz, scale)
    g2_tensor = tensor_fractions(g2_flops, t_gemm2, peaks, sm_mhz, scale)
    g1_hbm, g2_hbm = hbm_fractions(g1_bytes, t_gemm1, peaks), hbm_fractions(g2_bytes, t_gemm2, peaks)
    traffic = traffic_source = None
    if not (fp8 or mx) and name in NCU_TRAFFIC:
        traffic_source = NCU_TRAFFIC[name]
        traffic = int(traffic_source["bytes"] * traffic_source["scale"])
    if bound == "hbm":
        roofline = dict(bound="hbm", achieved=g1_hbm["achieved"], peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=g1_hbm["frac_measured_copy"], frac_measured_copy=g1_hbm["frac_measured_copy"],
                        frac_nominal=g1_hbm["frac_nominal"], algorithmic_per_launch=g1_bytes)
    else:
        roofline = dict(bound="tensor", achieved=g1_tensor["achieved"], peak=scale * peaks["tflops_sustained"],
                        unit="TFLOP/s", frac=g1_tensor["frac_sustained"], frac_sustained=g1_tensor["frac_sustained"],
                        frac_burst=g1_tensor["frac_burst"], frac_nominal=g1_tensor["frac_nominal"],
                        frac_at_clock=g1_tensor["frac_at_clock"], algorithmic_per_launch=g1_flops)
    def probe_fields(pr, flops):
        if pr is None or mx or fp8:
            return dict(kernel_clock_probe=None)
        return dict(kernel_clock_probe=dict(sm_mhz=round(pr["sm_mhz"], 1), kernel_ms=pr["ns"] * 1e-6,
                                            frac_of_pipe_cycles=flops / (pr["cycles"] * SM_COUNT * TENSOR_FLOP_PER_CLK_SM),
                                            how="block 0's cycle counter and the global timer across the kernel's last launch"))
    roofline.update(probe_fields(probes[0], g1_flops))
    roofline.update(kernel="gate/up GEMM (grouped_gemm_tc*_kernel<swiglu>)", kernel_ms=stage_ms["gemm1_swiglu"],
                    peak_source=f"of {peaks['source']}" + ("" if bound == "hbm" else
                                                           " (sustained: the kernel is timed inside a long step)"),
                    traffic=traffic, traffic_source=traffic_source,
                    down_gemm=dict(kernel="down GEMM (grouped_gemm_tc*_kernel<plain>)", kernel_ms=stage_ms["gemm2"],
                                   **probe_fields(probes[1], g2_flops),
                                   **({"algorithmic_per_launch": g2_bytes, **g2_hbm} if bound == "hbm" else
                                      {"algorithmic_per_launch": g2_flops, **g2_tensor})))
    step_s = total_ms * 1e-3 / steps
    active_weight_bytes = int(n_active * 3 * I * H * bytes_per_weight)
    # per-step latencies: from the timed steps when each has its own events, else from the instrumented pass
    per_step_ms = sorted(a.elapsed_time(b) for a, b in step_events) if need_flush else \
        sorted(ev[0].elapsed_time(ev[-1]) for ev in stage_events)
    tile_bound = int(views["tile_rows"]) if mx else moe.moe_token_tile_rows(T, H, I, E, k, args.flags)
    staged_sum = sum(stage_ms.values())
    non_gemm = stage_ms["route"] + stage_ms["gather"] + stage_ms["combine"]
    layer = dict(stage_ms={n: round(v, 5) for n, v in stage_ms.items()}, n_active_experts=n_active,
                 non_gemm_share_of_stages=non_gemm / staged_sum if staged_sum > 0 else None,
                 latency_ms_median=statistics.median(per_step_ms), latency_ms_min=per_step_ms[0],
                 latency_source="timed steps" if need_flush else "instrumented pass (events between the stages)",
                 stage_ms_source=f"instrumented pass of {n_staged} steps after the timed ones",
                 token_tile_bound=tile_bound,
                 padding_efficiency=rows_scheduled / max(1, computed_rows(counts, tile_bound, even=not mx)),
                 rows_per_expert_min=int(counts.min()), rows_per_expert_max=int(counts.max()),
                 weights=hbm_fractions(active_weight_bytes, step_s, peaks),
                 useful=tensor_fractions(6.0 * A * H * I, step_s, peaks, sm_mhz, scale))

    cpu_baseline = None
    if with_cpu_baseline and ctx.world == 1 and n_local == E and not fp8:
        if mx and mx_plain_scales is not None:
            cpu_baseline = time_oracle_mx(name, x, logits, w13, mx_plain_scales[0], w2, mx_plain_scales[1], k,
                                          args.cpu_seconds)
        elif not mx:
            cpu_baseline = time_oracle(name, inp, budget_s=args.cpu_seconds)

    return dict(value=aggregate_tokens_per_s(ctx.world, T, steps, total_ms), steps=steps, warmup=n_warm,
                ms_per_step=total_ms / steps, host_us_per_call=round(host_us, 2),
                dtype="mxfp8" if mx else "bf16",
                config=dict(workload=name, T=T, H=H, I=I, E=E, top_k=k, resident_experts=n_local,
                            weights="fp8 e4m3 codes + fp32 scale per 128x128 block" if fp8 else
                            "mxfp8: e4m3 codes + e8m0 scale per 32 elements, activations quantised on the fly" if mx else "bf16",
                            router=args.router, parallelism=f"replicas x{ctx.world}",
                            l2="flushed between steps" if need_flush else "weights larger than L2, no flush",
                            seed=args.seed),
                clocks=clocks, e2e=e2e, gpu_launches=moe.moe_forward_launch_count(T) * steps,
                roofline=roofline, layer=layer, cpu_baseline=cpu_baseline)


def measure_gqa(ctx: Ctx, name: str) -> dict:
    """The second workload (paged grouped-query decode attention, gqa_paged_decode): decode steps per second over a
    seeded batch of cached sequences, and the cache bytes streamed per second against the HBM roofline (every cached
    key and value is read once: 2 * Hkv * D * 2 bytes per cached token)."""
    moe, args, dev, peaks = ctx.moe, ctx.args, ctx.dev, ctx.peaks
    cfg = GQA_CONFIGS[name]
    inp = make_gqa_inputs(cfg, seed=args.seed + ctx.rank, device=dev)
    B, Hq, Hkv, D = inp["B"], inp["Hq"], inp["Hkv"], inp["D"]
    max_len = max(inp["kv_len"])
    ws = moe.alloc_workspace(moe.gqa_decode_workspace_bytes(B, Hq, Hkv, D, max_len), dev)
    out = torch.empty((B, Hq, D), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, Hq), dtype=torch.float32, device=dev)
    kv_bytes = sum(inp["kv_len"]) * 2 * Hkv * D * 2
    need_flush = kv_bytes < 2 * L2_BYTES
    flush_buf = torch.zeros(2 * L2_BYTES // 4, dtype=torch.float32, device=dev) if need_flush else None

    def step():
        moe.gqa_paged_decode(inp["q"], inp["k_cache"], inp["v_cache"], inp["kv_indptr"], inp["kv_indices"],
                             inp["kv_last_page_len"], max_len, inp["sm_scale"], out, ws, lse=lse)
    for _ in range(3):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); step(); e1.record(); e1.synchronize()
    est_ms = max(e0.elapsed_time(e1), 1e-3)
    steps = args.steps if args.few_launches else int(min(max(20, math.ceil(300.0 / est_ms)), 2000))
    for _ in range(3 if args.few_launches else min(steps, 200)):
        step()
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps if need_flush else 1)]
    ctx.barrier()
    sampler = ClockSampler(ctx.local) if ctx.rank == 0 else None
    if not need_flush:
        pairs[0][0].record()
    for s_ in range(steps):
        if need_flush:
            flush_l2(flush_buf)
            pairs[s_][0].record()
        step()
        if need_flush:
            pairs[s_][1].record()
    if not need_flush:
        pairs[0][1].record()
    ctx.barrier()
    clocks = sampler.stop() if sampler else None
    ms = max_over_ranks(ctx.dist, sum(a.elapsed_time(b) for a, b in pairs), dev) / steps
    cpu = None
    if not args.no_cpu_baseline and not args.few_launches and ctx.world == 1 and sum(inp["kv_len"]) * Hq <= 25_000_000:
        from oracle import gqa_oracle
        o = gqa_oracle.get("f64")
        host = [bf16_bits(inp[n]) for n in ("q", "k_cache", "v_cache")] + [inp[n].cpu().numpy() for n in
                                                                            ("kv_indptr", "kv_indices", "kv_last_page_len")]
        t0 = time.perf_counter()
        o.paged_decode(*host, inp["sm_scale"])
        wall = time.perf_counter() - t0
        cpu = dict(value=B / wall, unit="decode tokens/s", cores=o.num_threads, kind="oracle",
                   sample=f"the whole batch of '{name}' once, double-precision oracle, {wall:.2f} s wall")
    return dict(metric="gqa_paged_decode_tokens_per_s", value=ctx.world * B / (ms * 1e-3), unit="decode tokens/s",
                ms_per_step=ms, steps=steps, gpu_launches=steps,
                config=dict(workload=name, **{k_: cfg[k_] for k_ in ("B", "Hq", "Hkv", "D", "page_size")},
                            cached_tokens=sum(inp["kv_len"]), kv_len_min=min(inp["kv_len"]), kv_len_max=max_len,
                            split_tokens=moe.gqa_decode_split_tokens(B, Hq, Hkv, D, max_len),
                            l2="flushed between steps" if need_flush else "cache larger than L2, no flush"),
                roofline=dict(bound="hbm", kernel="gqa_paged_decode_kernel", algorithmic_per_launch=kv_bytes, peak=peaks["hbm_gbs"],
                              frac=kv_bytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], peak_source=f"of {peaks['source']}",
                              traffic=None, **hbm_fractions(kv_bytes, ms * 1e-3, peaks)),
                clocks=clocks, cpu_baseline=cpu, dtype="bf16")


def sweep_entry(r: dict) -> dict:
    """What the line keeps of a sweep workload."""
    return dict(ms_per_step=r["ms_per_step"], value=r["value"], unit=UNIT, steps=r["steps"], warmup=r["warmup"],
                host_us_per_call=r["host_us_per_call"], n_active_experts=r["layer"]["n_active_experts"],
                roofline=r["roofline"], stage_ms=r["layer"]["stage_ms"], latency_ms_min=r["layer"]["latency_ms_min"],
                weights=r["layer"]["weights"], useful=r["layer"]["useful"], clocks=r["clocks"], config=r["config"])


def run_ours(args):
    import paper_2602_19128_b200 as moe
    dist, rank, world, local = dist_setup(args.gpus)
    ctx = Ctx(moe, dist, rank, world, local, args)
    headline = args.config or HEADLINE
    do_sweep = (args.config is None or args.sweep) and world == 1 and args.weights == "bf16" and args.router == "softmax"
    sweep, shared = {}, None
    if do_sweep:
        for name in SWEEP:
            if name == headline:
                continue
            try:
                weights = None
                if name == "dsv3_decode" and headline == "dsv3_prefill":  # one model, two batch sizes: one draw of its weights
                    shared = make_inputs(CONFIGS[headline], seed=args.seed + rank, device=ctx.dev)
                    weights = (shared["w13"], shared["w2"])
                inp = make_inputs(CONFIGS[name], seed=args.seed + rank, device=ctx.dev, weights=weights)
                r = measure(ctx, name, inp, steps=None, warmup=args.warmup, with_e2e=False, with_cpu_baseline=False,
                            min_timed_s=args.sweep_seconds)
                sweep[name] = sweep_entry(r)
                if weights is not None:
                    sweep[name]["config"]["weights"] = "bf16 (the experts' weights are drawn once, for dsv3_prefill, and shared)"
                del inp, r
            except Exception as exc:  # the headline still has to be printed
                sweep[name] = dict(error=f"{type(exc).__name__}: {exc}")
            torch.cuda.empty_cache()
    second = None
    if do_sweep or args.gqa:  # the second workload of the paper (Sec. 4.6), reported beside the layer, never as the headline
        second = {}
        for name in ("gqa_decode_b64", "gqa_decode_b256", "gqa_decode_b1_long", "gqa_decode_b64_16k"):
            try:
                second[name] = measure_gqa(ctx, name)
            except Exception as exc:
                second[name] = dict(error=f"{type(exc).__name__}: {exc}")
            torch.cuda.empty_cache()
    inp = shared if shared is not None else make_inputs(CONFIGS[headline], seed=args.seed + rank, device=ctx.dev)
    r = measure(ctx, headline, inp, steps=args.steps, warmup=args.warmup, with_e2e=not args.few_launches,
                with_cpu_baseline=not args.no_cpu_baseline and not args.few_launches)
    if rank == 0:
        line = dict(metric=METRIC, value=r["value"], unit=UNIT, n_gpus=world, steps=r["steps"], warmup=r["warmup"],
                    ms_per_step=r["ms_per_step"], higher_is_better=True, scaling="weak", vs_baseline=None, dtype=r["dtype"],
                    data="synthetic", config=r["config"], clocks=r["clocks"], e2e=r["e2e"], gpu_launches=r["gpu_launches"],
                    host_us_per_call=r["host_us_per_call"], roofline=r["roofline"], layer=r["layer"],
                    cpu_baseline=r["cpu_baseline"], sweep=sweep if do_sweep else None, second_workload=second)
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", choices=list(CONFIGS), default=None,
                    help=f"measure this workload alone (default: headline {HEADLINE} plus a sweep of the other four)")
    ap.add_argument("--sweep", action="store_true", help="with --config: also run the sweep of the other workloads")
    ap.add_argument("--gqa", action="store_true", help="with --config: also measure the paged grouped-query decode workloads")
    ap.add_argument("--shape", default=None, help="custom T,H,I,E,top_k instead of a named workload (profiling)")
    ap.add_argument("--bound", choices=["hbm", "tensor"], default="hbm", help="with --shape: which roofline to report against")
    ap.add_argument("--weights", choices=["bf16", "fp8", "mxfp8"], default="bf16",
                    help="fp8: expert weights as E4M3 codes with one fp32 scale per 128 x 128 block (moe_forward_fp8w); "
                         "mxfp8: weights and activations in MX FP8 on the block-scaled MMA (moe_forward_mxfp8)")
    ap.add_argument("--router", choices=["softmax", "grouped"], default="softmax",
                    help="grouped: sigmoid scores, selection bias, 8 groups of which 4 eligible, weights x 2.5 (with --weights mxfp8)")
    ap.add_argument("--flags", type=int, default=0, help="MOE_FLAG_* bits for the device-resident bf16 steps (A/B timing)")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--warm-seconds", type=float, default=1.0,
                    help="warm-up lasts at least this long (and at least --warmup steps): the settled power state")
    ap.add_argument("--sweep-seconds", type=float, default=0.5, help="timed region of each sweep workload")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-oracle baseline leg")
    ap.add_argument("--few-launches", action="store_true",
                    help="for runs under a profiler: six warm-up steps, the K timed steps, at most three instrumented "
                         "ones, no end-to-end or host-time loops (the numbers of such a run are not benchmark values)")
    ap.add_argument("--watchdog-seconds", type=float, default=1200.0,
                    help="dump every thread's Python stack to stderr and exit(1) if the run is not over by then")
    args = ap.parse_args()
    if args.watchdog_seconds > 0:  # a stuck run ends by itself, with evidence of where it was
        faulthandler.dump_traceback_later(args.watchdog_seconds, exit=True)
    if args.few_launches:
        args.warm_seconds = 0.0
    if args.shape:
        T, H, I, E, k = (int(v) for v in args.shape.split(","))
        args.config = f"custom_{T}x{H}x{I}x{E}x{k}"
        CONFIGS[args.config] = dict(T=T, H=H, I=I, E=E, top_k=k, skew=False)
        BOUND[args.config] = args.bound
    if args.impl == "reference":
        if (args.config or HEADLINE) in LOCAL_CONFIGS:
            raise SystemExit("the reference arm covers the five whole-layer workloads")
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
