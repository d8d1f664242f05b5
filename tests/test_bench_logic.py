"""CPU checks of bench.py's host logic, including the multi-rank aggregation on two gloo ranks."""
import json
import os
import subprocess
import sys
from pathlib import Path

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))
import bench  # noqa: E402


def _rank_main(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(dist, 10.0 + 5.0 * rank, "cpu")      # rank 1 is the slow one
    dist.barrier()
    Path(out_dir, f"rank{rank}.json").write_text(json.dumps(dict(ms=ms)))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_on_two_gloo_ranks(tmp_path):
    world, port = 2, 29000 + os.getpid() % 2000
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [json.loads((tmp_path / f"rank{r}.json").read_text())["ms"] for r in range(world)]
    assert got == [15.0, 15.0]                                      # every rank sees the slowest time
    # replicas: N ranks x T tokens x K steps over the slowest rank's time
    assert bench.aggregate_tokens_per_s(2, 512, 10, 15.0) == 2 * 512 * 10 / 0.015
    assert bench.max_over_ranks(None, 3.5, "cpu") == 3.5


def test_peaks_fall_back_when_the_measured_file_is_absent(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", tmp_path)
    p = bench.load_peaks()
    assert p["source"] == "fallback" and p["hbm_gbs"] == 6650.0
    (tmp_path / "MEASURED_PEAKS.json").write_text(json.dumps(dict(hbm_gbs=6544.3, bf16_tflops=1644.9,
                                                                  bf16_tflops_sustained=1350.0)))
    p = bench.load_peaks()
    assert p["source"] == "measured" and p["tflops_sustained"] == 1350.0


def test_reference_arm_runs_on_rank_zero_only_and_prints_one_json_line():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--config", "tiny", "--steps", "2",
                        "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="1", CUDA_VISIBLE_DEVICES="")
    r = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--config", "tiny", "--steps", "2",
                        "--warmup", "1"], capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == bench.METRIC and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_every_workload_has_a_roofline_bound():
    assert set(bench.BOUND) >= set(bench.CONFIGS)


def test_headline_is_the_largest_workload_and_the_sweep_covers_the_other_four():
    weights = {n: 3 * c["H"] * c["I"] * c["E"] for n, c in bench.CONFIGS.items() if n not in bench.LOCAL_CONFIGS}
    flops = {n: 6 * c["T"] * c["top_k"] * c["H"] * c["I"] for n, c in bench.CONFIGS.items() if n not in bench.LOCAL_CONFIGS}
    assert bench.HEADLINE == max(flops, key=flops.get) and weights[bench.HEADLINE] == max(weights.values())
    assert set(bench.SWEEP) | {bench.HEADLINE} == set(weights)


def test_fraction_at_clock_and_the_three_tensor_denominators():
    peaks = dict(hbm_gbs=6544.3, tflops_burst=1644.9, tflops_sustained=1350.0, source="measured")
    # a kernel that does exactly what 148 SMs x 8192 flop/clk deliver in 1 ms at 1000 MHz
    flops = 148 * 8192 * 1000e6 * 1e-3
    assert abs(bench.fraction_at_clock(flops, 1e-3, 1000.0) - 1.0) < 1e-12
    assert bench.fraction_at_clock(flops, 1e-3, None) is None
    f = bench.tensor_fractions(flops, 1e-3, peaks, 1000.0)
    assert abs(f["achieved"] - 1212.416) < 1e-3 and abs(f["frac_sustained"] - 1212.416 / 1350.0) < 1e-9
    assert abs(f["frac_burst"] - 1212.416 / 1644.9) < 1e-9 and abs(f["frac_nominal"] - 1212.416 / 2250.0) < 1e-9
    h = bench.hbm_fractions(8e9, 1e-3, peaks)
    assert abs(h["frac_nominal"] - 1.0) < 1e-12 and abs(h["frac_measured_copy"] - 8000 / 6544.3) < 1e-9


def test_recorded_ncu_traffic_names_its_kernel_instance_and_commit():
    for entry in bench.NCU_TRAFFIC.values():
        assert entry["kernel"] and entry["commit"] and entry["source"].startswith("profiles/") and entry["scale"] >= 1
        assert (ROOT / entry["source"]).exists()
