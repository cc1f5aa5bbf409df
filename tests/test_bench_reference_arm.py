"""The benchmark's reference arm (`bench.py --impl reference`: the CPU oracle on a bounded row slab) runs without a
GPU; this checks its one-line JSON contract on the small configuration, and that a non-zero rank stays silent."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run(extra, env=None):
    e = dict(os.environ)
    e.update(env or {})
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1",
                          "--steps", "2", "--warmup", "3"] + extra, capture_output=True, text=True, env=e, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    return out.stdout.strip().splitlines()


def test_reference_arm_prints_one_json_line_with_the_contract_keys():
    lines = run([])
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"].startswith("join pair-TOPS") and d["unit"] == "TOPS"
    assert d["higher_is_better"] is True and d["steps"] == 2 and d["warmup"] == 3 and d["n_gpus"] == 1
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["gpu_launches"] == 0 and d["vs_baseline"] is None
    assert d["config"]["workload"].startswith("cfg1") and d["config"]["kind"] == "ip"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"] and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"] == {"value": d["value"], "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


def test_reference_arm_kind_override_and_silent_ranks():
    d = json.loads(run(["--kind", "cos", "--threshold", "0.6"])[0])
    assert d["config"]["kind"] == "cos" and d["config"]["threshold"] == 0.6
    assert run([], env={"RANK": "1", "WORLD_SIZE": "2", "LOCAL_RANK": "1"}) == []


def test_roofline_arithmetic_of_the_bench_line():
    """The fractions in the bench line are plain ratios of the kernel's rate: check them on made-up numbers."""
    import bench
    from paper_2006_12608_b200 import workloads as W
    w = W.make_workload(4, n=1024, m=2048, planted=0)
    peaks = {"hbm_gbs": 6000.0, "bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "source": "test"}
    ops = 2 * 1024 * 2048 * 128
    r = bench.roofline_of(w, kernel_ms=1.0, region_ms=1000.0, clocks={"sm_mhz": 1500.0}, peaks=peaks,
                          int8_peak={"burst_tops": 3000.0, "sustained_tops": 2500.0})
    achieved = ops / 1e-3 / 1e12
    assert abs(r["achieved"] - achieved) < 1e-12 and r["peak"] == 2800.0 and abs(r["frac"] - achieved / 2800.0) < 1e-15
    assert abs(r["frac_of_nominal"] - achieved / 4500.0) < 1e-15
    assert abs(r["frac_of_clock_ceiling"] - achieved / (148 * 8192 * 2 * 1.5e9 / 1e12)) < 1e-15
    assert abs(r["frac_of_int8_library_peak"] - achieved / 2500.0) < 1e-15
    assert r["traffic"] is None and r["traffic_source"] is None            # not the captured size
    burst = bench.roofline_of(w, 1.0, 100.0, {"sm_mhz": None}, peaks)
    assert burst["peak"] == 3200.0 and "frac_of_clock_ceiling" not in burst and "frac_of_int8_library_peak" not in burst
    assert bench.jl_level_dims(1024, 64) == [1024, 512, 512, 384, 64]
