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
