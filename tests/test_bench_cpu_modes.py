"""bench.py's CPU-only modes run without a GPU: the reference arm (the oracle timed on the C2
workload) and the per-configuration oracle suite."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_cpu_suite_prints_one_line_per_configuration_and_thread_count():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--cpu-suite", "--cpu-seconds", "0.1"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    rows = [json.loads(l) for l in out.stdout.splitlines() if l.startswith("{")]
    assert {r["cfg"] for r in rows} == {"C1", "C2", "C3", "C4", "C5"}
    assert all(r["impl"] == "cpu-oracle" and r["us"] > 0 and r["eff_gbs"] > 0 for r in rows)
    assert 1 in {r["threads"] for r in rows}


def test_reference_arm_prints_the_contract_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "1"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    r = json.loads(lines[0])
    assert r["impl"] == "reference" and r["metric"] == "effective collective GB/s" and r["unit"] == "GB/s"
    assert r["higher_is_better"] is True and r["n_gpus"] == 1 and r["steps"] == 1 and r["warmup"] == 1
    assert r["value"] > 0 and r["ms_per_step"] > 0 and r["vs_baseline"] is None
    assert r["cpu_baseline"]["kind"] == "oracle" and r["cpu_baseline"]["cores"] >= 1 and r["cpu_baseline"]["value"] == r["value"]
    assert r["e2e"] == {"value": r["value"], "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert "workload" in r["config"]
