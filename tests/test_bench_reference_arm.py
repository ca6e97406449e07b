"""`bench.py --impl reference` on CPU: the oracle-timed arm must print one JSON line with the
contract's keys, for the same metric and workload naming as the GPU arm (no GPU needed)."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(extra):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "1", "--steps", "1",
           "--warmup", "1", "--cpu-budget", "2"] + extra
    out = subprocess.run(cmd, capture_output=True, text=True, timeout=300, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    return json.loads(lines[0])


def test_reference_arm_prints_one_contract_line():
    d = _run([])
    assert d["impl"] == "reference" and d["metric"] == "worker_gradients_per_sec"
    assert d["unit"] == "worker-gradients/s" and d["higher_is_better"] is True
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] and "rounds" in d["cpu_baseline"]["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["config"]["workload"].startswith("lsq64_w8") and d["vs_baseline"] is None and d["gpu_launches"] == 0


def test_reference_arm_with_local_steps():
    d = _run(["--local-steps", "3"])
    assert "U=3 local steps" in d["config"]["workload"] and d["value"] > 0
