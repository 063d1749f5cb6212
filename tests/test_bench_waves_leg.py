"""bench.py's host-only leg for the wave planner runs here without a GPU and prints one well-formed JSON line."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_waves_leg_prints_one_json_line_and_agrees_with_the_oracle():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--waves", "--warmup", "0"], cwd=ROOT,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["unit"] == "decisions/s" and j["value"] > 0 and j["gpu_launches"] == 0
    assert j["config"]["decisions_identical_to_oracle"] is True and len(j["config"]["budgets_used"]) >= 2
    assert j["cpu_baseline"]["kind"] == "oracle" and j["cpu_baseline"]["value"] > 0
