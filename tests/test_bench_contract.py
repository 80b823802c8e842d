"""bench.py prints one JSON line with the agreed keys (small workload, few steps)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + list(extra),
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, out.stdout
    return json.loads(lines[0])


@pytest.mark.gpu
def test_gpu_arm_prints_the_contract_keys():
    d = _run("--config", "cfg1", "--steps", "5", "--warmup", "3", "--no-per-config", "--cpu-seconds", "0.5")
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
              "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert k in d, k
    assert d["metric"] == "draft positions verified/s" and d["n_gpus"] == 1 and d["steps"] == 5
    assert d["value"] > 0 and d["vs_baseline"] is None and d["config"]["workload"] == "cfg1"
    assert d["e2e"]["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] > 16_000_000 and d["e2e"]["d2h_bytes_per_step"] == 64
    assert d["e2e"]["value"] < d["value"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert d["gpu_launches"] == 2 * 5 and d["config"]["workload"] == "cfg1"
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0


def test_reference_arm_times_the_oracle_on_the_host():
    d = _run("--impl", "reference", "--config", "cfg0", "--steps", "2", "--warmup", "1")
    assert d["impl"] == "reference" and d["metric"] == "draft positions verified/s"
    assert d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
