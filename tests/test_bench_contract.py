"""The benchmark's one-line JSON contract: the reference arm (CPU oracle) here, the CUDA arm on a GPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
             "dtype", "data", "config", "cpu_baseline", "e2e", "gpu_launches"}


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, lines                      # exactly one JSON line on stdout
    return json.loads(lines[0])


def test_reference_arm_prints_the_contract_line():
    d = _run("--impl", "reference", "--workload", "tiny", "--steps", "2", "--warmup", "1")
    assert BASE_KEYS <= set(d) and d["impl"] == "reference"
    assert d["metric_key"] == "us_per_draft_attention_step" and d["unit"] == "us" and d["higher_is_better"] is False
    baseline = os.path.join(ROOT, "BASELINE.json")
    if os.path.exists(baseline):                       # the line names the metric as the benchmark description does
        assert d["metric"] == json.load(open(baseline))["metric"]
    assert d["value"] > 0 and d["steps"] == 2 and d["warmup"] == 1 and d["vs_baseline"] is None
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "us", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["gpu_launches"] == 0 and "workload" in d["config"]


@pytest.mark.gpu
@pytest.mark.parametrize("extra", [[], ["--kv-dtype", "fp8"]])
def test_cuda_arm_prints_the_contract_line(extra):
    d = _run("--workload", "tiny", "--steps", "3", "--warmup", "3", "--no-cpu-baseline", *extra)
    assert BASE_KEYS | {"roofline", "clocks", "variants"} <= set(d) and "impl" not in d
    assert d["value"] > 0 and d["n_gpus"] == 1 and d["scaling"] == "weak" and d["data"] == "synthetic"
    gamma = d["config"]["draft_steps_per_pass"] // 2
    assert d["gpu_launches"] == 3 * 2 * gamma                      # one kernel per draft step, nothing else in the timed region
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    assert {"windowed", "full", "draft_extend"} <= set(d["variants"])
