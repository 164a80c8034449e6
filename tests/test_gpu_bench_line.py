"""The benchmark's JSON line carries what its readers expect (a short run on the GPU)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT, capture_output=True,
                         text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, out.stdout[-2000:]
    return json.loads(lines[0])


def test_decode_line_has_the_contract_keys():
    d = run_bench("--steps", "3", "--warmup", "3", "--layers", "4", "--no-others")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "clocks", "gpu_launches"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["config"]["workload"] == "llama2-7b" and "model" not in d["config"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and 0.0 < r["frac"] < 1.5
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert abs(r["achieved"] - r["bytes_per_launch"] / (r["us_per_launch"] * 1e-6) / 1e9) < 1e-6 * r["achieved"]
    assert r["attention_only"]["frac"] >= r["frac"] * 0.9
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["sample"]
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["value"] < d["value"]
    assert d["gpu_launches"] >= 3 * 4
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])


def test_prefill_line():
    d = run_bench("--prefill", "--steps", "3", "--layers", "2")
    assert d["metric"] == "prefill_sdpa_causal_tflops" and d["value"] > 0
    assert d["roofline"]["bound"] == "tensor" and 0.0 < d["roofline"]["frac"] < 1.2
    assert 0 < d["ms_fused_store_and_attention"] < d["ms_store_then_attention"] * 1.2
