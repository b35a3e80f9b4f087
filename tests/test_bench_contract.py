"""The reference arm of bench.py (the CPU oracle timed on a bounded sample) runs without a GPU: its JSON line must
carry the keys the benchmark contract names.  The arm of the CUDA path is covered on the GPU (test below)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True, cwd=ROOT,
                         timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                   # exactly one JSON line
    return json.loads(lines[0])


def test_reference_arm_json_line():
    d = _run("--impl", "reference", "--steps", "1", "--warmup", "1")
    assert d["impl"] == "reference" and d["metric"] == "sc_gemm_stream_bitops_per_s" and d["unit"] == "bitop/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["n_gpus"] == 1 and d["steps"] == 1
    assert d["value"] > 0 and d["ms_per_step"] > 0
    assert d["config"]["workload"] == "vit_b16_fc1" and "sample" in d["config"]
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


@pytest.mark.gpu
def test_cuda_arm_json_line():
    d = _run("--steps", "3", "--warmup", "3", "--no-cpu-baseline", "--no-configs")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline"):
        assert key in d, key
    assert d["config"]["workload"] == "vit_b16_fc1" and d["gpu_launches"] > 0 and d["value"] > 1e14
    assert d["e2e"]["h2d_bytes_per_step"] > 0 and d["e2e"]["d2h_bytes_per_step"] > 0 and 0 < d["e2e"]["value"] <= d["value"] * 1.05
    r = d["roofline"]
    assert r["bound"] == "tensor" and 0.3 < r["frac"] < 1.1 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    # both denominators are reported; `peak` is the larger one, so `frac` is the smaller fraction
    assert r["frac"] <= min(r["frac_vs_bf16_x4"], r["frac_vs_issue_rate"]) + 1e-12
    assert abs(r["frac_vs_issue_rate"] - r["achieved"] / r["peak_issue_rate"]) < 1e-9
    assert 8000 < r["mxf4_mac_per_clk_per_sm"] < 17000
    assert d["clocks"]["sm_max_mhz"] >= d["clocks"]["sm_mhz"] > 0
