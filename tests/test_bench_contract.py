"""The one JSON line bench.py prints: keys and types the benchmark contract names.

The reference arm (the oracle timed on the host cores) runs anywhere; the device arm needs a GPU."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
COMMON = {"metric": str, "value": float, "unit": str, "n_gpus": int, "steps": int, "warmup": int,
          "ms_per_step": float, "higher_is_better": bool, "scaling": str, "dtype": str, "data": str, "config": dict,
          "e2e": dict, "cpu_baseline": dict}


def _run(*args):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT, capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, "bench.py must print exactly one line"
    return json.loads(lines[0])


def _check_common(d):
    for key, typ in COMMON.items():
        assert key in d, key
        assert isinstance(d[key], typ), (key, type(d[key]))
    assert "vs_baseline" in d and d["vs_baseline"] is None  # the paper has no number for this machine
    assert d["metric"] == "causal_attn_fwd_bwd_tflops" and d["unit"] == "TFLOP/s"
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["data"] == "synthetic"
    assert d["config"]["workload"] == "gpt2_small" and "model" not in d["config"]
    assert d["value"] > 0 and d["ms_per_step"] > 0
    for key in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step"):
        assert key in d["e2e"], key
    for key in ("value", "unit", "cores", "kind", "sample"):
        assert key in d["cpu_baseline"], key
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1


def test_reference_arm_line():
    d = _run("--impl", "reference", "--steps", "1", "--warmup", "0")
    _check_common(d)
    assert d["impl"] == "reference" and d["dtype"] == "f64" and d["n_gpus"] == 1 and d["steps"] == 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
    assert d["e2e"]["value"] == d["value"] == d["cpu_baseline"]["value"]


@pytest.mark.gpu
@pytest.mark.parametrize("launch", ["graph", "eager"])
def test_device_arm_line(launch):
    d = _run("--steps", "6", "--warmup", "3", "--launch", launch)
    _check_common(d)
    assert "impl" not in d or d["impl"] != "reference"
    assert d["dtype"] == "bf16" and d["n_gpus"] == 1 and d["steps"] == 6 and d["warmup"] >= 3
    assert d["gpu_launches"] == 5 * 6
    assert launch in d["config"]["launch"] and "l2" in d["config"]
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and 0.05 < r["frac"] < 1.2
    assert "burst" in r["peak_source"] and r["peak_sustained"] <= r["peak"]
    assert r["traffic"] is None or (r["traffic"] > 0 and r["traffic_source"].startswith("profiles/"))
    # the two fractions the targets are stated on: the forward, and the whole backward timed as one sequence
    t = r["targets"]
    assert t["fwd"]["target"] == 0.50 and t["bwd"]["target"] == 0.35
    for leg in ("fwd", "bwd"):
        assert t[leg]["ms"] > 0 and abs(t[leg]["frac"] - t[leg]["tflops"] / r["peak"]) < 1e-9
    k = r["kernel_ms"]
    assert t["bwd"]["ms"] > k["bwd_main"] * 0.9   # the sequence contains the main kernel
    assert set(r["kernel_ms_eager"]) == set(k) and "graph" in r["attribution"]
    assert all(k[n] <= r["kernel_ms_eager"][n] * 1.1 for n in k)   # back to back is never slower than with host gaps
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == e["d2h_bytes_per_step"] == 4 * 8 * 12 * 1024 * 64 * 2
    assert 0 < e["value"] < d["value"]  # the copies are inside the timed region
    c = d["clocks"]
    assert c["sm_mhz"] > 0 and c["sm_max_mhz"] >= c["sm_mhz"] and isinstance(c["reasons"], list)
