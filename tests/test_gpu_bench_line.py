"""`bench.py` on the GPU with a handful of steps: one JSON line carrying every key of the measurement contract, with
values that hang together (the throughput is the step's FLOPs over its time, the roofline fraction is achieved over
peak, the launches are the library's count times the steps)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_default_line_has_the_contract_keys():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "6", "--warmup", "3", "--oracle-tokens", "32",
                          "--no-tensor-ceiling"], capture_output=True, text=True, cwd=ROOT, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 6 and d["warmup"] == 3 and d["higher_is_better"] is True
    assert d["scaling"] == "weak" and d["vs_baseline"] is None and d["dtype"] == "fp8" and d["data"] == "synthetic"
    assert d["config"]["workload"].startswith("configs[1]") and "model" not in d["config"] and "l2" in d["config"]
    flops = d["config"]["gflop_per_step"] * 1e9
    assert abs(d["value"] - flops / (d["ms_per_step"] * 1e-3) / 1e12) < 1e-6 * d["value"]
    assert 500 < d["value"] < 4500
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["traffic"] is None or r["traffic"] > 1e6
    e = d["e2e"]
    assert e["unit"] == d["unit"] and 0 < e["value"] < d["value"] and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert d["gpu_launches"] == 30 * d["steps"]                      # 7 x (2 + 2) kernels + one batched proxy update of 2
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and "sample" in c
    assert set(("sm_mhz", "sm_max_mhz", "reasons")) <= set(d["clocks"])
    # both regimes are on the line, each with its own clock record; the headline steps follow a soak of the same loop
    assert d["clocks"]["samples"] >= 1 and d["clocks"]["soak_before"]["samples"] >= 20 and d["clocks"]["soak_before"]["seconds"] >= 2.0
    b = d["burst"]
    assert b["steps"] == 20 and abs(b["value"] - flops / (b["ms_per_step"] * 1e-3) / 1e12) < 1e-6 * b["value"] and "clocks" in b
    assert b["ms_per_step"] <= d["ms_per_step"] * 1.05          # a cold board is not slower than one at its power cap
    # the HBM-bound stages: achieved = stated bytes / stated time, fraction of the measured copy rate
    assert d["db"]["frac"] is None and "rider" in d["db"]["kernel"]      # no launch of its own on the default path ...
    own = d["db"]["as_a_kernel_of_its_own"]                              # ... and, for reference, timed as one
    assert 0 < own["frac"] < 1.2 and own["ms_per_step"] > 0 and own["gemm_dx_ms_per_step_with_rider"] > 0
    for key in ("quantize", "proxy_update"):
        q = d[key]
        assert abs(q["achieved_gbs"] - q["bytes_per_step"] / (q["ms_per_step"] * 1e-3) / 1e9) < 1e-6 * q["achieved_gbs"]
        assert abs(q["frac"] - q["achieved_gbs"] / q["peak_gbs"]) < 1e-9 and 0 < q["frac"] < 1.2
    assert d["quantize"]["bytes_per_elt"] == 3               # every tensor of configs[1] fits L2: one DRAM read, one write
    assert "sustained" in r["regime"] and "instrumented_pass" in d and d["instrumented_pass"]["clocks"]["samples"] >= 1
    ps = d["per_step"]            # single steps right after the timed region: the same regime, so the same time
    assert ps["n"] >= 20 and ps["min_ms"] <= ps["median_ms"] <= ps["max_ms"] and abs(ps["median_ms"] - d["ms_per_step"]) < 0.1 * d["ms_per_step"]
    assert d["device_status"] == 0
