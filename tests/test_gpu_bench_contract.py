"""bench.py's own arm on the GPU, at a reduced size so the test stays short: one JSON line
with the keys of the benchmark contract, a roofline object, an end-to-end figure measured
through host buffers, a clock record and a launch count."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--size", "2048",
                          "--steps", "5", "--warmup", "3", "--e2e-steps", "2", "--sustain-seconds", "0.5"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config",
                "roofline", "cpu_baseline", "clocks", "e2e", "gpu_launches", "precisions"):
        assert key in d, key
    assert d["steps"] == 5 and d["warmup"] == 3 and d["n_gpus"] == 1 and d["scaling"] == "weak"
    assert d["value"] > 0 and d["dtype"] == "f16" and d["data"] == "synthetic"
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    # the denominator follows the length of the timed region: a few milliseconds here
    assert r["timed_region_s"] < 1.0 and r["peak"] == r["peak_burst"] and r["frac"] == r["frac_burst"]
    assert r["frac_sustained"] is not None and r["peak_sustained"] > 0
    assert r["traffic"] is None and r["algorithmic_bytes"] == 2 * 2048 * 2048 * 2 + 4 * 2048 * 2048
    for p in ("fp16", "s8", "s4"):
        sus = d["precisions"][p]["sustained"]
        assert sus["seconds"] >= 0.5 and sus["value"] > 0 and sus["launches"] >= 5
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] == 2 * 2048 * 2048 * 2
    assert e["d2h_bytes_per_step"] == 2048 * 2048 * 4 and e["value"] < d["value"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] > 0
    assert d["clocks"]["sm_max_mhz"] >= d["clocks"]["sm_mhz"] > 0
    # FP16 + INT8 + INT4 per step; INT4 is one fused launch at this size
    assert d["gpu_launches"] == 5 * 3
    assert set(d["precisions"]) == {"fp16", "s8", "s4"}
