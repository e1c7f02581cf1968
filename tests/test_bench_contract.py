"""The one JSON line `bench.py` prints: keys and types of both arms, on the tiny workload so that it takes seconds.

The CPU test runs the reference arm (the oracle on the host cores); the GPU test runs the product arm through the
C ABI and checks the keys a reader of the line relies on (roofline, cpu_baseline, e2e, clocks, launch count)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

BASE_KEYS = {"metric": str, "value": float, "unit": str, "n_gpus": int, "steps": int, "warmup": int,
             "ms_per_step": float, "higher_is_better": bool, "scaling": str, "dtype": str, "data": str, "config": dict}


def _run(args, timeout):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, capture_output=True,
                         text=True, timeout=timeout)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, "exactly one JSON line expected, got %d" % len(lines)
    return json.loads(lines[0])


def _check_base(d, steps, warmup):
    for k, t in BASE_KEYS.items():
        assert k in d, k
        assert isinstance(d[k], t) or (t is float and isinstance(d[k], int)), (k, type(d[k]))
    assert "vs_baseline" in d and d["vs_baseline"] is None          # no published number for this metric and workload
    assert d["steps"] == steps and d["warmup"] == warmup and d["n_gpus"] == 1
    assert d["value"] > 0 and d["ms_per_step"] > 0
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["data"] == "synthetic"
    assert d["config"]["workload"].startswith("c1_tiny")
    assert "model" not in d["config"]


def test_reference_arm_line():
    d = _run(["--impl", "reference", "--workload", "c1", "--steps", "2", "--warmup", "1"], 300)
    _check_base(d, 2, 1)
    assert d["impl"] == "reference" and d["dtype"] == "f64"
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and isinstance(cb["sample"], str) and cb["value"] == d["value"]
    e = d["e2e"]
    assert e["value"] == d["value"] and e["unit"] == d["unit"]
    assert e["h2d_bytes_per_step"] == 0 and e["d2h_bytes_per_step"] == 0


@pytest.mark.gpu
def test_product_arm_line():
    d = _run(["--workload", "c1", "--steps", "3", "--warmup", "3", "--e2e-steps", "1"], 600)
    _check_base(d, 3, 3)
    assert "impl" not in d or d["impl"] == "ours"
    assert d["dtype"] == "bf16" and d["unit"] == "GB/s"
    r = d["roofline"]
    for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "kernel"):
        assert k in r, k
    assert r["bound"] in ("hbm", "tensor", "alu") and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    for name in ("score", "select", "pack", "decode"):
        assert name in d["rooflines"], name
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] > 0 and isinstance(cb["sample"], str)
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] < d["value"]                  # host buffers and copies inside the timed region
    assert d["gpu_launches"] > 0
    c = d["clocks"]
    assert c["sm_max_mhz"] > 0 and isinstance(c["reasons"], list)
    assert d["dev_status"] == 0
    for k in ("h2d", "score", "select_pack", "d2h", "decode"):
        assert k in d["stage_ms"], k
