"""The benchmark's one-line JSON contract, checked on a short run (a few timed steps).

The numbers of a run this short mean nothing; what is checked is that every key a reader of the line relies on
is there, has the right type and is consistent with the others, for the library's own arm and for the arm that
times the CPU oracle."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT, capture_output=True,
                         text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1, res.stdout[-2000:]
    return json.loads(lines[0])


def test_own_arm_line():
    d = run_bench("--steps", "3", "--warmup", "3")
    for key, typ in [("metric", str), ("value", float), ("unit", str), ("n_gpus", int), ("steps", int), ("warmup", int),
                     ("ms_per_step", float), ("higher_is_better", bool), ("scaling", str), ("dtype", str), ("data", str),
                     ("config", dict), ("clocks", dict), ("e2e", dict), ("gpu_launches", int), ("roofline", dict),
                     ("cpu_baseline", dict)]:
        assert isinstance(d[key], typ), key
    assert d["vs_baseline"] is None and d["n_gpus"] == 1 and d["steps"] == 3 and d["warmup"] == 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["data"] == "synthetic"
    assert "workload" in d["config"] and "l2" in d["config"] and "model" not in d["config"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert abs(r["achieved"] - d["value"]) <= 1e-6 * d["value"]           # one GPU: the step is 28 launches of that kernel
    assert r["launches"] == d["gpu_launches"] == 28 * d["steps"]
    assert r["traffic"] is None or 0 < r["traffic"] <= r["algorithmic_bytes_per_launch"] * 1.05
    e = d["e2e"]
    assert e["unit"] == d["unit"] and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert 0 < e["value"] < d["value"]                                     # the copies are inside that timed region
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and c["unit"] == d["unit"] and c["sample"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    assert d["parity"]["status"] == "ok" and d["device_error"] == 0
    assert 0.05 < d["frac_of_hbm_peak"] < 1.3
    assert abs(d["frac_of_nominal_8tbs"] - d["value"] / 8000.0) < 1e-9
    su = d["sustained"]
    assert su["steps"] >= d["steps"] and su["steps"] * su["ms_per_step"] >= 1000.0 and 0.05 < su["frac_of_hbm_peak"] < 1.3
    one = c["one_thread"]
    assert one is None or (one["cores"] == 1 and 0 < one["value"] < c["value"])
    assert "kroquant_quantize_host" in e["api"]


def test_sweep_point_line_carries_parity():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--sweep", "--points", "1024x1152", "--steps", "50"],
                         cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    d = json.loads([l for l in res.stdout.strip().splitlines() if l.startswith("{")][0])
    assert d["shape"] == "1024x1152" and d["parity"]["status"] == "ok" and d["device_error"] == 0
    assert d["parity"]["scale"]["code_mismatches"] == 0 and d["parity"]["plain_mxfp4"]["code_mismatches"] == 0
    assert d["parity"]["kroquant"]["rows"] == 1024 and d["cpu_oracle_rows"] == 1024 and d["cpu_oracle_s"] > 0
    assert set(d["us"]) == {"kroquant", "kroquant_onchip", "scale", "plain_mxfp4"}
    assert d["parity"]["kroquant_onchip"]["rows"] == 1024 and d["onchip_over_kroquant"] > 0


def test_reference_arm_line():
    d = run_bench("--impl", "reference", "--steps", "1", "--warmup", "1")
    assert d["impl"] == "reference" and d["gpu_launches"] == 0 and d["dtype"] == "f64"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["higher_is_better"] is True and d["value"] > 0


def test_boundary_floor_lines():
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--boundary-floor", "--spin-ns", "2000"],
                         cwd=ROOT, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0, res.stderr[-2000:]
    rows = [json.loads(l) for l in res.stdout.strip().splitlines() if l.startswith("{")]
    assert len(rows) >= 10
    for r in rows:
        assert r["idle_us"] == 2.0 and r["period_us"] > 2.0 and 0.2 < r["boundary_cost_us"] < 20.0
    plain = [r for r in rows if not r["boundary_floor"]["tcgen05_in_kernel"]]
    tmem = [r for r in rows if r["boundary_floor"]["permit_released"]]
    # a launch whose CTAs take tensor memory never costs less than the cheapest one that takes none
    assert min(r["boundary_cost_us"] for r in tmem) > min(r["boundary_cost_us"] for r in plain)
