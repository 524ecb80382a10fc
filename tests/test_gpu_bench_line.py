"""The benchmark's JSON line on a small workload: every key the contract names is present and
consistent (the full-size numbers are not asserted here, only the shape of the record)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("workload,extra", [("tiers64", []), ("zipf1k", ["--replicas", "8"])])
def test_bench_prints_one_complete_json_line(workload, extra):
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", workload, "--steps", "4", "--warmup", "3",
                          "--no-cpu-all-cores", "--sustain-s", "0.05"] + extra, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
              "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert k in d, k
    assert d["steps"] == 4 and d["warmup"] == 3 and d["n_gpus"] == 1 and d["scaling"] == "weak" and d["vs_baseline"] is None
    assert d["config"]["workload"] == workload and "model" not in d["config"]
    assert d["value"] > 0 and d["gpu_launches"] >= 3 * 4                     # advance, step, fold at least, per step
    assert abs(d["value"] - d["config"]["requests_per_step_per_gpu"] / (d["ms_per_step"] * 1e-3)) < 1e-6 * d["value"]
    e = d["e2e"]
    assert e["unit"] == d["unit"] and 0 < e["value"] and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] != d["value"]
    r = d["roofline"]
    assert r["bound"] in ("hbm", "tensor", "alu") and r["unit"] == "GB/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and "traffic" in r
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0 and c["sample"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
    # the K-step region repeated back to back, and the request path's line with the stated target beside it
    su = d["sustained"]
    assert su["repeats"] >= 3 and su["ms_per_step_min"] <= su["ms_per_step_median"] <= su["ms_per_step_max"]
    rq = d["roofline_request_path"]
    assert rq["target_frac"] == 0.6 and rq["target_met"] == (rq["frac"] >= 0.6) and rq["requests_per_s"] > 0
