"""The benchmark's contract on a GPU: one JSON line with the agreed keys, on a small batch."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*extra):
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "20", "--warmup", "3", "--no-cpu-baseline", *extra]
    res = subprocess.run(cmd, cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.strip()]
    assert len(lines) == 1, res.stdout
    return json.loads(lines[0])


def test_default_workload_line_has_the_contract_keys():
    d = _run("--batch", "4")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 20 and d["higher_is_better"] is True and d["scaling"] == "weak"
    assert d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["config"]["workload"].startswith("mha7b_b64_c2048")
    assert d["gpu_launches"] == 20                       # one kernel launch of the library per step
    assert d["value"] > 0 and d["ms_per_step"] > 0
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["value"] < d["value"] * 1.05
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["kernel"] == "decode_tc_kernel"
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and "traffic" in r
    # the rows the update rule rewrote, counted by the kernel, are part of the algorithmic bytes
    assert 0 < r["rows_rewritten_fraction"] < 0.2
    planes = 4 * 32 * 2048 * 128 * 2
    assert r["algorithmic_bytes_per_launch"] > 2 * planes
    p = d["parity"]                                 # the timed launch configuration replayed beside the oracle
    assert p["pass"] and p["max_abs_out_per_step"] <= p["tol"] == 2e-2 and p["max_abs_state_final"] <= p["tol"]
    assert p["units_checked"] >= 8 and p["steps"] >= 20
    rep = d["repeats"]
    assert rep["blocks"] == 5 and rep["min_ms_per_step"] <= rep["median_ms_per_step"] <= rep["max_ms_per_step"]
    assert d["paper_context"]["hardware"] == "not stated"
    sec = d["secondary_write_regime"]               # the diffuse write regime, timed on a second cache
    assert sec["ms_per_step"] > d["ms_per_step"] and 0 < sec["frac"] < 1.2 and abs(sec["write_scale"] - 128 ** -0.5) < 1e-9


def test_stream_workload_line_reports_the_tensor_roofline():
    d = _run("--workload", "stream_b8_c1024", "--batch", "2")
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s" and r["kernel"] == "stream_tc_kernel"
    assert d["config"]["tokens_per_step"] == 256 and d["gpu_launches"] == 20
    assert d["run"]["flags"] == 24 and d["run"]["call"] == "bct_prefill_stream"               # the flags at which the full-length stream holds 2e-2
    assert 0 < r["frac"] < r["frac_executed"] < 1.2  # on the method's flops, and on the flops the MMAs execute
    assert d["parity"]["pass"] and d["parity"]["steps"] == 1024 + 512
