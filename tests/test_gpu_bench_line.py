"""The bench's JSON line on a GPU: one short run of the smallest workload through `bench.py`
itself, checked for the keys and the internal consistency the measurement contract asks for."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*argv):
    # the environment of a user's run: no rank variables, and none of the suite's own kernel switches
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "LESS_SMALL_STEP")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], capture_output=True, text=True,
                       env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, "bench.py prints exactly one JSON line"
    return json.loads(lines[0])


def test_decode_line_of_the_smallest_workload():
    d = _run("--config", "1", "--steps", "4", "--warmup", "3", "--blocks", "3", "--cpu-seconds", "1")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "ms_per_step_min", "blocks",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e",
                "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["blocks"] == 3 and d["vs_baseline"] is None
    assert d["config"]["workload"].startswith("cfg1") and "model" not in d["config"]
    assert d["gpu_launches"] == 4 * 3                           # eight heads: a step is one launch
    assert abs(d["value"] - 8 / (d["ms_per_step"] * 1e-3)) < 1e-6 * d["value"]
    assert d["ms_per_step_min"] <= d["ms_per_step"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert r["kernels"]["decode"].startswith("small_step_kernel<8") and r["kernels"]["feature_map"] == ""
    assert r["kernel"] == r["kernels"]["decode"]
    assert set(r["kernel_us"]) == {"feature_map", "decode"} and r["kernel_us"]["decode"] > 0
    for k in ("step_frac", "step_frac_of_nominal_8TBs", "kv_state_scores_frac", "kv_state_scores_frac_of_nominal_8TBs"):
        assert 0 < r[k] < 1.5
    e = d["e2e"]
    assert e["h2d_bytes_per_step"] == 3 * 8 * 128 * 2 and e["d2h_bytes_per_step"] == 8 * 128 * 4
    assert 0 < e["value"] <= d["value"] * 1.05               # host buffers in the timed region: never faster
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0 and "instances" in c["sample"]


def test_prompt_line_reports_the_state_build_apart_from_the_scoring():
    d = _run("--config", "5", "--batch", "1", "--steps", "1", "--warmup", "3", "--blocks", "2", "--no-cpu-baseline")
    r = d["roofline"]
    assert r["bound"] == "tensor" and r["unit"] == "TFLOP/s"
    assert r["kernels"]["psi"].startswith("psi_tc_kernel<16, 1>")          # psi fused with the state build
    assert "build" not in r["kernel_ms"]                                   # no separate state-build launch
    assert 0 < r["state_build"]["frac"] < 1 and 0 < r["scoring"]["frac"] < 1
    assert r["state_build"]["ms"] < r["scoring"]["ms"]
