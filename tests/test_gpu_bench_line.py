"""The benchmark program end to end on a reduced stack (``-m gpu``): the JSON line it prints carries every key of
the measurement contract, the decode path ran as CUDA kernels of this library, and the phase-graph mode for a long
compression interval and the prefill mode run through."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(*args):
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT, capture_output=True, text=True,
                       timeout=900)
    assert r.returncode == 0, r.stderr[-2000:]
    return json.loads(r.stdout.strip().splitlines()[-1])


def test_decode_line_has_the_contract_keys():
    d = _run("--layers", "2", "--context", "4096", "--steps", "6", "--warmup", "3", "--no-cpu-baseline")
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "roofline", "e2e", "gpu_launches", "clocks"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 6 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["gpu_launches"] >= 6 * 2 * 10
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and 0 < r["frac"] < 1.5 and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9
    assert "alone" in r["schedule"] and r["in_step"]["us_per_launch"] > 0 and "schedule of the timed steps" in r["in_step"]["schedule"]
    # the step is one stack call over the layers; the layer-by-layer figure is reported next to it
    assert "im_decode_stack" in d["config"]["call"] and d["layer_calls"]["ms_per_step"] > 0
    assert d["clocks"]["samples"] >= 1
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert e["value"] <= d["value"] * 1.05            # copies inside the timed region cannot make the step faster


def test_long_interval_and_prefill_modes_run():
    d = _run("--layers", "2", "--context", "4096", "--steps", "8", "--warmup", "3", "--tau", "4", "--no-cpu-baseline")
    assert d["config"]["tau"] == 4 and d["value"] > 0 and d["e2e"]["value"] > 0
    p = _run("--mode", "prefill", "--steps", "1", "--warmup", "3", "--context", "4096", "--no-cpu-baseline")
    assert p["value"] > 0 and p["scoring"]["tensor_cores"]["us_per_launch"] > 0
