"""The benchmark's one-line JSON contract, on the smallest workload: the reference arm (the CPU
oracle; runs anywhere) and the CUDA arm (needs a GPU)."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
BASE_KEYS = {"metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
             "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config", "e2e"}


def _bench(*args):
    proc = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], cwd=ROOT,
                          capture_output=True, text=True, timeout=900)
    assert proc.returncode == 0, proc.stderr[-2000:]
    lines = [l for l in proc.stdout.splitlines() if l.strip()]
    assert len(lines) == 1, "exactly one line on stdout"
    return json.loads(lines[0])


def test_reference_arm_prints_the_contract_line():
    d = _bench("--impl", "reference", "--workload", "single-512", "--steps", "2", "--warmup", "1")
    assert BASE_KEYS <= set(d)
    assert d["impl"] == "reference" and d["steps"] == 2 and d["n_gpus"] == 1
    assert d["metric"] == "pruned_weights_per_sec" and d["unit"] == "weights/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["config"]["workload"] == "single-512" and "model" not in d["config"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["sample"] and cb["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}
    assert d["value"] > 0 and d["ms_per_step"] > 0 and "extrapolated" in d


@pytest.mark.gpu
def test_cuda_arm_prints_the_contract_line():
    d = _bench("--workload", "single-512", "--steps", "3", "--warmup", "3", "--ewma-blocks", "0")
    assert BASE_KEYS <= set(d) and "impl" not in d
    assert d["steps"] == 3 and d["warmup"] >= 3 and d["n_gpus"] == 1 and d["scaling"] == "weak"
    assert d["config"]["workload"] == "single-512" and "model" not in d["config"]
    total = d["config"]["total_weights"]
    assert abs(d["value"] - total / (d["ms_per_step"] * 1e-3)) <= 1e-6 * d["value"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and "traffic" in r
    e = d["e2e"]
    assert e["value"] > 0 and e["unit"] == d["unit"]
    assert e["h2d_bytes_per_step"] >= 2 * (total + 16 * 128 * 512)      # weights + activations
    assert e["d2h_bytes_per_step"] >= 2 * total                          # pruned weights (+ masks)
    assert e["value"] < d["value"]                                       # copies cost something
    assert d["gpu_launches"] >= 3 * 3                                    # calib, finalise, select per step
    assert {"sm_mhz", "sm_max_mhz", "reasons"} <= set(d["clocks"])
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] > 0 and cb["sample"]
