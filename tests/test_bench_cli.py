"""The benchmark's command line: the oracle arm on the CPU, and (on a GPU) a small run of the GPU arm, both checked
for the keys and the consistency the one-line JSON contract asks for."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
REQUIRED = ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
            "vs_baseline", "dtype", "data", "config", "e2e", "cpu_baseline")


def _run(*flags, timeout=600):
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *flags], capture_output=True, text=True, env=env,
                       timeout=timeout)
    assert r.returncode == 0, r.stderr[-3000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout[-2000:]
    return json.loads(lines[0])


def test_reference_arm_prints_one_line_for_the_same_metric_and_config():
    d = _run("--impl", "reference", "--config", "1", "--steps", "3", "--warmup", "2")
    for k in REQUIRED:
        assert k in d, k
    assert d["impl"] == "reference" and d["metric"] == "decode_tokens_per_s" and d["unit"] == "tok/s"
    assert d["steps"] == 3 and d["warmup"] == 2                      # the warm-up asked for is honoured
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["dtype"] == "f64"
    assert d["extrapolated_from_layers"] == 1
    assert abs(d["value"] - d["config"]["batch"] / (d["ms_per_step"] * 1e-3)) < 1e-6 * d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"]
    assert d["cpu_baseline"]["cores"] >= 1
    c = d["config"]
    assert c["workload"] == "c1_needle_4k" and c["ctx"] == 4096 and c["budget"] == 256 and c["layers"] == 1


@pytest.mark.gpu
def test_gpu_arm_line_on_a_small_case():
    d = _run("--layers", "2", "--phys-layers", "2", "--steps", "3", "--warmup", "3", "--no-extras", "--no-cpu-baseline")
    for k in REQUIRED:
        if k != "cpu_baseline":
            assert k in d, k
    assert d["n_gpus"] == 1 and d["steps"] == 3 and d["dtype"] == "bf16" and d["data"] == "synthetic"
    assert d["gpu_launches"] == 3 * 2 * 3                          # steps x layers x {attention, selection, gather}
    assert abs(d["value"] - 8 * 3 / (d["ms_per_step"] * 3e-3)) < 1e-6 * d["value"]
    r = d["roofline"]
    assert r["bound"] == "host_link" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and 0.5 < r["frac"] < 1.05
    assert r["peak_spread"]["min"] <= r["peak"] == r["peak_spread"]["max"]
    assert d["e2e"]["h2d_bytes_per_step"] > 2 * 64 * 2**20 and d["e2e"]["d2h_bytes_per_step"] > 0
    assert 0.5 * d["value"] < d["e2e"]["value"] < 1.2 * d["value"]
    assert d["clocks"]["sm_mhz"] and not set(d["clocks"]["reasons"]) & {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
    assert d["layer_step"]["hidden_fraction_target_0.9_met"] is False
    # the reference arm describes the same workload with the same dictionary
    ref_cfg = json.loads(json.dumps(d["config"]))
    assert ref_cfg["workload"] == "c2_llama8b_b8_32k" and ref_cfg["parallelism"] == "single GPU"
