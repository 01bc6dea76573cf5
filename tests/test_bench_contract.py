"""The reference arm of bench.py (the fp64 oracle on a bounded sample) prints one JSON line with the agreed keys."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_reference_arm_prints_one_json_line():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "single_fp32", "--steps", "20",
                          "--warmup", "1"],
                         capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "sbp_backward_tflops_kept_rows" and d["unit"] == "TFLOP/s"
    assert d["steps"] == 20 and d["warmup"] == 1 and d["n_gpus"] == 1 and d["higher_is_better"] is True
    assert d["value"] > 0 and d["ms_per_step"] > 0 and d["vs_baseline"] is None
    assert d["config"]["workload"] == "single_fp32"       # the small fp32 layer: the oracle takes milliseconds
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] == d["value"]
    assert d["e2e"] == {"value": d["value"], "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}


import pytest


@pytest.mark.gpu
def test_cuda_arm_prints_one_json_line_with_every_agreed_key():
    """The benchmark's own arm on a small block workload: one JSON line with the keys the contract names, a roofline
    object that adds up, declared copies in the end-to-end figure, and the same `config` object as the reference arm."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--workload", "tiny_block", "--steps", "6", "--warmup", "3"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for k in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
              "dtype", "data", "config", "roofline", "cpu_baseline", "e2e", "gpu_launches", "clocks", "keep_ratio_sweep"):
        assert k in d, k
    assert d["metric"] == "sbp_backward_tflops_kept_rows" and d["unit"] == "TFLOP/s" and d["n_gpus"] == 1
    assert d["steps"] == 6 and d["warmup"] == 3 and d["value"] > 0 and d["scaling"] == "weak" and d["vs_baseline"] is None
    r = d["roofline"]
    assert r["bound"] in ("tensor", "hbm", "alu") and r["achieved"] > 0 and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and r["launches_per_step"] == 2
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1 and d["cpu_baseline"]["value"] > 0
    e = d["e2e"]
    assert e["value"] > 0 and e["value"] < d["value"] and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert d["gpu_launches"] >= 6 * 5                         # sampler + two gathers + two backward kernels per step at least
    assert set(d["keep_ratio_sweep"]) == {"0.5", "1.0"} and d["keep_ratio_sweep"]["1.0"]["bwd_speedup_vs_keep1"] == 1.0
    ref = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "tiny_block", "--steps", "2",
                          "--warmup", "1"], capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert ref.returncode == 0
    assert json.loads(ref.stdout.strip().splitlines()[-1])["config"] == d["config"]
