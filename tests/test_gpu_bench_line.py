"""bench.py's own arm on a B200: one JSON line with the keys the measurement contract names."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def bench(*extra):
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *extra], capture_output=True, text=True, timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = p.stdout.strip().splitlines()
    assert len(lines) == 1
    return json.loads(lines[0])


def common(d, steps):
    assert d["unit"] == "positions/s" and d["n_gpus"] == 1 and d["steps"] == steps and d["warmup"] >= 3
    assert d["higher_is_better"] is True and d["scaling"] == "weak" and d["vs_baseline"] is None and d["data"] == "synthetic"
    assert d["value"] > 0 and abs(d["value"] * d["ms_per_step"] * 1e-3 - d["config"]["B_per_gpu"] * (d["config"]["K"] + 1)) < 1e-3 * d["value"] * d["ms_per_step"] * 1e-3 + 1e-6
    r = d["roofline"]
    assert r["bound"] in ("hbm", "tensor") and r["unit"] in ("GB/s", "TFLOP/s") and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and 0 < r["frac"] < 1.3 and r["traffic"] > 0
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["value"] < 1.5 * d["value"]
    assert d["gpu_launches"] >= steps and "l2" in d["config"] and "workload" in d["config"]
    c = d["clocks"]
    assert set(c) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_logits_path_line():
    d = bench("--steps", "400", "--warmup", "3", "--no-cpu-baseline")
    common(d, 400)
    assert d["config"]["workload"] == "llama3_vocab_batch" and d["roofline"]["bound"] == "hbm" and d["dtype"] == "f32"
    assert d["gpu_launches"] == 400 and d["serialized"]["ms_per_step"] >= d["ms_per_step"]


def test_fused_path_line():
    d = bench("--workload", "fused_lm_head", "--steps", "20", "--warmup", "3", "--no-cpu-baseline")
    common(d, 20)
    assert d["roofline"]["bound"] == "tensor" and d["dtype"] == "bf16" and d["gpu_launches"] == 60
    assert d["library_gemm_same_shape"]["tflops"] > 0
