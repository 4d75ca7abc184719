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
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and 0 < r["frac"] < 1.3
    assert r["traffic"] is None or r["traffic"] > 0.9 * r.get("bytes_per_launch", 0)
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0 and e["value"] < 1.5 * d["value"]
    assert d["gpu_launches"] >= steps and "l2" in d["config"] and "workload" in d["config"]
    c = d["clocks"]
    assert set(c) >= {"sm_mhz", "sm_max_mhz", "reasons"}


def test_logits_path_line():
    d = bench("--steps", "400", "--warmup", "3", "--no-cpu-baseline", "--no-extra")
    common(d, 400)
    assert d["config"]["workload"] == "llama3_vocab_batch" and d["roofline"]["bound"] == "hbm" and d["dtype"] == "f32"
    assert d["gpu_launches"] == 400 and "workloads" not in d
    # the headline is the plain-stream-order step; the overlapped figure is the labelled secondary
    assert "plain stream order" in d["config"]["order"]
    assert d["overlapped"]["ms_per_step"] < 1.1 * d["ms_per_step"] and d["roofline"]["frac_overlapped"] > 0
    e = d["e2e"]
    assert e["h2d_gbs_measured"] > 1 and 0 < e["frac_of_bound"] < 1.3


def test_default_line_carries_every_workload():
    d = bench("--no-cpu-baseline")
    names = {"tiny_verify", "llama3_vocab_batch", "long_draft_batch", "high_batch_serving", "fused_lm_head",
             "paper_default_70b", "paper_default_405b"}
    assert set(d["workloads"]) == names
    for n, row in d["workloads"].items():
        assert row["steps"] >= 1 and set(row["clocks"]) >= {"sm_mhz", "reasons"}
        if n == "fused_lm_head":
            assert row["tflops"] > 0 and 0 < row["frac_of_burst"] < 1.2 and row["library_gemm_same_shape"]["tflops"] > 0
            assert row["steps"] * row["us_per_step"] >= 40e3          # at least ~50 ms of timed work
        else:
            assert 0 < row["frac_serial"] < 1.3 and 0 < row["frac_overlapped"] < 1.3
            assert row["steps"] * row["us_per_step_serial"] >= 40e3


def test_vocabulary_parallel_mode_on_one_rank():
    d = bench("--shard", "vocab", "--steps", "50", "--warmup", "3")
    assert d["config"]["parallelism"] == "tp1" and d["scaling"] == "strong" and d["n_gpus"] == 1 and d["steps"] == 50
    assert d["value"] > 0 and d["roofline"]["bound"] == "hbm" and 0 < d["roofline"]["frac"] < 1.3
    assert d["gpu_launches"] == 4 * 50


def test_fused_path_line():
    d = bench("--workload", "fused_lm_head", "--steps", "20", "--warmup", "3", "--no-cpu-baseline")
    common(d, 20)
    assert d["roofline"]["bound"] == "tensor" and d["dtype"] == "bf16" and d["gpu_launches"] == 60
    assert d["library_gemm_same_shape"]["tflops"] > 0
