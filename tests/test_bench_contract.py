"""The benchmark's reference arm runs on the host cores alone: its JSON line must carry the keys the
contract names, and the CUDA arm must refuse to run without a GPU instead of falling back."""
import json
import os
import subprocess
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def run_bench(*args):
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *args], capture_output=True, text=True,
                          timeout=600, cwd=ROOT)


def test_reference_arm_prints_the_contract_line():
    r = run_bench("--impl", "reference", "--steps", "1", "--warmup", "0")
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["metric"] == "varlen_attn_fwd_bwd_tflops" and line["unit"] == "TFLOP/s"
    for key in ("value", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline", "dtype",
                "data", "config", "cpu_baseline", "e2e", "gpu_launches"):
        assert key in line, key
    assert line["value"] > 0 and line["dtype"] == "f64" and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["e2e"]["value"] == line["value"]


def test_cuda_arm_fails_loudly_without_a_gpu():
    if torch.cuda.is_available():
        return
    r = run_bench("--steps", "1", "--warmup", "0", "--no-cpu-baseline")
    assert r.returncode != 0
    assert "no CPU fallback" in (r.stderr + r.stdout)


import pytest  # noqa: E402


@pytest.mark.gpu
def test_cuda_arm_prints_the_contract_line():
    r = run_bench("--workload", "text", "--steps", "2", "--warmup", "3")
    assert r.returncode == 0, r.stderr[-2000:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in line, key
    assert line["dtype"] == "bf16" and line["data"] == "synthetic" and line["scaling"] == "weak" and line["n_gpus"] == 1
    assert line["value"] > 100 and line["gpu_launches"] == 2 * 10            # ten kernels per step
    assert "workload" in line["config"]
    roof = line["roofline"]
    assert roof["bound"] in ("tensor", "hbm") and 0 < roof["frac"] < 1.2 and roof["achieved"] > 0 and roof["peak"] > 0
    e2e = line["e2e"]
    assert e2e["value"] > 0 and e2e["h2d_bytes_per_step"] > 0 and e2e["d2h_bytes_per_step"] > 0
    assert line["clocks"]["sm_max_mhz"] >= line["clocks"]["sm_mhz"] > 0
    base = line["cpu_baseline"]
    assert base["kind"] == "oracle" and base["value"] > 0 and base["cores"] >= 1
    busy = line["sm_busy"]
    assert busy["fwd"]["ctas"] > 0 and busy["bwd_main"]["max_over_mean"] >= 1.0
    assert set(line["others"]) == {"video", "extreme", "stream", "spatial2d", "temporal2d", "spatial2d_d72", "temporal2d_d72",
                                   "balance_w8"}
    balance = line["others"].pop("balance_w8")
    assert 1.0 <= balance["max_over_mean_sharded"] <= balance["max_over_mean_as_drawn"]
    assert all("error" not in o and o["value"] > 0 for o in line["others"].values())
