"""bench.py's reference arm (the CPU oracle timed per step) runs without a GPU: check its JSON line against the
contract, that ranks other than 0 stay silent, and that the CUDA arm refuses to run without a device."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _run(args, env_extra=None):
    env = dict(os.environ)
    env.update(env_extra or {})
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py")] + args, cwd=ROOT, env=env,
                          capture_output=True, text=True, timeout=300)


def test_reference_arm_prints_one_contract_line():
    r = _run(["--impl", "reference", "--config", "c1_tiny", "--steps", "2", "--warmup", "1"])
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] and d["unit"] == "tokens/s"
    for key in ("value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling",
                "vs_baseline", "dtype", "data", "config", "cpu_baseline", "e2e"):
        assert key in d, key
    assert d["steps"] == 2 and d["warmup"] == 1 and d["higher_is_better"] is True and d["vs_baseline"] is None
    assert d["dtype"] == "f64" and d["data"] == "synthetic" and "workload" in d["config"]
    cb = d["cpu_baseline"]
    assert cb["kind"] == "oracle" and cb["cores"] >= 1 and cb["value"] == d["value"] and cb["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": d["unit"], "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
    assert d["value"] > 0 and abs(d["ms_per_step"] * 1e-3 * d["value"] - d["config"]["sample_tokens_per_step"]) < 1e-3 * d["config"]["sample_tokens_per_step"]


def test_reference_arm_is_silent_on_other_ranks():
    r = _run(["--impl", "reference", "--config", "c1_tiny", "--steps", "1", "--warmup", "0", "--gpus", "2"],
             {"RANK": "1", "LOCAL_RANK": "1", "WORLD_SIZE": "2"})
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_cuda_arm_refuses_to_run_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    r = _run(["--config", "c1_tiny", "--steps", "1", "--warmup", "0"])
    assert r.returncode != 0
    assert "CUDA" in (r.stderr + r.stdout)


def test_roofline_denominator_follows_the_sampled_clock():
    """The tensor ceiling bench.py divides by is the one measured in the clock regime of the timed region."""
    sys.path.insert(0, ROOT)
    import bench
    peaks = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 2000.0, "sustained_sm_mhz": 1300.0}
    assert bench.tensor_peak_for_clock(peaks, 2000.0) == (1600.0, "burst")
    assert bench.tensor_peak_for_clock(peaks, 1905.0) == (1600.0, "burst")           # within 5 % of the maximum
    assert bench.tensor_peak_for_clock(peaks, 1300.0) == (1400.0, "sustained")
    assert bench.tensor_peak_for_clock(peaks, 1200.0) == (1400.0, "sustained")
    pk, regime = bench.tensor_peak_for_clock(peaks, 1650.0)                           # half way between the two clocks
    assert regime == "between" and abs(pk - 1500.0) < 1e-9
    assert bench.tensor_peak_for_clock(peaks, None)[0] == 1600.0                      # no samples: the stricter ceiling
