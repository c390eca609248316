"""The C ABI used from plain C: a small program is compiled with gcc against include/director.h, linked to
libdirector.so and the CUDA runtime, and run on the GPU."""
import os
import shutil
import subprocess

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _build_and_run(tmp_path, name):
    from paper_2607_08782_b200 import build
    gcc = shutil.which("gcc")
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    if gcc is None or not os.path.exists(os.path.join(cuda, "include", "cuda_runtime_api.h")):
        pytest.skip("needs gcc and the CUDA runtime headers")
    lib = build.build_director()
    exe = tmp_path / name
    cmd = [gcc, "-std=c99", "-O1", "-Wall", "-I", os.path.join(ROOT, "include"), "-I", os.path.join(cuda, "include"),
           os.path.join(ROOT, "tests", "c_abi", name + ".c"), "-o", str(exe), str(lib),
           "-L", os.path.join(cuda, "lib64"), "-lcudart", "-lm",
           "-Wl,-rpath," + os.path.dirname(str(lib)), "-Wl,-rpath," + os.path.join(cuda, "lib64")]
    r = subprocess.run(cmd, capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
    r = subprocess.run([str(exe)], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stdout + r.stderr
    return r.stdout


def test_a_c_program_can_gate_a_batch_through_the_library(tmp_path):
    assert "0 mismatches" in _build_and_run(tmp_path, "route_from_c")


def test_a_c_program_drives_every_stage_and_the_one_call_layer(tmp_path):
    """dispatch, expert FFN, combine, placement cost and director_layer_forward from plain C, with the method's
    invariants checked in C: segment table, row <-> token, loads summing to T*K, identity round trip, stage calls
    equal to the one-call layer bit for bit."""
    out = _build_and_run(tmp_path, "layer_from_c")
    assert " 0 mismatches" in out and "identity exact" in out and "one-call layer identical" in out
