"""CPU-only checks of the product's host side: the C-ABI library loads and exports every declared
symbol, argument validation that needs no GPU, and the placement helpers against the oracle's."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import director_oracle as orc
from paper_2607_08782_b200 import binding, placement, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "director.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(director_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert len(names) >= 14
    lib = binding.load_library()
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTED) == names


def test_status_strings():
    assert binding.status_string(0) == "ok"
    for code in range(1, 9):
        assert binding.status_string(code) not in ("ok", "unknown status")
    assert binding.status_string(1234) == "unknown status"


def test_create_rejects_bad_arguments_before_touching_the_gpu():
    lib = binding.load_library()
    ctx = ctypes.c_void_p()
    assert lib.director_create(None, ctypes.byref(ctx)) == 1
    bad_shapes = [
        dict(T_max=64, H=250, F=512, E=8, K=2, S=0, R=4, C_max=2),     # H not a multiple of 256
        dict(T_max=64, H=256, F=100, E=8, K=2, S=0, R=4, C_max=2),     # F not a multiple of 128
        dict(T_max=64, H=256, F=512, E=8, K=9, S=0, R=4, C_max=2),     # K > 8
        dict(T_max=64, H=256, F=512, E=4, K=5, S=0, R=4, C_max=2),     # K > E
        dict(T_max=64, H=256, F=512, E=9, K=2, S=0, R=4, C_max=2),     # E > R*C_max
        dict(T_max=0, H=256, F=512, E=8, K=2, S=0, R=4, C_max=2),
        dict(T_max=64, H=256, F=512, E=300, K=2, S=0, R=64, C_max=16),
    ]
    for kw in bad_shapes:
        shp = binding.DirectorShape(**kw)
        assert lib.director_create(ctypes.byref(shp), ctypes.byref(ctx)) == 5, kw
        assert not ctx.value


def test_null_context_is_rejected_everywhere():
    lib = binding.load_library()
    assert lib.director_destroy(None) == 1
    assert lib.director_set_placement(None, None, None) == 1
    assert lib.director_route(None, 1, None, None, None, None) == 1
    assert lib.director_last_status(None, None) == 1
    assert lib.director_launch_count(None) == -1


@pytest.mark.parametrize("seed", range(6))
def test_greedy_balanced_matches_the_oracle_definition(seed):
    rng = np.random.default_rng(seed)
    E, R = int(rng.integers(4, 40)), int(rng.integers(2, 9))
    C = -(-E // R) + int(rng.integers(0, 3))
    N = (rng.zipf(1.5, size=E) * rng.integers(0, 2, size=E)).astype(np.int64)
    assert np.array_equal(placement.greedy_balanced(N, R, C), orc.balanced_placement(N, R, C))
    # fixed primaries that respect the capacity
    primary = np.repeat(np.arange(R), C)[rng.permutation(R * C)[:E]]
    assert np.array_equal(placement.greedy_balanced(N, R, C, primary), orc.balanced_placement(N, R, C, primary))


def test_replicate_hottest_matches_the_oracle_definition():
    for seed in range(5):
        rng = np.random.default_rng(100 + seed)
        E = R = 8
        N = rng.integers(0, 50, size=E)
        X = synth.placement_from_ranks(np.arange(E), R)
        assert np.array_equal(placement.replicate_hottest(N, X, 2), orc.replicate_hottest(N, X, 2))


def test_expert_counts_and_loads():
    W = np.array([[1, 2, 3], [4, 5, 6]])
    assert placement.expert_counts(W).tolist() == [5, 7, 9]
    X = np.array([[1, 0], [0, 1], [1, 0]], dtype=np.uint8)
    assert placement.single_copy_loads([5, 7, 9], X).tolist() == [14, 7]


def test_the_header_is_plain_c(tmp_path):
    """include/director.h is the C ABI: it must compile as C99 with warnings on, without any CUDA header."""
    import os
    import shutil
    import subprocess
    gcc = shutil.which("gcc")
    if gcc is None:
        import pytest
        pytest.skip("no C compiler")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_header.c"
    src.write_text('#include "director.h"\nint main(void) { director_shape s = {0}; (void)s; return DIRECTOR_OK; }\n')
    r = subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(root, "include"),
                        "-fsyntax-only", str(src)], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr
