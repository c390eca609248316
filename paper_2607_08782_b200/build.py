"""Builds the native pieces in-tree.

* ``libdirector.so``  - the CUDA C-ABI library (nvcc, sm_100a only).
* ``libsynth.so``     - the seeded synthetic-input generator (gcc + OpenMP, host only).

Both are rebuilt only when a source file is newer than the binary.  nvcc cross-compiles
sm_100a without a GPU, so this also works on a CPU-only machine.
"""
from __future__ import annotations

import os
import shutil
import subprocess
from pathlib import Path

PKG_DIR = Path(__file__).resolve().parent
CSRC = PKG_DIR / "csrc"
INCLUDE = PKG_DIR.parent / "include"

DIRECTOR_LIB = PKG_DIR / "libdirector.so"
SYNTH_LIB = PKG_DIR / "libsynth.so"

NVCC_FLAGS = [
    "-std=c++17", "-O3", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-Xcompiler", "-fPIC", "-shared",
    "--expt-relaxed-constexpr",
]


def _stale(target: Path, sources: list[Path]) -> bool:
    if not target.exists():
        return True
    t = target.stat().st_mtime
    return any(s.stat().st_mtime > t for s in sources)


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and Path(cand).exists():
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def director_sources() -> list[Path]:
    return sorted(CSRC.glob("director_*.cu"))


def build_director(force: bool = False, verbose: bool = False) -> Path:
    srcs = director_sources()
    deps = srcs + sorted(CSRC.glob("*.cuh")) + sorted(INCLUDE.glob("*.h"))
    if force or _stale(DIRECTOR_LIB, deps):
        cmd = [_nvcc(), *NVCC_FLAGS, f"-I{INCLUDE}", f"-I{CSRC}"]
        if verbose:
            cmd += ["-Xptxas", "-v"]
        cmd += ["-o", str(DIRECTOR_LIB), *map(str, srcs)]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose:
            print(res.stdout, res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return DIRECTOR_LIB


def build_synth(force: bool = False) -> Path:
    src = CSRC / "synth_gen.c"
    if force or _stale(SYNTH_LIB, [src]):
        cmd = ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", str(SYNTH_LIB), str(src), "-lm"]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("gcc failed:\n" + res.stdout + res.stderr)
    return SYNTH_LIB


def ptxas_summary() -> str:
    """Compiles every CUDA source with ``-Xptxas -v`` (objects are thrown away) and returns one line per kernel:
    source file, kernel, registers per thread, static shared memory, stack frame and spill bytes."""
    import re
    import tempfile
    rows = ["file | kernel | registers | static smem B | stack B | spill stores B | spill loads B", "---|---|---|---|---|---|---"]
    for src in director_sources():
        with tempfile.NamedTemporaryFile(suffix=".o") as obj:
            cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
                   "--expt-relaxed-constexpr", f"-I{INCLUDE}", f"-I{CSRC}", "-Xptxas", "-v", "-c", "-o", obj.name, str(src)]
            res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
        lines = (res.stdout + res.stderr).splitlines()
        for i, ln in enumerate(lines):
            m = re.search(r"Compiling entry function '([^']+)'", ln)
            if not m:
                continue
            name = subprocess.run(["c++filt", m.group(1)], capture_output=True, text=True).stdout.strip()
            name = name.replace("(anonymous namespace)::", "").replace("director::", "").replace("void ", "")
            name = re.sub(r"\(.*", "", name)
            blob = " ".join(lines[i + 1:i + 4])
            regs = re.search(r"Used (\d+) registers", blob)
            smem = re.search(r"(\d+) bytes smem", blob)
            spill = re.search(r"(\d+) bytes stack frame, (\d+) bytes spill stores, (\d+) bytes spill loads", blob)
            rows.append(" | ".join([src.name, name, regs.group(1) if regs else "?", smem.group(1) if smem else "0",
                                    *(spill.groups() if spill else ("?", "?", "?"))]))
    return "\n".join(rows)


def build_all(force: bool = False, verbose: bool = False) -> None:
    build_synth(force)
    build_director(force, verbose)


if __name__ == "__main__":
    import sys
    if "--ptxas-summary" in sys.argv:
        print(ptxas_summary())
    else:
        build_all(force="--force" in sys.argv, verbose="-v" in sys.argv)
        print(DIRECTOR_LIB, SYNTH_LIB)
