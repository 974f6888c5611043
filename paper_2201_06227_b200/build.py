"""Compile the CUDA library for sm_100a, in-tree (``python -m paper_2201_06227_b200.build``)."""
from __future__ import annotations

import os
import subprocess
import sys
from pathlib import Path

HERE = Path(__file__).resolve().parent
CSRC = HERE / "csrc"
LIB = HERE / "libegeria.so"
LIB_CHECKED = HERE / "libegeria_checked.so"   # the same sources with -DEGERIA_CHECKED (csrc/check.cuh)
SOURCES = [CSRC / "egeria_api.cu"]
HEADERS = sorted(CSRC.glob("*.cuh")) + sorted(CSRC.glob("*.h")) + [HERE.parent / "include" / "egeria.h"]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v",
]


def stale(lib: Path = LIB) -> bool:
    if not lib.exists():
        return True
    t = lib.stat().st_mtime
    return any(p.stat().st_mtime > t for p in SOURCES + HEADERS)


def _compile(lib: Path, extra, verbose: bool) -> None:
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib.with_suffix(f".so.tmp{os.getpid()}")
    cmd = [nvcc, *NVCC_FLAGS, *extra, "-o", str(tmp), *map(str, SOURCES)]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed building {lib.name}")
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False, checked: bool = True) -> Path:
    """Build libegeria.so (and, unless checked=False, libegeria_checked.so) if missing or older than
    the sources.  Raises on failure."""
    if force or stale(LIB):
        _compile(LIB, [], verbose)
    if checked and (force or stale(LIB_CHECKED)):
        _compile(LIB_CHECKED, ["-DEGERIA_CHECKED"], verbose)
    return LIB


if __name__ == "__main__":
    build(force="--force" in sys.argv, verbose=True)
    print(LIB)
    print(LIB_CHECKED)
