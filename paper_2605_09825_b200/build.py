"""Build ``libmxfp4.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU).

Run as ``python -m paper_2605_09825_b200.build`` or call :func:`build_library`.
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libmxfp4.so")
BOUNDS_LIB_PATH = os.path.join(PKG_DIR, "libmxfp4_bounds.so")   # debug build, -DMXFP4_BOUNDS

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-std=c++17", "-lineinfo",
    "-shared", "-Xcompiler", "-fPIC",
    "-Xptxas", "-v",
]


def _sources():
    out = [os.path.join(PKG_DIR, "..", "include", "mxfp4.h")]
    for f in sorted(os.listdir(CSRC)):
        if f.endswith((".cu", ".cuh", ".h")):
            out.append(os.path.join(CSRC, f))
    return out


def needs_build(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(s) > t for s in _sources())


def build_library(force: bool = False, verbose: bool = False, bounds: bool = False) -> str:
    """Build the library (``bounds=True``: the bounds-checking debug build, every computed
    shared-memory address checked, misses recorded in the status word instead of executed)."""
    path = BOUNDS_LIB_PATH if bounds else LIB_PATH
    if not force and not needs_build(path):
        return path
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = path + f".tmp{os.getpid()}"
    cmd = [nvcc] + NVCC_FLAGS + (["-DMXFP4_BOUNDS"] if bounds else []) + ["-o", tmp, os.path.join(CSRC, "libmxfp4.cu")]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError(f"nvcc failed building {os.path.basename(path)}")
    os.replace(tmp, path)
    return path


if __name__ == "__main__":
    print(build_library(force=True, verbose=True, bounds="--bounds" in sys.argv))
