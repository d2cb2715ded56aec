"""Build step of the CUDA library (nvcc, sm_100a only)."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libyoco_xattn.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "--shared", "-cudart", "static",
    "-I", os.path.join(_ROOT, "include"),
]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = _sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(
        os.path.join(_ROOT, "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build_cuda_library(force: bool = False, verbose: bool = False) -> str | None:
    """Compile csrc/*.cu into libyoco_xattn.so.  Returns the path, or None when there is no
    nvcc and a built library is already in place (a GPU machine that received the built file)."""
    if not _sources():
        raise RuntimeError("no CUDA sources under csrc/")
    if not force and not _stale():
        return LIB_PATH
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(nvcc):
        if os.path.exists(LIB_PATH):
            return None
        raise RuntimeError("nvcc not found and libyoco_xattn.so has not been built")
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB_PATH] + _sources()
    subprocess.run(cmd, check=True)
    return LIB_PATH
