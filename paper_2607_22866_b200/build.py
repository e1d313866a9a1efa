"""Builds the CUDA library in-tree for sm_100a with nvcc (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB_PATH = os.path.join(_HERE, "libgmagnus.so")
_SOURCES = ["gm_api.cu", "gm_planner.cpp"]


def _newest_source_mtime() -> float:
    t = os.path.getmtime(os.path.join(_INCLUDE, "gmagnus.h"))
    for f in os.listdir(_CSRC):
        t = max(t, os.path.getmtime(os.path.join(_CSRC, f)))
    return t


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/ into libgmagnus.so (sm_100a only).  Returns the library path."""
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-cudart", "shared", "-I", _INCLUDE, "-I", _CSRC, "-o", tmp]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(_CSRC, s) for s in _SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
