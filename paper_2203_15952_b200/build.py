"""Build the CUDA library (libaqt.so) in-tree with nvcc for sm_100a.

    python -m paper_2203_15952_b200.build [--force]
"""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INCLUDE = os.path.join(os.path.dirname(_HERE), "include")
LIB_PATH = os.path.join(_HERE, "libaqt.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _sources():
    files = [os.path.join(_CSRC, f) for f in sorted(os.listdir(_CSRC))]
    files.append(os.path.join(_INCLUDE, "aqt.h"))
    return files


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(f) > t for f in _sources())


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/aqt_api.cu (one translation unit) into libaqt.so if missing or out of date."""
    if force or is_stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = LIB_PATH + ".tmp.%d" % os.getpid()
        cmd = [nvcc, *NVCC_FLAGS, os.path.join(_CSRC, "aqt_api.cu"), "-o", tmp]
        if verbose:
            cmd.insert(1, "-Xptxas")
            cmd.insert(2, "-v")
        subprocess.check_call(cmd)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
