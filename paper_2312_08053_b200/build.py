"""Builds the CUDA library in-tree for sm_100a with nvcc (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB_PATH = os.path.join(_HERE, "libkimad.so")
CHECKED_LIB_PATH = os.path.join(_HERE, "libkimad_checked.so")  # -DKIMAD_CHECKED: index tests and canaries
SOURCES = [os.path.join(_HERE, "csrc", "kimad_api.cu")]
HEADERS = [os.path.join(_HERE, "csrc", "kimad_kernels.cuh"), os.path.join(_HERE, "csrc", "kimad_select.cuh"),
           os.path.join(_HERE, "csrc", "kimad_curve.cuh"), os.path.join(_HERE, "csrc", "kimad_common.h"),
           os.path.join(_HERE, "csrc", "kimad_receiver.cuh"),
           os.path.join(_ROOT, "include", "kimad.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    out = CHECKED_LIB_PATH if checked else LIB_PATH
    if not force and not is_stale(out):
        return out
    cmd = [_nvcc(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include"),
           "-I", os.path.join(_HERE, "csrc"), "-o", out] + (["-DKIMAD_CHECKED"] if checked else []) + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        sys.stderr.write(res.stderr)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
