"""Builds libodma.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2512_09427_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB_PATH = os.path.join(_HERE, "libodma.so")


def sources():
    src = sorted(glob.glob(os.path.join(_HERE, "csrc", "*.cu")) + glob.glob(os.path.join(_HERE, "csrc", "*.cpp")))
    hdr = sorted(glob.glob(os.path.join(_HERE, "csrc", "*.hpp")) + [os.path.join(_ROOT, "include", "odma.h")])
    return src, hdr


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    src, hdr = sources()
    return any(os.path.getmtime(f) > t for f in src + hdr)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA/C++ source into one shared library; returns its path."""
    if not force and not is_stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    src, _ = sources()
    cmd = [nvcc, "-std=c++17", "-O3", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include"),
           "-I", os.path.join(_HERE, "csrc"), "-o", LIB_PATH] + src
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libodma.so")
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
