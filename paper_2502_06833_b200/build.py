"""Builds the C-ABI CUDA library in-tree: ``paper_2502_06833_b200/libead_b200.so``.

sm_100a only (tcgen05 / TMEM / TMA); nvcc cross-compiles without a GPU.
Run as ``python -m paper_2502_06833_b200.build [--force] [--verbose]``.
"""
from __future__ import annotations

import os
import subprocess
import sys

_DIR = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_DIR, "csrc")
LIB_PATH = os.path.join(_DIR, "libead_b200.so")
SOURCES = [os.path.join(_CSRC, "ead_api.cu")]


def _deps():
    inc = os.path.join(os.path.dirname(_DIR), "include", "ead.h")
    return [inc] + [os.path.join(_CSRC, f) for f in sorted(os.listdir(_CSRC))]


def nvcc_command(verbose: bool = False):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC,-O2,-Wall", "-shared", "-cudart", "static",
           "-o", LIB_PATH] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    return cmd


def build(force: bool = False, verbose: bool = False) -> str:
    stale = (not os.path.exists(LIB_PATH)
             or any(os.path.getmtime(d) > os.path.getmtime(LIB_PATH) for d in _deps()))
    if force or stale:
        res = subprocess.run(nvcc_command(verbose), capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed building libead_b200.so")
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
