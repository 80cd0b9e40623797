"""Build the C-ABI CUDA library for sm_100a with nvcc (no GPU needed to compile)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libpicospec.so")
SOURCES = [os.path.join(CSRC, "picospec_api.cu")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden"]


def _deps():
    out = list(SOURCES)
    for root in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(root):
            if f.endswith((".cuh", ".h", ".cu")):
                out.append(os.path.join(root, f))
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libpicospec.so in-tree if it is missing or older than its sources."""
    stale = force or not os.path.exists(LIB)
    if not stale:
        t = os.path.getmtime(LIB)
        stale = any(os.path.getmtime(p) > t for p in _deps())
    if stale:
        nvcc = os.environ.get("NVCC", "nvcc")
        extra = os.environ.get("PICOSPEC_NVCC_FLAGS", "").split()     # e.g. -DPICOSPEC_STAGES_BF16=3
        cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB] + SOURCES
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed building libpicospec.so")
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
