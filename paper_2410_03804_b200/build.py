"""Builds libmoa.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmoa.so")
LIB_TRACE = os.path.join(HERE, "libmoa_trace.so")      # same sources with -DMOA_TRACE: kernels stamp a stage trace
LIB_CHECKS = os.path.join(HERE, "libmoa_checks.so")    # same sources with -DMOA_CHECKS: device-side index checks
SOURCES = ["moa_api.cu"]


def _newest_source() -> float:
    t = 0.0
    for root in (CSRC, os.path.join(os.path.dirname(HERE), "include")):
        for f in os.listdir(root):
            if f.endswith((".cu", ".cuh", ".h", ".inc")):
                t = max(t, os.path.getmtime(os.path.join(root, f)))
    return t


def build(force: bool = False, verbose: bool = False, trace: bool = False, checks: bool = False) -> str:
    lib = LIB_TRACE if trace else LIB_CHECKS if checks else LIB
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= _newest_source():
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-o", lib] + [os.path.join(CSRC, s) for s in SOURCES]
    cmd[1:1] = os.environ.get("MOA_NVCC_FLAGS", "").split() + (["-DMOA_TRACE"] if trace else []) + (["-DMOA_CHECKS"] if checks else [])
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libmoa.so")
    if verbose:
        sys.stderr.write(res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, trace="--trace" in sys.argv, checks="--checks" in sys.argv))
