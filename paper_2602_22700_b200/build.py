"""Builds libimm.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2602_22700_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libimm.so")
SOURCES = ["imm_kernels.cu", "imm_api.cu", "imm_ldd.cu", "imm_commit.cu", "imm_glue.cu"]
DEPS = SOURCES + ["sha256.cuh", "gl64.cuh", "imm_plan.h", "imm_kernels.h", "imm_mma.cuh", "imm_fused.cuh", os.path.join("..", "..", "include", "imm.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "shared"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += os.environ.get("IMM_NVCC_FLAGS", "").split()      # e.g. -DIMM_TUNING (tile-geometry overrides for sweeps)
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
