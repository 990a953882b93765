"""Builds libsdq_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libsdq_b200.so")
SOURCES = ["sdq_api.cu", "sdq_pack.cu", "sdq_quant_act.cu", "sdq_linear.cu", "sdq_linear_pair.cu", "sdq_linear_group.cu", "sdq_plain.cu", "sdq_calib.cu", "sdq_diag.cu"]
HEADERS = ["sdq_internal.h", "sdq_layout.h", "sdq_linear.h", "sdq_plain.h", "sdq_ptx.cuh", "sdq_codec.cuh", os.path.join("..", "..", "include", "sdq.h"), os.path.join("..", "..", "include", "sdq_diag.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC"]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or _stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", LIB + ".tmp"] + SOURCES
        subprocess.check_call(cmd, cwd=CSRC)
        os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
