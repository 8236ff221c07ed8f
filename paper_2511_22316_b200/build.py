"""Builds libsinglequant.so (the C-ABI library) in-tree with nvcc for sm_100a.

Usage: python -m paper_2511_22316_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libsinglequant.so")
SOURCES = ["sq_all.cu"]
DEPS = ["sq_all.cu", "sq_gemm.cu", "sq_gemm_pair.cu", "sq_gemm_decode.cu", "sq_gemv.cu", "sq_gemm_wo.cu", "sq_rotate_quant.cu", "sq_rotate_quant_tc.cu", "sq_rotate_quant_st.cu", "sq_linear_fused.cu", "sq_rotate_quant_pair.cu", "sq_rotation_host.cu", "sq_api.cu", "sq_noalloc.cu",
        "sq_ptx.cuh", "sq_internal.h", os.path.join("..", "..", "include", "singlequant.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(os.path.join(CSRC, d)) > t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    cmd = [_nvcc(), "-shared", "-Xcompiler", "-fPIC", "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static",
           "-o", LIB] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libsinglequant.so")
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
