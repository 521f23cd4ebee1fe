"""Compile libflat_attn.so for sm_100a with nvcc (in-tree, next to this file)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libflat_attn.so")
SOURCES = ["flat_attn_api.cu", "simt_kernels.cu", "fused_tc.cu", "fused_tc2.cu", "fused_tc3.cu", "fused_rgran.cu", "proj_gemm.cu", "naive_tc.cu", "naive_static.cu", "bwd_tc.cu", "layernorm.cu", "fused_tf32.cu"]
HEADERS = ["flat_internal.cuh", "ptx_sm100.cuh", "tc_common.cuh", os.path.join("..", "..", "include", "flat_attn.h")]


def nvcc_path() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libflat_attn.so cannot be built")


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return LIB
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = [nvcc_path(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "static", "--threads", "0"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(CSRC, s) for s in SOURCES] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
