"""Build ``libsalad.so`` (CUDA, sm_100a only) in-tree with nvcc.

    python -m paper_2601_16515_b200.build

The library statically links the CUDA runtime and does not link libcuda, so it loads on a
machine without a GPU driver (where only the argument checks can run).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsalad.so")
SOURCES = ["salad_api.cu"]
HEADERS = ["ptx.cuh", "tmap.cuh", "mask_kernels.cuh", "linear_state_kernel.cuh", "fused_kernel.cuh",
           "dynamic_scale_kernel.cuh", "linear_apply_kernel.cuh", "topk_mask_kernels.cuh", "permute_kernel.cuh", "proj_gemm_kernel.cuh",
           "rope_table_kernel.cuh", "selftest_kernel.cuh", "work_order_kernel.cuh",
           os.path.join("..", "..", "include", "salad.h")]


def nvcc_command(out: str, verbose: bool = False):
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC,-fvisibility=hidden", "-cudart", "static",
           "-o", out] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    return cmd


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if force or needs_build():
        tmp = LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(nvcc_command(tmp, verbose))
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
