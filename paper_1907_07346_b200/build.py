"""Build libdeepsqueeze.so (CUDA, sm_100a only) in-tree with nvcc.

    python -m paper_1907_07346_b200.build [--force] [--verbose]

-fmad=false: the kernels spell out every fused multiply-add themselves
(__fmaf_rn); the compiler must not contract any other a*b+c, because packed
codes have to match a plain IEEE evaluation bit for bit.
"""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libdeepsqueeze.so")
SOURCES = ["ds_api.cu", "ds_kernels_tma.cu", "ds_kernels_fused.cu", "ds_kernels_wide.cu", "ds_kernels_wide_tma.cu", "ds_kernels_compress.cu",
           "ds_kernels_misc.cu", "ds_noalloc.cu"]
HEADERS = ["ds_device.cuh", "ds_internal.h", "ds_column_kernel.cuh", "ds_fused_tma_kernel.cuh", "ds_wide_fused_kernel.cuh", "ds_wide_tma_kernel.cuh"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-Xcompiler", "-fPIC", "-Xcompiler", "-O2"]


def _newest_input() -> float:
    paths = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    paths.append(os.path.join(os.path.dirname(HERE), "include", "deepsqueeze.h"))
    paths.append(os.path.abspath(__file__))
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_input():
        return LIB
    os.makedirs(OBJ, exist_ok=True)
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJ, src.replace(".cu", ".o"))
        cmd = ["nvcc", *NVCC_FLAGS, *extra, "-c", os.path.join(CSRC, src), "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        return obj

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    subprocess.run(["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
                    "-o", LIB, *objs], check=True)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
