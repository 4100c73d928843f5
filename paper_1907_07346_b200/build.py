"""Build libdeepsqueeze.so (CUDA, sm_100a only) in-tree with nvcc.

    python -m paper_1907_07346_b200.build [--force] [--verbose] [--debug]

-fmad=false: the kernels spell out every fused multiply-add themselves
(__fmaf_rn); the compiler must not contract any other a*b+c, because packed
codes have to match a plain IEEE evaluation bit for bit.
"""
from __future__ import annotations

import os
import re
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
OBJ = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libdeepsqueeze.so")
SOURCES = ["ds_api.cu", "ds_kernels_tma.cu", "ds_kernels_tma_a.cu", "ds_kernels_tma_b.cu", "ds_kernels_tma_c.cu", "ds_kernels_fused.cu", "ds_kernels_wide.cu", "ds_kernels_wide_tma.cu", "ds_kernels_compress.cu",
           "ds_kernels_misc.cu", "ds_noalloc.cu", "ds_kernels_resident.cu", "ds_kernels_tma_pair.cu", "ds_kernels_tma_ecsgd.cu",
           "ds_kernels_wide_norm.cu", "ds_kernels_wide_tma_norm.cu", "ds_kernels_reduce_norm.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-fmad=false", "-Xcompiler", "-fPIC", "-Xcompiler", "-O2"]


def _deps(path: str, seen: set | None = None) -> set:
    """The file and every file it includes with #include "...", recursively."""
    seen = set() if seen is None else seen
    path = os.path.normpath(path)
    if path in seen or not os.path.exists(path):
        return seen
    seen.add(path)
    with open(path) as f:
        for line in f:
            m = re.match(r'\s*#\s*include\s+"([^"]+)"', line)
            if m:
                _deps(os.path.join(os.path.dirname(path), m.group(1)), seen)
    return seen


def _newest(paths) -> float:
    return max(os.path.getmtime(p) for p in list(paths) + [os.path.abspath(__file__)])


LIB_DEBUG = os.path.join(HERE, "libdeepsqueeze_debug.so")
OBJ_DEBUG = os.path.join(HERE, "_build_debug")


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """debug=True: the checked build (-DDS_DEBUG: the kernels validate their index
    arithmetic and report instead of touching memory out of range) as
    libdeepsqueeze_debug.so; load it with DEEPSQUEEZE_LIB=<that path>."""
    obj_dir, lib = (OBJ_DEBUG, LIB_DEBUG) if debug else (OBJ, LIB)
    extra = (["-Xptxas", "-v"] if verbose else []) + (["-DDS_DEBUG"] if debug else [])
    if not force and os.path.exists(lib):
        # an up-to-date library is enough (its object files need not be kept)
        sources = set()
        for src in SOURCES:
            _deps(os.path.join(CSRC, src), sources)
        if os.path.getmtime(lib) >= _newest(sources):
            return lib
    os.makedirs(obj_dir, exist_ok=True)

    def compile_one(src: str) -> str:
        obj = os.path.join(obj_dir, src.replace(".cu", ".o"))
        path = os.path.join(CSRC, src)
        # an object is rebuilt when its source or anything it includes is newer
        if not force and os.path.exists(obj) and os.path.getmtime(obj) >= _newest(_deps(path)):
            return obj
        cmd = ["nvcc", *NVCC_FLAGS, *extra, "-c", path, "-o", obj]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        return obj

    with ThreadPoolExecutor(max_workers=len(SOURCES)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    if force or not os.path.exists(lib) or os.path.getmtime(lib) < max(os.path.getmtime(o) for o in objs):
        subprocess.run(["nvcc", "-shared", "-gencode", "arch=compute_100a,code=sm_100a",
                        "-o", lib, *objs], check=True)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
