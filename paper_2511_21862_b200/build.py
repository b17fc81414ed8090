"""Compile the CUDA sources into `libooco.so` next to this file (sm_100a only, in-tree)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libooco.so")
LIB_CHECKED = os.path.join(HERE, "libooco_checked.so")   # the same sources with -DOOCO_CHECKS
SOURCES = ["ooco_api.cu", "ooco_sched.cpp"]
HEADERS = ["decode_kernels.cuh", "chunk_kernels.cuh", "chunk_tc_kernels.cuh", "chunk_tc2_kernels.cuh", "block_copy_kernels.cuh", "ptx.cuh", os.path.join("..", "..", "include", "ooco.h"),
           os.path.join("..", "..", "include", "ooco_sched.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "--expt-relaxed-constexpr"]


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Run nvcc if the library is missing or older than its sources; returns the library path.
    `checked`: the variant whose kernels range-check every device-derived index (libooco_checked.so)."""
    lib = LIB_CHECKED if checked else LIB
    if force or is_stale(lib):
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc] + NVCC_FLAGS + (["-DOOCO_CHECKS"] if checked else []) + (["-Xptxas", "-v"] if verbose else []) + \
              ["-o", lib] + [os.path.join(CSRC, f) for f in SOURCES]
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            sys.stderr.write(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError(f"nvcc failed building {os.path.basename(lib)}")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
