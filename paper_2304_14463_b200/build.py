"""Builds libmoc_b200.so (nvcc, sm_100a only) next to this file.  ``python -m paper_2304_14463_b200.build``"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmoc_b200.so")
SOURCES = ["moc_api.cu", "moc_search.cu", "moc_intervals.cu", "moc_edits.cu"]
HEADERS = ["moc_kernels.cuh", "moc_pair_kernel.cuh", "moc_lane_kernel.cuh", "moc_quad_kernel.cuh", "moc_host.cuh", "moc_search_kernels.cuh", "moc_search_score_kernel.cuh", "moc_edit_pass.cuh", "moc_edit_lanes_kernel.cuh", "moc_interval_kernels.cuh", "moc_edit_kernels.cuh", "moc_cache_host.cuh", os.path.join("..", "..", "include", "moc.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "--use_fast_math"]


def _stale():
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
          ["-t", "4", "-o", tmp] + [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.run(cmd, check=True)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
