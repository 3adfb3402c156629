"""Builds libmoe_b200.so (sm_100a) in-tree with nvcc.

    python -m paper_2609_07536_b200.build [--force] [--verbose] [--timeline]

--timeline builds libmoe_b200_timeline.so instead: the same sources with -DMOE_TIMELINE=1 (kernels that
record per-CTA time stamps for `bench.py --timeline`); the normal library carries no instrumentation.

nvcc cross-compiles without a GPU, so this also runs on a CPU-only machine.
"""

from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmoe_b200.so")
TIMELINE_LIB = os.path.join(HERE, "libmoe_b200_timeline.so")
SOURCES = ["api.cu", "routing.cu", "gemm2_combine.cu", "gemm1_act.cu", "solver.cpp"]
HEADERS = [os.path.join(CSRC, "moe_internal.h"), os.path.join(CSRC, "sm100_device.cuh"),
           os.path.join(os.path.dirname(HERE), "include", "moe_b200.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, timeline: bool = False) -> str:
    lib = TIMELINE_LIB if timeline else LIB
    if not force and not needs_build(lib):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC,-ffp-contract=off", "-shared", "-cudart", "static",
           "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    if timeline:
        cmd.insert(1, "-DMOE_TIMELINE=1")
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, timeline="--timeline" in sys.argv))
