"""Builds libmoe_b200.so (sm_100a only) in-tree with nvcc.  `python -m paper_2606_26453_b200.build`."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libmoe_b200.so")
# Test-only variant: device-side waits give up after 20 ms instead of 2 s, and a switch exists that withholds one
# barrier arrival so that a wait really runs out (tests/test_gpu_wait_timeout.py).  Never loaded by the binding.
WAITTEST_LIB_PATH = os.path.join(PKG_DIR, "libmoe_b200_waittest.so")
WAITTEST_FLAGS = ["-DMOE_TEST_HOOKS", "-DMOE_WAIT_LIMIT_NS=20000000ull"]
SOURCES = ["api.cu", "movement.cu", "router.cu", "grouped_gemm.cu", "mxfp8.cu"]
HEADERS = ["common.cuh", "tc_ptx.cuh", os.path.join("..", "..", "include", "moe_b200.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def needs_build(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, waittest: bool = False) -> str:
    path = WAITTEST_LIB_PATH if waittest else LIB_PATH
    if not force and not needs_build(path):
        return path
    cmd = [_nvcc(), "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v" if verbose else "-warn-spills",
           "-o", path] + (WAITTEST_FLAGS if waittest else []) + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stdout + res.stderr)
    return path


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
    print(build_library(force=True, waittest=True))
