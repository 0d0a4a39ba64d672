"""Builds libdrk.so (hand-written CUDA for sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_PATH = os.path.join(HERE, "libdrk.so")
# the same sources with -DDRK_BOUNDS_CHECK: every index derived on the device is range-checked (status bit, no trap)
CHECKED_LIB_PATH = os.path.join(HERE, "libdrk_check.so")
SOURCES = ["api.cu", "trloo.cu", "mrs.cu", "simt.cu", "umma_kernels.cu", "noalloc.cu", "compact.cu", "reward.cu", "diag.cu"]
HEADERS = ["common.cuh", "umma.cuh", "umma_plan.cuh", os.path.join("..", "..", "include", "drk.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found; set NVCC")


def needs_build(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, bounds_check: bool = False) -> str:
    out = CHECKED_LIB_PATH if bounds_check else LIB_PATH
    if not force and not needs_build(out):
        return out
    cmd = [_nvcc(), "-shared", "-Xcompiler", "-fPIC", "-O3", "-std=c++17", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a", "-cudart", "static",
           "-o", out] + (["-DDRK_BOUNDS_CHECK"] if bounds_check else []) + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return out


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose="-v" in sys.argv, bounds_check="--check" in sys.argv))
