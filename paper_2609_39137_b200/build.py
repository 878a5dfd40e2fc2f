"""Builds the CUDA library (sm_100a only) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "moe_route.cu")
LIB = os.path.join(HERE, "libmoe_route_b200.so")
LIB_DEBUG = os.path.join(HERE, "libmoe_route_b200_debug.so")   # -DMOE_DEBUG: index guards + workspace canaries
LIB_TIMERS = os.path.join(HERE, "libmoe_route_b200_timers.so")  # -DMOE_KERNEL_TIMERS: cycle accounting per warp role


def sources():
    d = os.path.join(HERE, "csrc")
    out = [os.path.join(d, f) for f in sorted(os.listdir(d)) if f.endswith((".cu", ".cuh"))]
    out.append(os.path.join(os.path.dirname(HERE), "include", "moe_route.h"))
    return out


def up_to_date(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    return all(os.path.getmtime(s) <= t for s in sources())


def build(force: bool = False, verbose: bool = False, debug: bool = False, timers: bool = False) -> str:
    lib = LIB_TIMERS if timers else LIB_DEBUG if debug else LIB
    if not force and up_to_date(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-fmad=false", "-shared", "-Xcompiler", "-fPIC", "-o", lib, SRC]
    if timers:
        cmd.insert(1, "-DMOE_KERNEL_TIMERS")
    elif debug:
        cmd.insert(1, "-DMOE_DEBUG")
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + r.stdout + r.stderr)
    return lib


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv, timers="--timers" in sys.argv))
