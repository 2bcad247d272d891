"""Builds the in-tree CUDA library (sm_100a only) with nvcc.  No JIT, no torch extension:
the result is a plain C-ABI shared object next to this file."""
from __future__ import annotations

import glob
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmoe_apk.so")
NVCC = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
         "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        [os.path.join(HERE, "..", "include", "moe_apk.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_probe(verbose: bool = False) -> str:
    """The same library with the in-kernel timers compiled in (-DMOE_TIMING_PROBE): the MMA, producer
    and epilogue warps of one CTA record clock64 stamps per k-block into the tile-log area, which
    moe_read_tile_log then returns as raw 64-bit words (the log itself is off in this build).  For
    kernel studies only; never loaded by the package."""
    out = os.path.join(HERE, "libmoe_apk_probe.so")
    res = subprocess.run([NVCC] + FLAGS + ["-DMOE_TIMING_PROBE", "-o", out] + sources(), capture_output=True, text=True)
    if verbose or res.returncode != 0:
        print(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed")
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        cmd = [NVCC] + FLAGS + ["-o", LIB] + sources()
        res = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or res.returncode != 0:
            print(res.stdout + res.stderr)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed")
    return LIB


if __name__ == "__main__":
    import sys
    if "--probe" in sys.argv:
        print(build_probe(verbose=True))
    else:
        build(force=True, verbose=True)
