"""Build step: compiles the CUDA sources under csrc/ into libharp.so (sm_100a only),
in-tree, next to this file.  ``python -m paper_2605_29843_b200.build`` or build()."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libharp.so")


def sources():
    return sorted(glob.glob(os.path.join(HERE, "csrc", "*.cu")))


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(HERE, "csrc", "*.h")) + glob.glob(os.path.join(HERE, "csrc", "*.cuh")) \
        + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(p) > t for p in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-shared", "-Xcompiler", "-fPIC", "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a",
           "-I", os.path.join(ROOT, "include"), "-I", os.path.join(HERE, "csrc")]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if os.environ.get("HARP_TM_TIMING"):          # per-section cycle counters in the tensor-memory kernels
        cmd += ["-DHARP_TM_TIMING"]
    if os.environ.get("HARP_FAST_TIMING"):        # ... and in the whole-row kernel
        cmd += ["-DHARP_FAST_TIMING"]
    if os.environ.get("HARP_UPPER_TIMING"):       # ... and in the dense upper pass (printed by CTA 0)
        cmd += ["-DHARP_UPPER_TIMING"]
    cmd += sources() + ["-o", LIB]
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
