"""Builds libamla.so (the C-ABI library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libamla.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared", "--use_fast_math=false",
]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + [os.path.join(_HERE, "..", "include", "amla.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_trace(level: int = 1) -> str:
    """Developer aid: libamla_trace.so, the same sources with -DAMLA_TRACE=level (per-role cycle stamps;
    level 2 adds several stamps per ring slot, which slows the issuer loops it measures)."""
    out = os.path.join(_HERE, "libamla_trace.so")
    nvcc = os.environ.get("NVCC", "nvcc")
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")] + [f"-DAMLA_TRACE={level}"]
    subprocess.check_call([nvcc] + flags + sources() + ["-o", out])
    return out


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    nvcc = os.environ.get("NVCC", "nvcc")
    flags = [f for f in NVCC_FLAGS if not f.startswith("--use_fast_math")]
    if verbose:
        flags += ["-Xptxas", "-v"]
    tmp = LIB + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + flags + sources() + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    if "--trace" in sys.argv:
        print(build_trace(2 if "--full" in sys.argv else 1))
        sys.exit(0)
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
