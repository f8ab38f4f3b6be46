"""Build the CUDA library (`libhann.so`) in-tree with nvcc for sm_100a.

    python -m paper_2608_21131_b200.build [--force] [--verbose]

`build(extra_flags=...)` passes further compiler flags, e.g. `-DHANN_NO_B8T` / `-DHANN_NO_MAC_BULK` to build the
transform's pass B / the multiply-accumulate without their bulk-copy kernels (A/B comparisons; results are identical).
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhann.so")
SOURCES = ["api.cu", "ntt.cu", "keyswitch.cu", "mac.cu", "encode.cu", "static_scratch.cu", "hostmath.cpp"]
HEADERS = ["internal.h", "modarith.cuh", "nttcore.cuh", "bulkcopy.cuh", os.path.join("..", "..", "include", "hann.h")]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, out: str = LIB, extra_flags=()) -> str:
    if not force and out == LIB and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out + ".%d.tmp" % os.getpid()
    cmd = [
        nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "--fmad=false",  # the encode kernels pin every floating-point rounding
        "--extended-lambda",
        "-Xcompiler", "-fPIC,-O2,-Wall", "-shared", "-o", tmp,
    ]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += list(extra_flags)
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
