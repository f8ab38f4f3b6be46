"""Build the CUDA library (`libhann.so`) in-tree with nvcc for sm_100a.

    python -m paper_2608_21131_b200.build [--force] [--verbose]

Every source file is compiled to an object file of its own (in parallel, only when it or a header is newer than the
object), then the objects are linked.  `build(extra_flags=...)` passes further compiler flags, e.g. `-DHANN_NO_B8T` /
`-DHANN_NO_MAC_BULK` to build the transform's pass B / the multiply-accumulate without their bulk-copy kernels, or
`-DHANN_DEBUG` for the build whose kernels check their index ranges (A/B comparisons; results are identical).
"""
from __future__ import annotations

import hashlib
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libhann.so")
DEBUG_LIB = os.path.join(HERE, "libhann_debug.so")  # the -DHANN_DEBUG build (index range checks in the kernels)
OBJDIR = os.path.join(HERE, "build")
SOURCES = ["api.cu", "ntt.cu", "keyswitch.cu", "mac.cu", "encode.cu", "static_scratch.cu", "project.cu", "probe.cu", "membership.cu", "hostmath.cpp"]
HEADERS = ["internal.h", "modarith.cuh", "nttcore.cuh", "bulkcopy.cuh", "debugcheck.cuh", os.path.join("..", "..", "include", "hann.h")]


def _deps():
    return [os.path.join(CSRC, s) for s in SOURCES + HEADERS]


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(d) > t for d in _deps())


def build_debug(force: bool = False) -> str:
    return build(force=force, out=DEBUG_LIB, extra_flags=("-DHANN_DEBUG",))


def build(force: bool = False, verbose: bool = False, out: str = LIB, extra_flags=()) -> str:
    if not force and out in (LIB, DEBUG_LIB) and not stale(out):
        return out
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = [
        "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "--fmad=false",  # the encode kernels pin every floating-point rounding
        "--extended-lambda",
        "-Xcompiler", "-fPIC,-O2,-Wall",
    ]
    if verbose:
        flags += ["-Xptxas", "-v"]
    flags += list(extra_flags)
    # objects of different flag sets never mix
    tag = hashlib.sha1(" ".join(flags).encode()).hexdigest()[:10]
    objdir = os.path.join(OBJDIR, tag)
    os.makedirs(objdir, exist_ok=True)
    newest_header = max(os.path.getmtime(os.path.join(CSRC, h)) for h in HEADERS)

    def compile_one(src):
        path = os.path.join(CSRC, src)
        obj = os.path.join(objdir, src + ".o")
        if not force and os.path.exists(obj) and os.path.getmtime(obj) > max(os.path.getmtime(path), newest_header):
            return obj
        tmp = obj + ".%d.tmp" % os.getpid()
        subprocess.check_call([nvcc] + flags + ["-c", "-o", tmp, path])
        os.replace(tmp, obj)
        return obj

    with ThreadPoolExecutor(max_workers=min(len(SOURCES), os.cpu_count() or 1)) as ex:
        objs = list(ex.map(compile_one, SOURCES))
    tmp = out + ".%d.tmp" % os.getpid()
    subprocess.check_call([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", tmp] + objs)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    if "--debug" in sys.argv:
        print(build_debug(force="--force" in sys.argv))
