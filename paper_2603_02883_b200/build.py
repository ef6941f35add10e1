"""Builds libfb4.so (the CUDA kernels and the C-ABI of include/fb4.h) in-tree with nvcc for sm_100a.

    python -m paper_2603_02883_b200.build [--force] [--verbose]

nvcc cross-compiles without a GPU.  Objects go to _build/ (git-ignored); the shared
library lands next to this file so that it travels with the source tree.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
OBJDIR = os.path.join(HERE, "_build")
LIB = os.path.join(HERE, "libfb4.so")

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps() -> list[str]:
    return sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + \
        glob.glob(os.path.join(INCLUDE, "*.h")) + glob.glob(os.path.join(INCLUDE, "*.cuh")) + [os.path.abspath(__file__)]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not stale():
        return LIB
    os.makedirs(OBJDIR, exist_ok=True)
    nvcc = os.environ.get("NVCC", "nvcc")
    extra = ["-Xptxas", "-v"] if verbose else []

    def compile_one(src: str) -> str:
        obj = os.path.join(OBJDIR, os.path.basename(src)[:-3] + ".o")
        cmd = [nvcc, *NVCC_FLAGS, *extra, "-c", src, "-o", obj]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if verbose or r.returncode != 0:
            sys.stderr.write(" ".join(cmd) + "\n" + r.stdout + r.stderr)
        if r.returncode != 0:
            raise RuntimeError(f"nvcc failed on {src}")
        return obj

    with ThreadPoolExecutor(max_workers=min(8, len(sources()))) as ex:
        objs = list(ex.map(compile_one, sources()))
    tmp = LIB + f".{os.getpid()}.tmp"
    subprocess.check_call([nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", tmp, *objs,
                           "-cudart", "static"])
    os.replace(tmp, LIB)
    return LIB


HOSTCOST = os.path.join(HERE, "fb4_hostcost")


def build_hostcost(force: bool = False) -> str:
    """The C program that times the host side of the ABI (hostcost/fb4_hostcost.c), linked against libfb4.so."""
    src = os.path.join(HERE, "hostcost", "fb4_hostcost.c")
    if not force and os.path.exists(HOSTCOST) and os.path.getmtime(HOSTCOST) >= max(os.path.getmtime(src), os.path.getmtime(LIB)):
        return HOSTCOST
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    subprocess.check_call(["gcc", "-O2", "-std=c99", "-I", INCLUDE, "-I", os.path.join(cuda, "include"), src, "-o", HOSTCOST,
                           "-L", HERE, "-lfb4", "-L", os.path.join(cuda, "lib64"), "-lcudart",
                           "-Wl,-rpath," + HERE, "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    return HOSTCOST


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv))
    print(build_hostcost(force="--force" in sys.argv))
