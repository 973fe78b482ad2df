"""Builds libttf_b200.so (the C-ABI library) in-tree with nvcc for sm_100a.

    python -m paper_2605_07355_b200.build [--force] [--verbose]
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libttf_b200.so")
LIB_CHECKED = os.path.join(HERE, "libttf_b200_checked.so")     # the same sources with -DTTF_DEBUG (index checks)
INCLUDE = os.path.join(os.path.dirname(HERE), "include")

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared", "-I", INCLUDE,
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))
    return any(os.path.getmtime(d) > os.path.getmtime(lib) for d in deps)


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Builds the library (checked=True: the variant with device-side index checks) unless it is up to date."""
    lib = LIB_CHECKED if checked else LIB
    if not force and not stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib + f".tmp{os.getpid()}"
    cmd = ([nvcc] + NVCC_FLAGS + (["-DTTF_DEBUG"] if checked else []) + (["-Xptxas", "-v"] if verbose else [])
           + ["-o", tmp] + sources())
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, checked="--checked" in sys.argv))
