"""Builds libfcsim.so (CUDA kernels + C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfcsim.so")
SOURCES = [os.path.join(CSRC, "fcsim.cu")]
HEADERS = [os.path.join(CSRC, "fcsim_device.cuh"), os.path.join(ROOT, "include", "fcsim.h")]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


LIB_CHECKED = os.path.join(HERE, "libfcsim_checked.so")


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile if the sources are newer than the library; returns the library path.
    ``checked`` builds the index-checked diagnostic variant (libfcsim_checked.so)."""
    if checked:
        if not force and not _stale(LIB_CHECKED):
            return LIB_CHECKED
        return _compile(LIB_CHECKED, verbose, ["-DFCSIM_CHECKED"])
    if not force and not _stale():
        return LIB
    return _compile(LIB, verbose, [])


def _compile(lib: str, verbose: bool, extra) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    # -split-compile 0: the kernels (one instantiation per policy and variant) are optimised on all host cores
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-split-compile", "0",
           "-Xcompiler", "-fPIC,-Wall", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += list(extra) + SOURCES + ["-o", lib + ".tmp"]
    subprocess.run(cmd, check=True)
    os.replace(lib + ".tmp", lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
