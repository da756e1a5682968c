"""Builds libfcsim.so (CUDA kernels + C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfcsim.so")
HOST_SOURCE = os.path.join(CSRC, "fcsim.cu")
KERNEL_SOURCE = os.path.join(CSRC, "fcsim_step_kernels.cu")   # compiled once per policy
N_KERNEL_POLICIES = 7
SOURCES = [HOST_SOURCE, KERNEL_SOURCE]
HEADERS = [os.path.join(CSRC, "fcsim_device.cuh"), os.path.join(ROOT, "include", "fcsim.h")]
OBJ_DIR = os.path.join(HERE, "_build")


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
    """One object per policy's step kernels plus the host file, compiled side by side, then linked.  Every object
    is a module of its own to the compiler, so the result does not depend on how many cores built it."""
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tag = os.path.splitext(os.path.basename(lib))[0]
    os.makedirs(OBJ_DIR, exist_ok=True)
    common = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC,-Wall", "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        common += ["-Xptxas", "-v"]
    common += list(extra)
    jobs = [(HOST_SOURCE, [], os.path.join(OBJ_DIR, f"{tag}_host.o"))]
    for pol in range(N_KERNEL_POLICIES):
        jobs.append((KERNEL_SOURCE, [f"-DFCSIM_KERNEL_POLICY={pol}"], os.path.join(OBJ_DIR, f"{tag}_policy{pol}.o")))

    def one(job):
        src, defs, obj = job
        return subprocess.run(common + defs + ["-c", src, "-o", obj], capture_output=True, text=True)

    with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as pool:
        results = list(pool.map(one, jobs))
    for (src, defs, obj), r in zip(jobs, results):
        if r.stdout or r.stderr:
            sys.stderr.write(f"[{os.path.basename(obj)}]\n{r.stdout}{r.stderr}")
        if r.returncode != 0:
            raise subprocess.CalledProcessError(r.returncode, r.args)
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", lib + ".tmp"]
                   + [obj for _, _, obj in jobs], check=True)
    os.replace(lib + ".tmp", lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, checked="--checked" in sys.argv))
