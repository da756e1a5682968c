"""TEST INFRASTRUCTURE: compiles the CPU checker (fcsim_oracle.cpp) into a shared object with g++."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "fcsim_oracle.cpp")
LIB = os.path.join(HERE, "libfcsim_oracle.so")


def build(force: bool = False, sanitize: bool = False) -> str:
    """Build (if stale) and return the path of the checker's shared object."""
    lib = LIB if not sanitize else os.path.join(HERE, "libfcsim_oracle_asan.so")
    if not force and os.path.exists(lib) and os.path.getmtime(lib) >= os.path.getmtime(SRC):
        return lib
    cmd = ["g++", "-std=c++17", "-O2", "-Wall", "-Wextra", "-shared", "-fPIC", SRC, "-o", lib + ".tmp"]
    if sanitize:
        cmd[3:3] = ["-g", "-fsanitize=address,undefined", "-fno-sanitize-recover=all"]
    subprocess.run(cmd, check=True)
    os.replace(lib + ".tmp", lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv))
