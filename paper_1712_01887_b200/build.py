"""Build the CUDA library in-tree: nvcc, sm_100a only."""
from __future__ import annotations

import fcntl
import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(_HERE)
SRC = os.path.join(_HERE, "csrc", "dgc.cu")
LIB = os.path.join(_HERE, "libdgc.so")
INCLUDE = os.path.join(ROOT, "include")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def _fresh(deps) -> bool:
    return os.path.exists(LIB) and all(os.path.getmtime(LIB) >= os.path.getmtime(d) for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    deps = [SRC, os.path.join(_HERE, "csrc", "dgc_kernels.cuh"), os.path.join(INCLUDE, "dgc.h")]
    if not force and _fresh(deps):
        return LIB
    # several ranks of one job may get here at once: one of them compiles (into a file of its
    # own, moved into place when complete), the others wait for the lock and find the result
    with open(LIB + ".lock", "w") as lock:
        fcntl.flock(lock, fcntl.LOCK_EX)
        try:
            if not force and _fresh(deps):
                return LIB
            nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
            extra = os.environ.get("NVCC_EXTRA_FLAGS", "").split()   # e.g. -D switches of variants
            tmp = f"{LIB}.{os.getpid()}.tmp"
            cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + \
                  ["-I", INCLUDE, "-o", tmp, SRC]
            try:
                subprocess.run(cmd, check=True)
                os.replace(tmp, LIB)
            finally:
                if os.path.exists(tmp):
                    os.remove(tmp)
        finally:
            fcntl.flock(lock, fcntl.LOCK_UN)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in __import__("sys").argv))
