"""Build the CUDA library in-tree for sm_100a:  python -m paper_2410_15240_b200.build"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfastrack.so")
SOURCES = [os.path.join(CSRC, "fastrack.cu")]
DEPS = SOURCES + [os.path.join(CSRC, "fastrack_device.cuh"), os.path.join(CSRC, "fastrack_keysetup.h"), os.path.join(CSRC, "fastrack_plan.h"),
                  os.path.join(os.path.dirname(HERE), "include", "fastrack.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC,-fvisibility=hidden"]


def _compile(target: str, sources, deps, force: bool, verbose: bool) -> None:
    stale = (not os.path.exists(target)) or any(os.path.getmtime(target) < os.path.getmtime(d) for d in deps)
    if force or stale:
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = target + f".{os.getpid()}.tmp"
        cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + list(sources)
        subprocess.check_call(cmd)
        os.replace(tmp, target)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libfastrack.so if it is missing or older than its sources.  Returns its path."""
    _compile(LIB, SOURCES, DEPS, force, verbose)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
