"""Builds the CUDA library in-tree: ``csrc/*.cu`` -> ``libkvsched.so`` (sm_100a only)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB = os.path.join(_HERE, "libkvsched.so")
LIB_CHECKED = os.path.join(_HERE, "libkvsched_checked.so")
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "-cudart", "shared"]


UNITS = ["api.cu", "argmin_static.cu", "probe.cu"]          # translation units; the .cuh files are included by api.cu


def sources():
    return sorted(os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cu", ".cuh"))) + \
        [os.path.join(os.path.dirname(_HERE), "include", "kvsched.h")]


def stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(s) > t for s in sources())


def build(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """``checked``: the checked build (-DKVSCHED_CHECKED -> libkvsched_checked.so), in which every
    index a kernel computes is range-checked before use."""
    lib = LIB_CHECKED if checked else LIB
    if force or stale(lib):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = lib + ".%d.tmp" % os.getpid()
        cmd = [nvcc] + NVCC_FLAGS + (["-DKVSCHED_CHECKED"] if checked else []) + (["-Xptxas", "-v"] if verbose else []) + \
            [os.path.join(CSRC, f) for f in UNITS] + ["-o", tmp]
        subprocess.check_call(cmd)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose=True))
    if "--checked" in sys.argv[1:]:
        print(build(force=True, checked=True))
