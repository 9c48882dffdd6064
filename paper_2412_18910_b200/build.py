"""Builds the CUDA library (sm_100a) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
LIB = os.path.join(_HERE, "libada.so")
SOURCES = [os.path.join(_HERE, "csrc", "ada.cu"), os.path.join(_HERE, "csrc", "ada_static.cu")]
DEPS = SOURCES + [os.path.join(_HERE, "csrc", "ada_kernels.cuh"), os.path.join(_HERE, "csrc", "ada_pass.cuh"),
                  os.path.join(_HERE, "csrc", "ada_ring.h"), os.path.join(_HERE, "csrc", "ada_gemm_tc.cuh"), os.path.join(_HERE, "csrc", "ada_attn_rows.cuh"), os.path.join(_ROOT, "include", "ada.h")]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/*.cu into libada.so for sm_100a (nvcc cross-compiles without a GPU)."""
    if not force and not stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
           "-Xcompiler", "-fPIC", "-I", os.path.join(_ROOT, "include"), "-I", os.path.join(_HERE, "csrc"),
           "-o", tmp] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
