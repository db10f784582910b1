"""Build the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
LIB = os.path.join(_PKG, "libtahq.so")
SOURCES = [os.path.join(_CSRC, "tahq_api.cu")]
_DEPS = [os.path.join(_CSRC, f) for f in ("tahq_api.cu", "tahq_kernels.cuh", "tahq_stream.cuh", "tahq_device.cuh", "qnaive.cuh")] + [
    os.path.join(os.path.dirname(_PKG), "include", "tahq.h")]

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-fmad=false",            # only the fused multiply-adds written in the source are fused
    "-Xcompiler", "-fPIC", "-shared",
]


def stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(d) > t for d in _DEPS if os.path.exists(d))


def build(force: bool = False, verbose: bool = False) -> str:
    if force or stale():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = LIB + f".tmp{os.getpid()}"
        cmd = [nvcc, *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", tmp, *SOURCES]
        subprocess.run(cmd, check=True, cwd=_CSRC)
        os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose=True))
