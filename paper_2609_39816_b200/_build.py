"""Build libfmm_b200.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
_INC = os.path.join(os.path.dirname(_HERE), "include")
LIB_PATH = os.path.join(_HERE, "libfmm_b200.so")
SOURCES = ["api.cu", "kernels_stream.cu", "gemm_tcgen05.cu", "noalloc.cu", "int8_path.cu", "int8_control.cu", "rotate.cu", "repairs.cu", "scheme_host.cpp"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)] + [os.path.join(_INC, "fmm_b200.h")]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "--threads", "0",
           "-Xcompiler", "-fPIC", "-shared", "-I", _INC, "-I", _CSRC, "-o", LIB_PATH]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += [os.path.join(_CSRC, s) for s in SOURCES]
    subprocess.run(cmd, check=True)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
