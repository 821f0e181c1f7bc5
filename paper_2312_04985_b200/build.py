"""Compile the CUDA library in-tree for sm_100a with nvcc (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
SOURCES = [os.path.join(_PKG, "csrc", f) for f in ("api.cu", "sparq_decode.cu", "sparq_decode_pipe.cu", "sparq_decode_wide.cu", "sparq_decode_grouped.cu",
                                                     "dense_decode.cu", "cache.cu")]
HEADERS = [os.path.join(_ROOT, "include", "sparq.h")] + [os.path.join(_PKG, "csrc", f)
                                                        for f in ("common.cuh", "decode_common.cuh", "kernels.h")]
LIB_PATH = os.path.join(_PKG, "libsparq_b200.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "static"]


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Build ``libsparq_b200.so`` next to this file if it is missing or stale; return its path."""
    if force or needs_build():
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        if not os.path.exists(nvcc):
            nvcc = "nvcc"
        tmp = LIB_PATH + ".%d.tmp" % os.getpid()
        cmd = [nvcc, *NVCC_FLAGS, "-I", os.path.join(_ROOT, "include"), "-o", tmp, *SOURCES]
        if verbose:
            cmd.insert(1, "-Xptxas=-v")
        subprocess.run(cmd, check=True)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
