"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libgws.so")
SOURCES = [os.path.join(CSRC, "gws_api.cu")]
HEADERS = [os.path.join(CSRC, "gws_kernels.cuh"), os.path.join(CSRC, "gws_math.cuh"), os.path.join(CSRC, "gws_gemm.cuh"), os.path.join(CSRC, "gws_probe.cuh"), os.path.join(CSRC, "gws_compare.cuh"), os.path.join(CSRC, "gws_gemm_cluster.cuh"), os.path.join(CSRC, "gws_gemm_wide.cuh"), os.path.join(CSRC, "gws_train.cuh"),
           os.path.join(INCLUDE, "gws.h")]

# -fmad=false: the add-then-cast path must round the multiply and the add separately.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-fmad=false",
              "-shared", "-Xcompiler", "-fPIC", "-I" + INCLUDE, "-I" + CSRC]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


CHECK_LIB_PATH = os.path.join(_PKG, "libgws_check.so")   # the self-checking variant (-DGWS_SELF_CHECK)


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    built = os.path.getmtime(path)
    return any(os.path.getmtime(p) > built for p in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False, self_check: bool = False) -> str:
    """Compile ``libgws.so`` (or the self-checking ``libgws_check.so``) next to the package if it is missing
    or older than its sources."""
    path = CHECK_LIB_PATH if self_check else LIB_PATH
    if force or is_stale(path):
        tmp = path + ".tmp.%d" % os.getpid()
        cmd = [_nvcc(), *NVCC_FLAGS, *(["-DGWS_SELF_CHECK"] if self_check else []),
               *(["-Xptxas", "-v"] if verbose else []), "-o", tmp, *SOURCES]
        subprocess.run(cmd, check=True)
        os.replace(tmp, path)
    return path


if __name__ == "__main__":
    print(build(force=True, verbose=True))
