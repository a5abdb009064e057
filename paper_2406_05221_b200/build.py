"""In-tree build of the native sources: the CUDA library (nvcc, sm_100a) and the generator."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
CUDA_SRC = os.path.join(_HERE, "csrc", "gcaps_rta.cu")
CUDA_SRCS = [CUDA_SRC, os.path.join(_HERE, "csrc", "gcaps_rta_any.cu"),
             os.path.join(_HERE, "csrc", "gcaps_gpu_priority.cu"),
             os.path.join(_HERE, "csrc", "gcaps_igen.cu"), os.path.join(_HERE, "csrc", "gcaps_diag.cu")]
CUDA_DEPS = CUDA_SRCS + [os.path.join(_HERE, "csrc", "rta_common.cuh"), os.path.join(_HERE, "csrc", "igen.h")]
CUDA_LIB = os.path.join(_HERE, "libgcaps_rta.so")
HEADER = os.path.join(os.path.dirname(_HERE), "include", "gcaps_rta.h")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "--threads", "5"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def cuda_lib_is_stale() -> bool:
    if not os.path.exists(CUDA_LIB):
        return True
    m = os.path.getmtime(CUDA_LIB)
    return any(m < os.path.getmtime(f) for f in CUDA_DEPS + [HEADER])


def build_cuda(force: bool = False, verbose: bool = False) -> str:
    """Compiles the CUDA sources of csrc/ for sm_100a into libgcaps_rta.so beside this file."""
    if force or cuda_lib_is_stale():
        tmp = CUDA_LIB + ".%d.tmp" % os.getpid()
        if os.path.exists(CUDA_LIB):
            os.remove(CUDA_LIB)  # a failed build must not leave an older library behind
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + CUDA_SRCS
        subprocess.check_call(cmd)
        os.replace(tmp, CUDA_LIB)
    return CUDA_LIB


def build_all(force: bool = False) -> None:
    from . import taskgen
    taskgen.build_taskgen(force)
    build_cuda(force)


if __name__ == "__main__":
    build_all(force="--force" in sys.argv)
    print(CUDA_LIB)
