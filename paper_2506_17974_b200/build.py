"""Builds liblqsgd.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
SOURCES = [os.path.join(_HERE, "csrc", f) for f in ("lqsgd_kernels.cu", "lqsgd_api.cu", "lqsgd_noalloc.cu", "lqsgd_stream.cu", "lqsgd_tc.cu", "lqsgd_resident.cu", "lqsgd_stats.cu")]
HEADERS = [os.path.join(_HERE, "csrc", "lqsgd_dev.h"), os.path.join(_HERE, "csrc", "lqsgd_stream_common.cuh"),
           os.path.join(_HERE, "csrc", "lqsgd_factor.cuh"), os.path.join(_HERE, "csrc", "lqsgd_stats.h"),
           os.path.join(os.path.dirname(_HERE), "include", "lqsgd.h")]
TARGET = os.path.join(_HERE, "liblqsgd.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "shared", "-ldl"]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def is_stale() -> bool:
    if not os.path.exists(TARGET):
        return True
    t = os.path.getmtime(TARGET)
    return any(os.path.getmtime(s) > t for s in SOURCES + HEADERS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    if not force and not is_stale():
        return TARGET
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + SOURCES + ["-o", TARGET]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return TARGET
