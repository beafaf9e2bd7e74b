"""Builds librt3d.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

Run as `python -m paper_2007_09835_b200.build` or call build().  The shared object is
written next to this file so it travels with the source tree; nothing is installed.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "librt3d.so")
SOURCES = ["api.cu", "pack.cpp", "simt_kernels.cu", "umma_conv.cu", "umma_conv_pair.cu", "umma_conv_halo.cu", "umma_conv_st.cu", "umma_conv_sub.cu", "umma_smallc.cu", "reweight.cu", "debug_poison.cu"]
HEADERS = ["kernels.h", "rt3d_internal.h", "umma_common.cuh", "umma_pair.cuh", "pdl.cuh", "tile_consts.h"]
MICROBENCH = os.path.join(HERE, "rt3d_microbench")       # stand-alone instruction-rate microbenchmarks


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(ROOT, "include", "rt3d.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "static",
           "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", tmp] + [os.path.join(CSRC, f) for f in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


def build_microbench(force: bool = False) -> str:
    """Compiles csrc/microbench_mma.cu into the stand-alone program `rt3d_microbench` (prints a markdown report)."""
    src = os.path.join(CSRC, "microbench_mma.cu")
    deps = [src, os.path.join(CSRC, "umma_common.cuh"), os.path.join(CSRC, "umma_pair.cuh")]
    if not force and os.path.exists(MICROBENCH) and all(os.path.getmtime(d) <= os.path.getmtime(MICROBENCH) for d in deps):
        return MICROBENCH
    tmp = MICROBENCH + f".tmp{os.getpid()}"
    subprocess.check_call([_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                           "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", tmp, src])
    os.replace(tmp, MICROBENCH)
    return MICROBENCH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    if "--microbench" in sys.argv:
        print(build_microbench(force="--force" in sys.argv))
