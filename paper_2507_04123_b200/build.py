"""Builds libemc2_bridge.so (CUDA, sm_100a only) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libemc2_bridge.so")
SOURCES = ["bridge.cu", "voxelize.cu", "project_gather.cu", "route_dispatch.cu", "voxel_image.cu", "occlusion.cu", "rulebook.cu", "dedup_arms.cu"]
HEADERS = [os.path.join(CSRC, "bridge_internal.cuh"), os.path.join(ROOT, "include", "emc2_bridge.h")]


def nvcc_command(verbose_ptxas: bool = False):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
           "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"), "-I", CSRC,
           "--fmad=true", "-o", LIB]
    if verbose_ptxas:
        cmd += ["-Xptxas", "-v"]
    return cmd + [os.path.join(CSRC, s) for s in SOURCES]


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose_ptxas: bool = False) -> str:
    if force or verbose_ptxas or needs_build():
        subprocess.run(nvcc_command(verbose_ptxas), check=True)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose_ptxas="-v" in sys.argv))
