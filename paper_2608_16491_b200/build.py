"""Compile the two in-tree shared libraries.

``libfrog.so``       the search library (CUDA, sm_100a only), declared in include/frog.h
``libfrog_build.so`` the host index builder, declared in include/frog_build.h

Run as ``python -m paper_2608_16491_b200.build``; nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB_SEARCH = os.path.join(HERE, "libfrog.so")
LIB_BUILD = os.path.join(HERE, "libfrog_build.so")

CUDA_SOURCES = ["frog_index.cu", "frog_search.cu", "frog_exact.cu", "frog_build_gpu.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--fmad=false", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _newer(target: str, sources) -> bool:
    if not os.path.exists(target):
        return True
    t = os.path.getmtime(target)
    return any(os.path.getmtime(s) > t for s in sources)


def _headers():
    hs = [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    hs += [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".h", ".cuh"))]
    return hs


def build_builder(force: bool = False, verbose: bool = False) -> str:
    src = os.path.join(CSRC, "frog_build.cpp")
    if force or _newer(LIB_BUILD, [src] + _headers()):
        cmd = ["g++", "-std=c++17", "-O3", "-mavx2", "-mfma", "-ffp-contract=off", "-fopenmp",
               "-shared", "-fPIC", "-I", INCLUDE, "-o", LIB_BUILD, src]
        if verbose:
            print(" ".join(cmd))
        subprocess.check_call(cmd)
    return LIB_BUILD


def build_search(force: bool = False, verbose: bool = False) -> str:
    srcs = [os.path.join(CSRC, s) for s in CUDA_SOURCES]
    if force or _newer(LIB_SEARCH, srcs + _headers()):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        cmd = [nvcc] + NVCC_FLAGS + ["-shared", "-I", INCLUDE, "-I", CSRC, "-o", LIB_SEARCH] + srcs
        if verbose:
            print(" ".join(cmd))
        out = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        if verbose or out.returncode != 0:
            print(out.stdout)
        if out.returncode != 0:
            raise RuntimeError("nvcc failed")
    return LIB_SEARCH


def build_all(force: bool = False, verbose: bool = False):
    return build_search(force, verbose), build_builder(force, verbose)


if __name__ == "__main__":
    build_all(force="--force" in sys.argv, verbose=True)
