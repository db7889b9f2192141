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

CUDA_SOURCES = ["frog_index.cu", "frog_search.cu", "frog_search_lean.cu", "frog_exact.cu", "frog_build_gpu.cu"]
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
    """Compile every .cu file to an object of its own (in parallel, only those older than their
    sources or any header) and link them into libfrog.so."""
    from concurrent.futures import ThreadPoolExecutor
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(HERE, "build")
    os.makedirs(objdir, exist_ok=True)
    heads = _headers()
    jobs = []
    for name in CUDA_SOURCES:
        src = os.path.join(CSRC, name)
        obj = os.path.join(objdir, name.replace(".cu", ".o"))
        if force or _newer(obj, [src] + heads):
            jobs.append((name, [nvcc] + NVCC_FLAGS + ["-c", "-I", INCLUDE, "-I", CSRC, "-o", obj, src]))

    def run(job):
        name, cmd = job
        if verbose:
            print(" ".join(cmd))
        out = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
        return name, out.returncode, out.stdout

    failed = []
    with ThreadPoolExecutor(max_workers=max(1, len(jobs))) as ex:
        for name, rc, text in ex.map(run, jobs):
            if verbose or rc != 0:
                print(text)
            if rc != 0:
                failed.append(name)
    if failed:
        raise RuntimeError("nvcc failed on " + ", ".join(failed))
    objs = [os.path.join(objdir, n.replace(".cu", ".o")) for n in CUDA_SOURCES]
    if jobs or force or _newer(LIB_SEARCH, objs):
        cmd = [nvcc, "-shared", "-gencode", "arch=compute_100a,code=sm_100a", "-o", LIB_SEARCH] + objs
        if verbose:
            print(" ".join(cmd))
        subprocess.check_call(cmd)
    return LIB_SEARCH


def build_all(force: bool = False, verbose: bool = False):
    return build_search(force, verbose), build_builder(force, verbose)


if __name__ == "__main__":
    build_all(force="--force" in sys.argv, verbose=True)
