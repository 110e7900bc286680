"""Builds libef.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libef.so")
DEBUG_LIB = os.path.join(PKG, "libef_debug.so")      # the checked build (-DEF_DEBUG)
SOURCES = [os.path.join(CSRC, n) for n in ("ef_lib.cu", "ef_vote.cu", "ef_topk.cu")]
DEPS = SOURCES + [os.path.join(CSRC, "ef_kernels.cuh"), os.path.join(CSRC, "ef_internal.h"),
                  os.path.join(ROOT, "include", "ef.h")]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-fmad=false",                      # no implicit contraction: every fused op is explicit
    "-Xcompiler", "-fPIC", "-shared",
    "-ldl",                             # NVTX (header-only) looks for an attached tool with dlopen
]


def nvcc_path() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds libef.so, or with debug=True the checked build libef_debug.so (every kernel
    validates its work item against the problem's sizes)."""
    lib = DEBUG_LIB if debug else LIB
    if not force and os.path.exists(lib):
        newest = max(os.path.getmtime(p) for p in DEPS)
        if os.path.getmtime(lib) >= newest:
            return lib
    cmd = ([nvcc_path()] + NVCC_FLAGS + (["-DEF_DEBUG"] if debug else [])
           + (["-Xptxas", "-v"] if verbose else []) + ["-o", lib] + SOURCES)
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
