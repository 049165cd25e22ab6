"""Builds the CUDA library in-tree with nvcc for sm_100a (no torch headers involved)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libblockserve.so")
SOURCES = ["engine.cu", "sched_index.cu", "elementwise.cu", "gemm_tcgen05.cu", "attention.cu", "attention_tc.cu",
           "rope_static.cu"]
NVCC_FLAGS = ["-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _newer(a: str, b: str) -> bool:
    return not os.path.exists(b) or os.path.getmtime(a) > os.path.getmtime(b)


LIB_DEBUG = os.path.join(HERE, "libblockserve_dbg.so")


def build(force: bool = False, verbose: bool = False, debug=None) -> str:
    """debug=True builds libblockserve_dbg.so: the same sources with -DBS_BOUNDS_CHECK (index checks in the gather /
    scatter and index kernels).  debug=None follows the environment (BS_DEBUG_LIB), like the binding does."""
    if debug is None:
        debug = bool(os.environ.get("BS_DEBUG_LIB"))
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    lib = LIB_DEBUG if debug else LIB
    flags = NVCC_FLAGS + (["-DBS_BOUNDS_CHECK"] if debug else [])
    suffix = ".dbg.o" if debug else ".o"
    headers = [os.path.join(CSRC, f) for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))]
    headers.append(os.path.join(os.path.dirname(HERE), "include", "blockserve.h"))
    objs = []
    for src in SOURCES:
        s = os.path.join(CSRC, src)
        o = os.path.join(CSRC, src.replace(".cu", suffix))
        if force or _newer(s, o) or any(_newer(h, o) for h in headers):
            cmd = [nvcc, *flags, "-c", s, "-o", o]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if verbose or r.returncode != 0:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode != 0:
                raise RuntimeError(f"nvcc failed on {src}")
        objs.append(o)
    if force or any(_newer(o, lib) for o in objs):
        r = subprocess.run([nvcc, "-shared", "-o", lib, *objs, "-lcudart"], capture_output=True, text=True)
        if r.returncode != 0:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
