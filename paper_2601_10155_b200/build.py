"""Builds liblookat.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2601_10155_b200.build [--force] [--verbose] [--debug]

nvcc cross-compiles without a GPU.  The library links the static CUDA
runtime, so loading it needs no CUDA libraries on the search path.
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(PKG, "liblookat.so")
LIB_DEBUG = os.path.join(PKG, "liblookat_debug.so")
SOURCES = ["api.cu", "attend.cu", "attend_multi.cu", "attend_static.cu", "attend_pqv.cu", "prefill.cu", "prefill_umma.cu", "lut.cu", "encode.cu", "encode_mma.cu", "fit.cu", "probe.cu", "linear_umma.cu", "gpt2_ops.cu", "gpt2.cu"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compiles every kernel for sm_100a; returns the path of the shared library.  debug: the build whose attend kernels
    check every code they read (-DLOOKAT_DEBUG), as liblookat_debug.so."""
    lib = LIB_DEBUG if debug else LIB
    if not force and not _stale(lib):
        return lib
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "--threads", "0", "-O3", "-std=c++20", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-cudart", "static", "-I", INCLUDE, "-I", CSRC]
    if debug:
        cmd += ["-DLOOKAT_DEBUG"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        if os.path.exists(tmp):
            os.remove(tmp)
        raise RuntimeError("nvcc failed building liblookat.so")
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv, debug="--debug" in sys.argv))
