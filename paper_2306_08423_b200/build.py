"""Builds the engine's shared library in-tree with nvcc for sm_100a.

``python -m paper_2306_08423_b200.build`` or ``build()``.  Objects go to ``_build/`` next
to the sources; the library is ``paper_2306_08423_b200/libdistsim.so``.
"""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_PKG, "csrc")
_OBJ = os.path.join(_PKG, "_build")
LIB = os.path.join(_PKG, "libdistsim.so")
BENCH_LIB = os.path.join(_PKG, "libdistsim_bench.so")       # measurement probes, a library of their own
SOURCES = ["distsim_api.cu", "setup_kernels.cu", "eval_kernels.cu", "select_kernels.cu", "emit_kernels.cu"]
BENCH_SOURCES = ["probe_kernels.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _newest_header() -> float:
    hdrs = [os.path.join(_SRC, f) for f in os.listdir(_SRC) if f.endswith((".h", ".cuh"))]
    inc = os.path.join(os.path.dirname(_PKG), "include")
    hdrs += [os.path.join(inc, f) for f in os.listdir(inc) if f.endswith(".h")]
    return max(os.path.getmtime(h) for h in hdrs)


def _build_library(lib: str, sources, force: bool, verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    os.makedirs(_OBJ, exist_ok=True)
    hdr_time = _newest_header()
    objs, rebuilt = [], False
    for src in sources:
        s = os.path.join(_SRC, src)
        o = os.path.join(_OBJ, src.replace(".cu", ".o"))
        objs.append(o)
        if force or not os.path.exists(o) or os.path.getmtime(o) < max(os.path.getmtime(s), hdr_time):
            cmd = [nvcc, *NVCC_FLAGS, "-c", s, "-o", o]
            r = subprocess.run(cmd, capture_output=True, text=True)
            if verbose or r.returncode:
                sys.stderr.write(r.stdout + r.stderr)
            if r.returncode:
                raise RuntimeError(f"nvcc failed on {src}")
            with open(o + ".ptxas.txt", "w") as f:
                f.write(r.stderr)
            rebuilt = True
    if rebuilt or not os.path.exists(lib):
        cmd = [nvcc, "-shared", "-o", lib, *objs, "-cudart", "static"]
        r = subprocess.run(cmd, capture_output=True, text=True)
        if r.returncode:
            sys.stderr.write(r.stdout + r.stderr)
            raise RuntimeError("link failed")
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    """Builds the engine's library and the benchmark's probe library; returns the engine's path."""
    _build_library(BENCH_LIB, BENCH_SOURCES, force, verbose)
    return _build_library(LIB, SOURCES, force, verbose)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True))
