"""Builds the CUDA shared library in-tree with nvcc (sm_100a only)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "liblazyev.so")
LIB_DEBUG = os.path.join(HERE, "liblazyev_debug.so")     # the same sources with -DLAZYEV_DEBUG_BOUNDS
SOURCES = ["api.cu", "decode.cu", "cache_ops.cu", "evict.cu", "prompt.cu"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    built = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(HERE, "..", "include", "lazyev.h"))
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile csrc/*.cu into liblazyev.so (or, with debug_bounds, into liblazyev_debug.so with every
    kernel index range-checked) next to this file; returns its path."""
    lib = LIB_DEBUG if debug_bounds else LIB
    if not force and not needs_build(lib):
        return lib
    cmd = [_nvcc(), "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
           "-Xptxas", "-v", "-Xcompiler", "-fPIC", "-shared", "-o", lib]
    if debug_bounds:
        cmd.append("-DLAZYEV_DEBUG_BOUNDS")
    cmd += [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    with open(os.path.join(HERE, "build_debug.log" if debug_bounds else "build.log"), "w") as f:
        f.write(" ".join(cmd) + "\n" + res.stdout + res.stderr)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed; see build.log")
    if verbose:
        sys.stderr.write(res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose=True, debug_bounds="--debug-bounds" in sys.argv))
