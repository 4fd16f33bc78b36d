"""Compiles the CUDA sources under csrc/ into libmona.so (sm_100a only), next to this file."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libmona.so")
LIB_DEBUG = os.path.join(HERE, "libmona_debug.so")      # -DMONA_DEBUG: kernels check their own indices
LIB_TRACE = os.path.join(HERE, "libmona_trace.so")      # -DMONA_TRACE: the Newton-Schulz kernel accounts for its waits
SOURCES = ["mona_api.cu", "elementwise.cu", "ns_fp32.cu", "ns_tc.cu"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the library cannot be built")
    return exe


def needs_build(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(HERE, "..", "include", "mona.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False, trace: bool = False) -> str:
    if debug and trace:
        raise ValueError("one build variant at a time")
    lib = LIB_DEBUG if debug else LIB_TRACE if trace else LIB
    if not force and not needs_build(lib):
        return lib
    defines = ["-DMONA_DEBUG"] if debug else ["-DMONA_TRACE"] if trace else []
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-o", lib] + defines + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        sys.stderr.write(res.stderr)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv, trace="--trace" in sys.argv))
