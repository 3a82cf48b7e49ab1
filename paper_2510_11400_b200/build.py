"""Build step: compile the CUDA library for sm_100a into the package directory."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libfh_sm100a.so")
SOURCES = [os.path.join(CSRC, "fh.cu"), os.path.join(CSRC, "fh_plan.cpp")]
DEPS = SOURCES + [os.path.join(CSRC, f) for f in ("fh_device.cuh", "fh_channel.cuh", "fh_compress.cuh", "fh_decompress.cuh")] + \
    [os.path.join(os.path.dirname(HERE), "include", "fh.h")]


def nvcc_cmd(extra=()):
    return ["nvcc", "-std=c++17", "-O3", "-lineinfo", "-gencode", "arch=compute_100a,code=sm_100a",
            "-Xcompiler", "-fPIC", "-shared", "--fmad=false", "-o", LIB, *extra, *SOURCES]


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile when the library is missing or older than a source.  Returns the library path."""
    if not force and os.path.exists(LIB):
        t = os.path.getmtime(LIB)
        if all(os.path.getmtime(d) <= t for d in DEPS):
            return LIB
    cmd = nvcc_cmd(["-Xptxas", "-v"] if verbose else [])
    r = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(r.stderr)
    if r.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + r.stderr)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
