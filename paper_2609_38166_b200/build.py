"""Builds the C-ABI CUDA library in-tree: ``paper_2609_38166_b200/liblq.so`` for sm_100a.

``-fmad=false`` is part of the numerics contract: products are fused with additions only where the
kernels write fmaf(), which is what makes results reproducible bit for bit.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "liblq.so")
# the same library with per-CTA time stamps compiled in (a development aid: bench.py --timeline reads them)
LIB_STAMPS = os.path.join(HERE, "liblq_stamps.so")
SOURCES = ["lq_api.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-fmad=false", "-std=c++17",
              "--shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v"]


def _newest_source() -> float:
    inc = os.path.join(os.path.dirname(HERE), "include")
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(inc, f) for f in os.listdir(inc)]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False, stamps: bool = False) -> str:
    """Compile if the library is missing or older than its sources; returns the library path.
    ``stamps``: the variant with the time stamps (-DLQ_TIMING -DLQ_STAMPS_ONLY) instead of the product."""
    LIB = LIB_STAMPS if stamps else globals()["LIB"]
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    extra = ["-DLQ_TIMING", "-DLQ_STAMPS_ONLY"] if stamps else []
    cmd = [nvcc, *NVCC_FLAGS, *extra, *[os.path.join(CSRC, s) for s in SOURCES], "-o", LIB + ".tmp"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed")
    if verbose:
        sys.stderr.write(res.stderr)
    os.replace(LIB + ".tmp", LIB)
    return LIB


if __name__ == "__main__":
    stamps_ = "--stamps" in sys.argv[1:]
    print(build(force=True, verbose=True, stamps=stamps_))
