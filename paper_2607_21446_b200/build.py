"""Build libkroquant.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

``python -m paper_2607_21446_b200.build`` or :func:`build`.  nvcc cross-compiles
without a GPU, so this also runs on a CPU-only box.
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libkroquant.so")
SOURCES = [os.path.join(CSRC, "kroquant_api.cu")]
HEADERS = [os.path.join(CSRC, n) for n in ("kq_common.cuh", "kq_stream.cuh", "kq_umma.cuh", "kq_gemm.cuh", "kq_gemm2.cuh", "kq_gemm_fp4.cuh", "kq_gemm_fp4_pair.cuh", "kq_calib.cuh",
                                               "kroquant_calib_api.cuh")] + [
    os.path.join(os.path.dirname(PKG), "include", "kroquant.h")]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-lineinfo",
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-shared", "-Xcompiler", "-fPIC",
    "-Xptxas", "-v",
]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS + [os.path.abspath(__file__)])


LIB_TIMELINE = os.path.join(PKG, "libkroquant_timeline.so")


def build_timeline(force: bool = False) -> str:
    """The same library with per-CTA timeline marks compiled in (-DKQ_TIMELINE): a measuring aid for
    `bench.py --timeline`, never loaded by the product path.  Rebuilt when any source is newer."""
    if not force and os.path.exists(LIB_TIMELINE):
        t = os.path.getmtime(LIB_TIMELINE)
        if not any(os.path.getmtime(p) > t for p in SOURCES + HEADERS + [os.path.abspath(__file__)]):
            return LIB_TIMELINE
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    res = subprocess.run([nvcc] + NVCC_FLAGS + ["-DKQ_TIMELINE", "-o", LIB_TIMELINE] + SOURCES, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libkroquant_timeline.so")
    return LIB_TIMELINE


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc] + NVCC_FLAGS + ["-o", LIB] + SOURCES
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libkroquant.so")
    return LIB


if __name__ == "__main__":
    if "--timeline" in sys.argv[1:]:
        print(build_timeline(force=True))
    else:
        print(build(force=True, verbose=True))
