"""Builds ``libsd2.so`` (sm_100a) in-tree from ``csrc/``.

``python -m paper_2504_08838_b200.build`` or ``build.build()``.  ``SD2_CHECKED=1`` in the environment builds
the checked variant: the tensor-core kernel verifies every record offset and store address it derives
from compressed data, records a violation in the device error word (``sd2_stream_check`` then returns
``SD2_ERR_CORRUPT``) and skips the access.  nvcc cross-compiles
without a GPU; the shared object sits next to this file so that it travels with the
source tree and is the one the binding loads.
"""

from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libsd2.so")
SOURCES = ["sd2_api.cu"]
DEPS = ["sd2_api.cu", "sd2_kernels.cuh", "sd2_mma_kernel.cuh", "sd2_glue.cuh", "sd2_format.hpp", "sd2_format_mma.hpp", os.path.join("..", "..", "include", "sd2.h")]


def nvcc_path() -> str:
    cand = os.environ.get("NVCC") or os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def up_to_date() -> bool:
    if not os.path.exists(LIB):
        return False
    t = os.path.getmtime(LIB)
    return all(os.path.getmtime(os.path.join(CSRC, d)) <= t for d in DEPS)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB
    tmp = LIB + ".%d.tmp" % os.getpid()
    cmd = [nvcc_path(), "-shared", "-o", tmp,
           "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC,-fopenmp,-O3,-Wall,-Wno-unknown-pragmas",
           "-Xptxas", "-v" if verbose else "-O3",
           ] + (["-DSD2_CHECKED"] if os.environ.get("SD2_CHECKED") == "1" else []) + [
           ] + [os.path.join(CSRC, s) for s in SOURCES] + ["-lgomp", "-ldl"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libsd2.so")
    os.replace(tmp, LIB)
    return LIB


if __name__ == "__main__":
    print(build(force=True, verbose="-v" in sys.argv))
