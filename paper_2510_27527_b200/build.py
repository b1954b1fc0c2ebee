"""Builds the CUDA library (sm_100a only) in-tree with nvcc: ``python -m paper_2510_27527_b200.build``."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libnvfp4_b200.so")
SOURCES = ["api.cu", "quantize.cu", "gemm.cu", "hp.cu", "noalloc.cu", "calib.cu", "osci.cu", "w16.cu", "fp6.cu"]
# measurement aids (the tensor-core issue loop): a library of their own, loaded by the benchmark only
MEASURE_LIB = os.path.join(HERE, "libnvfp4_measure.so")
MEASURE_SOURCES = ["probe.cu"]
HEADERS = ["nvfp4_device.cuh", "nvfp4_internal.h", "nvfp4_tc.cuh", os.path.join("..", "..", "include", "nvfp4.h"),
           os.path.join("..", "..", "include", "nvfp4_measure.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared", "--threads", "4",
]


def _stale(lib, sources) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(os.path.join(CSRC, f)) > t for f in sources + HEADERS)


def _compile(lib, sources, verbose):
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + os.environ.get("NVFP4_NVCC_EXTRA", "").split() + (["-Xptxas", "-v"] if verbose else []) + [os.path.join(CSRC, f) for f in sources] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False) -> str:
    for lib, sources in ((LIB, SOURCES), (MEASURE_LIB, MEASURE_SOURCES)):
        if force or _stale(lib, sources):
            _compile(lib, sources, verbose)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
