"""Build libprq.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
TRACE = os.environ.get("PRQ_TRACE") == "1"   # developer build: clock-stamp tracing compiled into the kernels
LIB = os.path.join(HERE, "libprq_trace.so" if TRACE else "libprq.so")
SOURCES = ["prq_api.cu", "prq_prep.cu", "prq_prep_device.cu", "prq_quant.cu", "prq_gemm.cu", "prq_gemm_prefill_pair.cu", "prq_gemm_decode.cu", "prq_peak_probe.cu", "prq_fp8.cu"]


def _newest_source_mtime() -> float:
    paths = [os.path.join(CSRC, f) for f in os.listdir(CSRC)] + [os.path.join(INCLUDE, "prq.h")]
    return max(os.path.getmtime(p) for p in paths)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source into one shared library; returns its path."""
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= _newest_source_mtime():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [
        nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
        "-Xcompiler", "-fPIC", "-shared", "-cudart", "static", "-I", INCLUDE, "-I", CSRC,
        "-o", LIB,
    ] + [os.path.join(CSRC, s) for s in SOURCES] + ["-lpthread"]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    if TRACE:
        cmd.insert(1, "-DPRQ_TRACE=1")
    subprocess.check_call(cmd)
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
