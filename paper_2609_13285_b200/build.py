"""Builds libgva.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libgva.so")
PROBE_LIB = os.path.join(HERE, "libgva_probe.so")      # the benchmark's read-only streaming probe (not part of the C ABI)
SOURCES = ["gva_api.cu"]
HEADERS = ["gva_common.cuh", "gva_small_kernels.cuh", "gva_decode_fma.cuh", "gva_decode_mma.cuh", "gva_decode_fp8.cuh", "gva_prefill.cuh", "gva_project.cuh",
           os.path.join("..", "..", "include", "gva.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    for f in SOURCES + HEADERS:
        p = os.path.join(CSRC, f)
        if os.path.exists(p) and os.path.getmtime(p) > t:
            return True
    return False


def build(force: bool = False, verbose: bool = False) -> str:
    if os.environ.get("GVA_LIBRARY"):      # a prebuilt library was named explicitly: nothing to do
        return os.environ["GVA_LIBRARY"]
    if not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
             "-Xcompiler", "-fPIC"]
    if os.path.exists(os.path.join(CSRC, "gva_decode_mma.cuh")):
        flags.append("-DGVA_WITH_MMA")
    flags += os.environ.get("GVA_EXTRA_NVCC_FLAGS", "").split()   # e.g. tuning macros such as -DGVA_MMA_WPG64=1
    if verbose:
        flags += ["-Xptxas", "-v"]
    cmd = [nvcc] + flags + [os.path.join(CSRC, s) for s in SOURCES] + ["-o", LIB]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed building libgva.so")
    return LIB


def build_probe(force: bool = False) -> str:
    """Builds the benchmark's read-only streaming probe (csrc/stream_probe.cu) into its own shared object."""
    src = os.path.join(CSRC, "stream_probe.cu")
    if not force and os.path.exists(PROBE_LIB) and os.path.getmtime(PROBE_LIB) >= os.path.getmtime(src):
        return PROBE_LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared", "-Xcompiler", "-fPIC",
           src, "-o", PROBE_LIB]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        sys.stderr.write(res.stdout + res.stderr)
        raise RuntimeError("nvcc failed building libgva_probe.so")
    return PROBE_LIB


if __name__ == "__main__":
    build_probe(force=True)
    print(build(force=True, verbose="-v" in sys.argv))
