"""Build the C-ABI shared library (sm_100a only) in-tree with nvcc."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_PKG, "csrc")
LIB_DIR = os.path.join(_PKG, "lib")
LIB_PATH = os.environ.get("FLUXBIN_LIB") or os.path.join(LIB_DIR, "libfluxbin.so")
SOURCES = ["fluxbin_api.cu", "fluxbin_pack.cpp", "fluxbin_pack_device.cu", "fluxbin_noalloc.cu", "fluxbin_rc_decomp.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC,-fopenmp", "-shared"]


def _sources():
    return [os.path.join(CSRC, s) for s in SOURCES if os.path.exists(os.path.join(CSRC, s))]


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps.append(os.path.join(os.path.dirname(_PKG), "include", "fluxbin.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile libfluxbin.so if it is missing or older than its sources; returns its path."""
    if not force and os.environ.get("FLUXBIN_LIB") and os.path.exists(LIB_PATH):
        return LIB_PATH          # an explicitly chosen library is used as it is
    if not force and not _stale():
        return LIB_PATH
    os.makedirs(LIB_DIR, exist_ok=True)
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    extra = ["-DFB_TRACE"] if os.environ.get("FLUXBIN_TRACE") == "1" else []    # the instrumented build (per-CTA phase timestamps)
    cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + _sources()
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
