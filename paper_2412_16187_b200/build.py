"""Builds the CUDA library in-tree (nvcc, sm_100a only). nvcc cross-compiles, so no GPU is needed to build."""
from __future__ import annotations

import glob
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "libhashevict.so")
_SOURCES = sorted(glob.glob(os.path.join(_PKG, "csrc", "*.cu")))
_HEADERS = sorted(glob.glob(os.path.join(_ROOT, "include", "*.h")) + glob.glob(os.path.join(_PKG, "csrc", "*.cuh")))

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-shared",
]


def nvcc_path() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


DEBUG_LIB_PATH = os.path.join(_PKG, "libhashevict_debug.so")


def build_cuda(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile csrc/*.cu into libhashevict.so; rebuilds only when a source or header is newer.

    debug=True builds libhashevict_debug.so with -DHE_BOUNDS_CHECK instead: every slot and token index is range-checked
    before it is used as an address, a failed check skips the access and raises he_device_error_count(). The binding
    loads that library when HE_DEBUG_LIB=1 is set before the first call."""
    out = DEBUG_LIB_PATH if debug else LIB_PATH
    deps = _SOURCES + _HEADERS
    if not force and os.path.exists(out) and all(os.path.getmtime(out) >= os.path.getmtime(p) for p in deps):
        return out
    tmp = out + f".tmp{os.getpid()}"
    cmd = [nvcc_path()] + NVCC_FLAGS + (["-DHE_BOUNDS_CHECK"] if debug else []) + (["-Xptxas", "-v"] if verbose else []) + \
        ["-I", os.path.join(_ROOT, "include"), "-o", tmp] + _SOURCES
    subprocess.run(cmd, check=True)
    os.replace(tmp, out)
    return out
