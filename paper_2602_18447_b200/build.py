"""Build the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libconfspec.so")
DEBUG_LIB_PATH = os.path.join(_HERE, "libconfspec_debug.so")      # the same sources with -DCS_DEBUG (device-side range checks)
SOURCES = ["api.cu", "gemm_tcgen05.cu", "attention.cu", "attention_short.cu", "lmhead.cu", "elementwise.cu"]
HEADERS = ["common.cuh", "gemm.h", "kernels.h", os.path.join("..", "..", "include", "confspec.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; the CUDA library cannot be built")
    return exe


def needs_build(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    t = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile csrc/*.cu into libconfspec.so (debug: libconfspec_debug.so, with -DCS_DEBUG) next to this file and
    return its path."""
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and not needs_build(lib_path):
        return lib_path
    cmd = [_nvcc()] + NVCC_FLAGS + (["-DCS_DEBUG"] if debug else []) + (["-Xptxas", "-v"] if verbose else []) + \
          [os.path.join(CSRC, f) for f in SOURCES] + ["-o", lib_path]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        print(res.stderr)
    return lib_path


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build(force=True, debug=True))
