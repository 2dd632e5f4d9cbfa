"""In-tree build of the CUDA library (nvcc, sm_100a only).  Cross-compiles without a GPU."""
from __future__ import annotations

import glob
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(_PKG, "csrc")
LIB = os.path.join(_PKG, "libspade_b200.so")
LIB_DEBUG = os.path.join(_PKG, "libspade_b200_debug.so")     # the same sources with -DSPADE_DEBUG (index checks, guard words)
SOURCES = ["api.cu", "plan.cu", "selection.cu", "scores.cu", "attn.cu"]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-Xcompiler", "-fPIC", "-shared"]


def _stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = glob.glob(os.path.join(CSRC, "*")) + [os.path.join(_PKG, "..", "include", "spade.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile csrc/*.cu into libspade_b200.so next to this file (only when sources changed);
    debug=True builds libspade_b200_debug.so with -DSPADE_DEBUG instead."""
    lib = LIB_DEBUG if debug else LIB
    if force or _stale(lib):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        tmp = lib + f".tmp{os.getpid()}"
        extra = os.environ.get("SPADE_NVCC_EXTRA", "").split() + (["-DSPADE_DEBUG"] if debug else [])
        cmd = [nvcc] + NVCC_FLAGS + extra + (["-Xptxas", "-v"] if verbose else []) + \
              [os.path.join(CSRC, s) for s in SOURCES] + ["-o", tmp]
        subprocess.check_call(cmd)
        os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose=True, debug="--debug" in sys.argv))
