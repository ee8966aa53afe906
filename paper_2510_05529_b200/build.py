"""Builds libh1b.so (the CUDA library behind include/h1b.h) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
# H1B_DEBUG_BOUNDS=1 in the environment selects the bounds-checked build (the kernels' index checks compiled in): a
# library of its own beside the ordinary one, so that both can be built ahead of time.
DEBUG_BOUNDS = os.environ.get("H1B_DEBUG_BOUNDS", "0") not in ("", "0")
LIB_PATH = os.path.join(_PKG, "libh1b_bounds.so" if DEBUG_BOUNDS else "libh1b.so")
SOURCES = ["h1b_api.cu", "h1b_kernels.cu", "h1b_prompt.cu"]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--use_fast_math=false", "-Xcompiler", "-fPIC", "-shared"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: libh1b.so cannot be built")


def _inputs():
    out = []
    for root, _, files in os.walk(_CSRC):
        out += [os.path.join(root, f) for f in files]
    out.append(os.path.join(os.path.dirname(_PKG), "include", "h1b.h"))
    return out


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(f) > t for f in _inputs())


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources. Returns its path."""
    if not force and not is_stale():
        return LIB_PATH
    tmp = LIB_PATH + ".tmp.%d" % os.getpid()
    flags = [f for f in NVCC_FLAGS if f != "--use_fast_math=false"] + (["-DH1B_DEBUG_BOUNDS"] if DEBUG_BOUNDS else [])
    cmd = [_nvcc()] + flags + (["-Xptxas", "-v"] if verbose else []) + \
          [os.path.join(_CSRC, s) for s in SOURCES] + ["-o", tmp]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n%s\n%s" % (res.stdout, res.stderr))
    if verbose:
        print(res.stderr)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose="-v" in sys.argv))
