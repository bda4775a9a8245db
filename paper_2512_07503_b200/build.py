"""Compile the CUDA library (libsjd.so) in-tree for sm_100a with nvcc."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
_INC = os.path.join(os.path.dirname(_PKG), "include")
LIB_PATH = os.path.join(_PKG, "libsjd.so")

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-shared",
              "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr", "--extended-lambda"]


def _nvcc() -> str:
    for c in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if c and os.path.exists(c):
            return c
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def sources():
    return sorted(glob.glob(os.path.join(_CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(_CSRC, "*.cuh")) + glob.glob(os.path.join(_INC, "*.h"))


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(p) > t for p in _deps())


def build(force: bool = False, verbose: bool = False) -> str:
    override = os.environ.get("SJD_LIBRARY")
    if override:  # a library built elsewhere (the tests build variants with build_variant())
        return override
    if not force and not is_stale():
        return LIB_PATH
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = [_nvcc(), *NVCC_FLAGS, "-I", _INC, *(["-Xptxas", "-v"] if verbose else []), *sources(), "-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


def build_variant(out_path: str, defines) -> str:
    """The library with extra -D definitions (test builds: short wait limits, a dropped copy), written to
    `out_path`.  Load it in a process of its own by setting SJD_LIBRARY to that path."""
    cmd = [_nvcc(), *NVCC_FLAGS, "-I", _INC, *[f"-D{d}" for d in defines], *sources(), "-o", out_path]
    subprocess.check_call(cmd)
    return out_path


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv))
