"""Builds libspeckv.so (sm_100a) in-tree with nvcc.  `python -m paper_2605_02888_b200.build`."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
_INC = os.path.join(os.path.dirname(_PKG), "include")
LIB_PATH = os.path.join(_CSRC, "libspeckv.so")
_SOURCES = ["speckv.cu"]
_DEPS = ["speckv.cu", "speckv_kernels.cuh", "speckv_pipeline.cuh", "speckv_shard.cuh", "speckv_sample.cuh"]

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared"]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


DEBUG_LIB_PATH = os.path.join(_CSRC, "libspeckv_debug.so")


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    deps = [os.path.join(_CSRC, d) for d in _DEPS] + [os.path.join(_INC, h) for h in ("speckv.h", "speckv_internal.h")]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; return its path.
    debug=True builds the bounds-checked variant (-DSPECKV_DEBUG) beside it: every logit load and
    workspace access is compared with the call's extents, skipped and counted when outside."""
    out = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and not is_stale(out):
        return out
    tmp = out + f".tmp{os.getpid()}"
    cmd = [_nvcc(), *NVCC_FLAGS, *(["-DSPECKV_DEBUG"] if debug else []), "-I", _INC, "-o", tmp] + [os.path.join(_CSRC, s) for s in _SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
        print(" ".join(cmd), file=sys.stderr)
    subprocess.check_call(cmd)
    os.replace(tmp, out)
    return out


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
