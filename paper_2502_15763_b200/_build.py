"""Builds libhos.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libhos.so")
DEBUG_LIB_PATH = os.path.join(_PKG, "libhos_debug.so")   # the bounds-checked build (-DHOS_DEBUG_BOUNDS)

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC", "--expt-relaxed-constexpr"]


def _sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return _sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(CSRC, "*.h")) + \
        glob.glob(os.path.join(INCLUDE, "*.h"))


def source_hash() -> str:
    """SHA-256 over the library's sources (names and contents, in name order): what a set of
    profiler counters was taken on."""
    import hashlib
    h = hashlib.sha256()
    for path in sorted(_deps()):
        h.update(os.path.basename(path).encode() + b"\0")
        with open(path, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def is_stale(debug: bool = False) -> bool:
    path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(f) > t for f in _deps())


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Compile every .cu under csrc/ into libhos.so (debug: the bounds-checked libhos_debug.so);
    returns its path."""
    path = DEBUG_LIB_PATH if debug else LIB_PATH
    if not force and not is_stale(debug):
        return path
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = path + f".{os.getpid()}.tmp"
    cmd = [nvcc] + NVCC_FLAGS + (["-DHOS_DEBUG_BOUNDS"] if debug else []) + (["-Xptxas", "-v"] if verbose else []) + \
        ["-I", INCLUDE, "-I", CSRC, "-o", tmp] + _sources()
    subprocess.check_call(cmd)
    os.replace(tmp, path)
    return path


if __name__ == "__main__":
    import sys
    print(build(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
