"""In-tree build of the CUDA library (``liblaga.so``) with nvcc for sm_100a.

Run as ``python -m paper_2607_17644_b200.build`` or call :func:`build`.  nvcc cross-compiles
without a GPU present.  The library is rebuilt only when a source is newer than it.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
ROOT = os.path.dirname(PKG_DIR)
LIB_PATH = os.path.join(PKG_DIR, "liblaga.so")
DEBUG_LIB_PATH = os.path.join(PKG_DIR, "liblaga_debug.so")   # the checked build (-DLAGA_DEBUG), see sm100_ptx.cuh

NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "--expt-relaxed-constexpr"]


def sources():
    return (sorted(glob.glob(os.path.join(CSRC, "*.cu"))),
            sorted(glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))))


def build(force: bool = False, verbose: bool = False, extra_flags=(), debug: bool = False) -> str:
    """Build the library (debug=True: the checked build, whose kernels verify their own index arithmetic
    and report LAGA_ERR_DEVICE_CHECK instead of making a bad access; selected at run time by LAGA_DEBUG=1)."""
    cus, deps = sources()
    target = DEBUG_LIB_PATH if debug else LIB_PATH
    newest = max(os.path.getmtime(p) for p in cus + deps)
    if not force and os.path.exists(target) and os.path.getmtime(target) >= newest:
        return target
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = target + f".tmp{os.getpid()}"
    cmd = [nvcc, *NVCC_FLAGS, *(("-DLAGA_DEBUG=1",) if debug else ()), *extra_flags, "-o", tmp, *cus]
    if verbose:
        print(" ".join(cmd), file=sys.stderr)
    subprocess.run(cmd, check=True)
    os.replace(tmp, target)
    return target


if __name__ == "__main__":
    flags = ("-Xptxas", "-v") if "--ptxas-v" in sys.argv else ()
    print(build(force="--force" in sys.argv, verbose=True, extra_flags=flags))
    print(build(force="--force" in sys.argv, verbose=True, extra_flags=flags, debug=True))
