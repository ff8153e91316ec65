"""In-tree build of the CUDA library: nvcc for sm_100a into ``paper_2503_17513_b200/libxq.so``.

Run ``python -m paper_2503_17513_b200.build`` (add ``-v`` for ptxas register/shared-memory
statistics).  nvcc cross-compiles without a GPU.

``--debug-bounds`` builds a second library, ``libxq_debug.so``, from the same sources with
``-DXQ_DEBUG_BOUNDS``: the product kernels then test their computed indices (weight-stream source
ranges, ring stages, token-slice and partial-tile stores, output offsets) before using them; a
failing test stores XQ_ERR_BOUNDS in the workspace status word and skips the access.  Load it in
place of the normal library by setting ``XQ_LIBRARY`` to its path before importing the binding.
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys
from concurrent.futures import ThreadPoolExecutor

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libxq.so")
LIB_DEBUG = os.path.join(PKG, "libxq_debug.so")


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _stale(lib: str) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile every .cu to an object (in parallel, only those older than their dependencies) and link."""
    lib = LIB_DEBUG if debug_bounds else LIB
    if not force and not _stale(lib):
        return lib
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    objdir = os.path.join(ROOT, "_build", "debug") if debug_bounds else os.path.join(ROOT, "_build")
    os.makedirs(objdir, exist_ok=True)
    headers = glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(ROOT, "include", "*.h"))
    t_hdr = max(os.path.getmtime(h) for h in headers)
    flags = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17", "-Xcompiler", "-fPIC",
             "-I", os.path.join(ROOT, "include"), "-I", CSRC]
    if verbose:
        flags += ["-Xptxas", "-v"]
    if debug_bounds:
        flags += ["-DXQ_DEBUG_BOUNDS"]

    def compile_one(src: str) -> str:
        obj = os.path.join(objdir, os.path.basename(src)[:-3] + ".o")
        if force or not os.path.exists(obj) or os.path.getmtime(obj) < max(os.path.getmtime(src), t_hdr):
            subprocess.run([nvcc, *flags, "-c", src, "-o", obj], check=True)
        return obj

    with ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        objs = list(pool.map(compile_one, sources()))
    subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-shared", "-o", lib, *objs], check=True)
    return lib


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv, debug_bounds="--debug-bounds" in sys.argv))
