"""Builds the CUDA library in-tree for sm_100a with nvcc (no GPU needed to compile)."""
from __future__ import annotations

import os
import shutil
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_DIR = os.path.join(HERE, "lib")
LIB_PATH = os.path.join(LIB_DIR, "liblt_indexer.so")
DEBUG_LIB_PATH = os.path.join(LIB_DIR, "liblt_indexer_dbg.so")  # bounds-checking build (-DLT_DEBUG_BOUNDS)
SOURCES = ["lt_api.cu", "lt_scan_mma.cu", "lt_scan_fp8.cu", "lt_select.cu", "lt_sampler.cu", "lt_dsa_union.cu", "lt_scan_knn.cu", "lt_umma_stream.cu"]
HEADERS = ["lt_common.cuh", "lt_host.h", "lt_ptx.cuh", os.path.join("..", "..", "include", "lt_indexer.h")]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; cannot build liblt_indexer.so")
    return exe


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    built = os.path.getmtime(path)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """Compile csrc/*.cu into lib/liblt_indexer.so; returns the library path.

    debug_bounds=True builds lib/liblt_indexer_dbg.so instead: the same sources with -DLT_DEBUG_BOUNDS, whose
    kernels check the index of every global store / gather they were given a bound for, skip an access that
    fails the check and record LT_STATUS_BOUNDS in the status word (they never trap)."""
    out = DEBUG_LIB_PATH if debug_bounds else LIB_PATH
    if not force and not is_stale(out):
        return out
    os.makedirs(LIB_DIR, exist_ok=True)
    cmd = [_nvcc(), "-shared", "-Xcompiler", "-fPIC", "-std=c++17", "-O3", "-lineinfo",
           "-gencode", "arch=compute_100a,code=sm_100a"]
    if debug_bounds:
        cmd += ["-DLT_DEBUG_BOUNDS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += ["-o", out] + [os.path.join(CSRC, s) for s in SOURCES]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + proc.stdout + proc.stderr)
    if verbose:
        print(proc.stderr)
    return out


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build(force=True, debug_bounds=True))
