"""Builds libswiftprune.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a.

    python -m paper_2501_16376_b200.build [--force] [--verbose] [--debug]
"""
from __future__ import annotations

import glob
import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB = os.path.join(HERE, "libswiftprune.so")
LIB_DEBUG = os.path.join(HERE, "libswiftprune_debug.so")   # same ABI, index checks compiled in

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17",
    "-Xcompiler", "-fPIC",
    "--expt-relaxed-constexpr",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _deps():
    return sources() + glob.glob(os.path.join(CSRC, "*.h")) + \
        glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(INCLUDE, "*.h"))


def is_current(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    return all(os.path.getmtime(p) <= t for p in _deps())


def build(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """Builds the release library, or with debug=True the debug build (-DSP_DEBUG_CHECKS:
    out-of-range stores are skipped and recorded, see sp_debug_status)."""
    lib = LIB_DEBUG if debug else LIB
    if not force and is_current(lib):
        return lib
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-shared", "-o", tmp, "-I", INCLUDE, "-I", CSRC] + NVCC_FLAGS
    if debug:
        cmd += ["-DSP_DEBUG_CHECKS"]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    cmd += sources()
    proc = subprocess.run(cmd, stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed (exit %d)" % proc.returncode)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="--verbose" in sys.argv,
                debug="--debug" in sys.argv))
