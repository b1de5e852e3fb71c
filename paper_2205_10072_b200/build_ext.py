"""Compiles the CUDA sources of this package for sm_100a into libbcs.so (in-tree, next to this file)."""
from __future__ import annotations

import glob
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "libbcs.so")
SOURCES = sorted(glob.glob(os.path.join(_PKG, "csrc", "*.cu")))
HEADERS = sorted(glob.glob(os.path.join(_ROOT, "include", "*.h")) +
                 glob.glob(os.path.join(_PKG, "csrc", "*.cuh")))
# The benchmark's integer-rate probe is a library of its own: it is not part of the product and
# only bench.py loads it.
PROBE_LIB_PATH = os.path.join(_PKG, "libbcs_probe.so")
PROBE_SOURCES = sorted(glob.glob(os.path.join(_PKG, "csrc", "probe", "*.cu")))
PROBE_HEADERS = sorted(glob.glob(os.path.join(_PKG, "csrc", "probe", "*.h")))

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a",
    "-O3", "-lineinfo", "-std=c++17",
    "--shared", "-Xcompiler", "-fPIC",
    "-I", os.path.join(_ROOT, "include"),
]


def _stale(lib: str, deps: list) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in deps)


def stale() -> bool:
    return _stale(LIB_PATH, SOURCES + HEADERS)


def _nvcc(lib: str, sources: list, verbose: bool, extra: list = ()) -> None:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = lib + ".%d.tmp" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + sources
    subprocess.check_call(cmd)
    os.replace(tmp, lib)


def build(force: bool = False, verbose: bool = False) -> str:
    """Runs nvcc (cross-compiles without a GPU).  Returns the path of the shared library."""
    if force or stale():
        _nvcc(LIB_PATH, SOURCES, verbose)
    return LIB_PATH


def build_probe(force: bool = False, verbose: bool = False) -> str:
    """The benchmark's probe library (bcs_probe_int_rate), separate from libbcs.so."""
    if force or _stale(PROBE_LIB_PATH, PROBE_SOURCES + PROBE_HEADERS + HEADERS):
        _nvcc(PROBE_LIB_PATH, PROBE_SOURCES, verbose, ["-I", os.path.join(_PKG, "csrc")])
    return PROBE_LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
    print(build_probe(force=True, verbose=True))
