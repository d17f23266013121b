"""Builds ``librudra_ps.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_PKG = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_PKG, "csrc")
_INCLUDE = os.path.join(os.path.dirname(_PKG), "include")
LIB_PATH = os.path.join(_PKG, "librudra_ps.so")
SOURCES = ["ps.cu", "update.cu", "snapshot.cu", "leaf.cu", "noalloc.cu", "sched.cpp"]
# measurement utility of the benchmark, a library of its own: not part of the product interface
PROBE_LIB_PATH = os.path.join(_PKG, "librudra_probe.so")
PROBE_SOURCES = ["probe.cu"]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-cudart", "static", "-shared",
]


def _deps():
    out = [os.path.join(_CSRC, f) for f in os.listdir(_CSRC)]
    out += [os.path.join(_INCLUDE, f) for f in os.listdir(_INCLUDE)]
    return out


def needs_build(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(d) > t for d in _deps())


def _compile(path, sources, verbose):
    nvcc = os.environ.get("NVCC", "nvcc")
    tmp = path + ".tmp.%d" % os.getpid()
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-I", _INCLUDE, "-o", tmp]
    cmd += os.environ.get("RUDRA_NVCC_DEFINES", "").split()   # e.g. "-DRUDRA_MID_THREADS=128" for a tile sweep
    cmd += [os.path.join(_CSRC, s) for s in sources]
    subprocess.check_call(cmd)
    os.replace(tmp, path)
    return path


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB_PATH
    return _compile(LIB_PATH, SOURCES, verbose)


def build_probe(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build(PROBE_LIB_PATH):
        return PROBE_LIB_PATH
    return _compile(PROBE_LIB_PATH, PROBE_SOURCES, verbose)


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
    print(build_probe(force="--force" in sys.argv, verbose="-v" in sys.argv))
