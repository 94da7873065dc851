"""Builds the C-ABI library ``libampq.so`` in-tree with nvcc for sm_100a.

Run as ``python -m paper_2505_13060_b200.build``; ``build()`` is also what the
repository's ``__graft_entry__.build`` calls.  nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libampq.so")
SOURCES = ["ampq_kernels.cu", "ampq_lib.cu", "ampq_noalloc.cu", "ampq_select.cpp", "ampq_graph.cpp"]
HEADERS = ["ampq_device.h", "ampq_kernels.h", "ampq_select.h", os.path.join("..", "..", "include", "ampq.h")]
NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "-Xcompiler", "-fPIC", "-Xcompiler", "-fvisibility=hidden",
]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.sep not in cand or os.path.exists(cand)):
            return cand
    return "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, out: str | None = None, defines=()) -> str:
    """Builds the library.  ``out``/``defines`` make a second build beside the
    default one, e.g. ``defines=["AMPQ_BOUNDS_CHECK"]`` for the self-checking
    debug build (load it with the AMPQ_LIBRARY environment variable)."""
    lib = out or LIB
    if out is None and not force and not needs_build():
        return LIB
    tmp = lib + ".tmp.%d" % os.getpid()
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-D" + d for d in defines]
    cmd += ["-shared", "-o", tmp] + [os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
