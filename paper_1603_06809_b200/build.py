"""Build the C-ABI library (libbcast_b200.so) in-tree with nvcc for sm_100a.

Run as ``python -m paper_1603_06809_b200.build`` or call :func:`build`.  The shared object is
placed next to this file so that it travels with the source tree.
"""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
REPO_DIR = os.path.dirname(PKG_DIR)
LIB_PATH = os.path.join(PKG_DIR, "libbcast_b200.so")
SOURCES = [os.path.join(PKG_DIR, "csrc", f) for f in ("plan.cpp", "walk_tables.cpp", "shard.cpp", "exec.cu")]
HEADERS = [os.path.join(REPO_DIR, "include", "bcast.h")] + [os.path.join(PKG_DIR, "csrc", f) for f in ("plan_internal.h", "walk_tables.h", "exec_internal.h", "kernels.cuh")]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(REPO_DIR, "include"),
]


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; return its path."""
    if force or needs_build():
        nvcc = os.environ.get("NVCC", "nvcc")
        tmp = LIB_PATH + f".{os.getpid()}.tmp"
        cmd = [nvcc, *NVCC_FLAGS, *(["-Xptxas", "-v"] if verbose else []), "-o", tmp, *SOURCES]
        subprocess.check_call(cmd)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


def ensure_built() -> str:
    """Build the library if it is missing; if it is merely older than its sources, try to rebuild
    and keep the existing one when no compiler is at hand.  Returns the path of the library."""
    if not os.path.exists(LIB_PATH):
        return build(force=True)
    if needs_build():
        try:
            return build(force=True)
        except (OSError, subprocess.CalledProcessError):
            pass
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
