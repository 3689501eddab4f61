"""Compile libcstr.so in-tree with nvcc for sm_100a."""

from __future__ import annotations

import os
import shutil
import subprocess

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
CSRC = os.path.join(PKG_DIR, "csrc")
INCLUDE = os.path.join(ROOT, "include")
LIB_PATH = os.path.join(PKG_DIR, "libcstr.so")
# Checking build: every kernel index range-checked into a status record (no trap), plus
# the test-only setters of include/cstr_debug.h.  Tests run their small cases against it.
CHECK_LIB_PATH = os.path.join(PKG_DIR, "libcstr_check.so")
CHECK_FLAGS = ["-DCSTR_BOUNDS_CHECK", "-DCSTR_TESTING"]
SOURCES = ["cstr_host.cu", "cstr_build.cu", "cstr_step.cu", "cstr_pda.cu"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found; libcstr needs the CUDA toolkit to build")
    return exe


def _stale(path: str) -> bool:
    if not os.path.exists(path):
        return True
    built = os.path.getmtime(path)
    deps = [os.path.join(CSRC, f) for f in os.listdir(CSRC)]
    deps += [os.path.join(INCLUDE, f) for f in os.listdir(INCLUDE)]
    return any(os.path.getmtime(d) > built for d in deps)


def build_library(force: bool = False, verbose: bool = False, check: bool = False) -> str:
    """Build ``libcstr.so`` (or, with ``check``, the checking build ``libcstr_check.so``)
    next to this file if it is missing or out of date."""
    path = CHECK_LIB_PATH if check else LIB_PATH
    if not force and not _stale(path):
        return path
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
           "-std=c++17", "-shared", "-Xcompiler", "-fPIC", "-I", INCLUDE, "-I", CSRC]
    if check:
        cmd += CHECK_FLAGS
    cmd += ["-o", path] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.run(cmd, check=True)
    return path


if __name__ == "__main__":
    import sys
    print(build_library(force=True, verbose="-v" in sys.argv, check="--check" in sys.argv))
