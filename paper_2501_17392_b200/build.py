"""Build the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""

from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG_DIR)
LIB_PATH = os.path.join(PKG_DIR, "libbrace.so")
DEBUG_LIB_PATH = os.path.join(PKG_DIR, "libbrace_debug.so")
SOURCES = [os.path.join(PKG_DIR, "csrc", "brace.cu")]
DEPS = SOURCES + [os.path.join(PKG_DIR, "csrc", "brace_kernels.cuh"), os.path.join(ROOT, "include", "brace.h")]


def _nvcc() -> str:
    cand = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(cand):
        raise RuntimeError("nvcc not found: the BRACE CUDA library cannot be built")
    return cand


def needs_build(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(p) > t for p in DEPS)


def _compile(out_path: str, defines, verbose: bool) -> str:
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-I", os.path.join(ROOT, "include"),
           "-I", os.path.join(PKG_DIR, "csrc")] + list(defines) + ["-o", out_path] + SOURCES
    if verbose:
        cmd[1:1] = ["-Xptxas", "-v"]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        sys.stderr.write(res.stderr)
    return out_path


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB_PATH
    return _compile(LIB_PATH, [], verbose)


def build_debug(force: bool = False, verbose: bool = False) -> str:
    """The same library with -DBRACE_DEBUG: ring kernels check their index ranges and report through
    brace_debug_status instead of trapping.  Load it by setting BRACE_LIBRARY to the returned path."""
    if not force and not needs_build(DEBUG_LIB_PATH):
        return DEBUG_LIB_PATH
    return _compile(DEBUG_LIB_PATH, ["-DBRACE_DEBUG"], verbose)


if __name__ == "__main__":
    if "--debug" in sys.argv:
        print(build_debug(force="--force" in sys.argv, verbose="-v" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
