"""Compile the CUDA library in-tree for sm_100a with nvcc (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libfreebalance.so")
SOURCES = ["fb_api.cu"]
HEADERS = sorted(f for f in os.listdir(CSRC) if f.endswith((".cuh", ".h"))) + \
          [os.path.join("..", "..", "include", h) for h in ("freebalance.h", "freebalance_aids.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found")


_EXTERNAL = False        # True once use_library() has chosen a file this module does not rebuild


def is_stale() -> bool:
    if _EXTERNAL:
        return False
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def _compile(out_path: str, extra_flags, verbose: bool) -> str:
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xptxas", "-v", "-DNDEBUG"] + list(extra_flags) + \
          ["-o", out_path] + [os.path.join(CSRC, s) for s in SOURCES] + ["-lcudart"]
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if verbose or proc.returncode != 0:
        sys.stderr.write(proc.stdout + proc.stderr)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + proc.stderr[-4000:])
    return out_path


def build(force: bool = False, verbose: bool = False) -> str:
    """Build libfreebalance.so if missing or older than its sources; return its path."""
    if not force and not is_stale():
        return LIB_PATH
    return _compile(LIB_PATH, [], verbose)


def build_variant(suffix: str, flags, force: bool = False, verbose: bool = False) -> str:
    """Build libfreebalance_<suffix>.so with extra compiler flags (e.g. the phase-stamp build,
    -DFB_TIMING) beside the normal library; return its path."""
    path = os.path.join(PKG_DIR, f"libfreebalance_{suffix}.so")
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    if force or not os.path.exists(path) or any(os.path.getmtime(d) > os.path.getmtime(path) for d in deps):
        _compile(path, flags, verbose)
    return path


def use_library(path: str) -> None:
    """Make binding.lib() load this library file instead of the default one (call before the first
    binding call of the process)."""
    global LIB_PATH, _EXTERNAL
    LIB_PATH = path
    _EXTERNAL = True


if __name__ == "__main__":
    print(build(force=True, verbose=True))
