"""Builds the C-ABI shared library (sm_100a only) in-tree with nvcc."""
from __future__ import annotations

import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB_NAME = "libsol_attn3d.so"
LIB_PATH = os.path.join(HERE, LIB_NAME)
# the same library with device-side index checks compiled in (see sol_attn3d_status_word in the header)
DEBUG_LIB_PATH = os.path.join(HERE, "libsol_attn3d_debug.so")
DEBUG_FLAGS = ("-DSOL_ATTN3D_DEBUG=1",)
SOURCES = ["sol_attn3d.cu"]
HEADERS = sorted(f for f in os.listdir(CSRC) if f.endswith(".cuh")) + [os.path.join("..", "..", "include", "sol_attn3d.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def is_stale(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    t = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


def build_library(force: bool = False, verbose: bool = False, extra_flags=(), out: str = LIB_PATH) -> str:
    if not force and not is_stale(out):
        return out
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-std=c++17", "-lineinfo",
           "-Xcompiler", "-fPIC", "-shared", "-Xptxas", "-v" if verbose else "-O3",
           "-o", out] + list(extra_flags) + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stdout + res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
    return out


def build_debug_library(force: bool = False) -> str:
    return build_library(force=force, extra_flags=DEBUG_FLAGS, out=DEBUG_LIB_PATH)


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv))
    if "--debug" in sys.argv:
        print(build_debug_library(force=True))
