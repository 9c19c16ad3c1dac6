"""Builds libgk.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libgk.so")
DEBUG_LIB_PATH = os.path.join(_HERE, "libgk_debug.so")   # the bounds-checked build (-DGK_DEBUG)

_SOURCES = ["gk_api.cu"]
_DEPS = ["gk_api.cu", "gk_kernels.cuh", "gk_device.cuh", "gk_sha256.cuh", "gk_gf2_generated.inc", "gen_tables.py",
         os.path.join("..", "..", "include", "gk.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def build(force: bool = False, verbose: bool = False, extra_flags: list[str] | None = None, debug: bool = False) -> str:
    """Builds libgk.so, or with debug=True libgk_debug.so: the same sources with -DGK_DEBUG, in which the
    streaming kernels compare every access to caller memory with the extent of its object (use it through
    GK_LIB_PATH)."""
    lib_path = DEBUG_LIB_PATH if debug else LIB_PATH
    if debug:
        extra_flags = list(extra_flags or []) + ["-DGK_DEBUG"]
    sys.path.insert(0, _CSRC)
    try:
        import gen_tables
        gen_tables.main()
    finally:
        sys.path.pop(0)
    deps = [os.path.join(_CSRC, d) for d in _DEPS]
    newest = max(os.path.getmtime(d) for d in deps if os.path.exists(d))
    if not force and os.path.exists(lib_path) and os.path.getmtime(lib_path) >= newest:
        return lib_path
    tmp = lib_path + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-Wall", "--use_fast_math",
           "-I", os.path.join(_HERE, "..", "include")]
    if verbose:
        cmd += ["-Xptxas", "-v"]
    if extra_flags:
        cmd += extra_flags
    if os.environ.get("GK_NVCC_FLAGS"):
        cmd += os.environ["GK_NVCC_FLAGS"].split()
    cmd += [os.path.join(_CSRC, s) for s in _SOURCES] + ["-o", tmp, "-lcudart"]
    subprocess.check_call(cmd)
    os.replace(tmp, lib_path)
    return lib_path


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
