"""Builds libgk.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libgk.so")

_SOURCES = ["gk_api.cu"]
_DEPS = ["gk_api.cu", "gk_kernels.cuh", "gk_device.cuh", "gk_sha256.cuh", "gk_gf2_generated.inc", "gen_tables.py",
         os.path.join("..", "..", "include", "gk.h")]


def _nvcc() -> str:
    for cand in (os.environ.get("NVCC"), "/usr/local/cuda/bin/nvcc", "nvcc"):
        if cand and (os.path.isabs(cand) and os.path.exists(cand) or not os.path.isabs(cand)):
            return cand
    return "nvcc"


def build(force: bool = False, verbose: bool = False, extra_flags: list[str] | None = None) -> str:
    sys.path.insert(0, _CSRC)
    try:
        import gen_tables
        gen_tables.main()
    finally:
        sys.path.pop(0)
    deps = [os.path.join(_CSRC, d) for d in _DEPS]
    newest = max(os.path.getmtime(d) for d in deps if os.path.exists(d))
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= newest:
        return LIB_PATH
    tmp = LIB_PATH + f".tmp{os.getpid()}"
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
    os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
