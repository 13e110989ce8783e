"""Build the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import shutil
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
INCLUDE = os.path.join(_ROOT, "include")
LIB_PATH = os.path.join(_PKG, "libsuperoffload.so")
SOURCES = [os.path.join(CSRC, "superoffload.cu"), os.path.join(CSRC, "so_static_check.cu")]
_DEPS = SOURCES + [os.path.join(CSRC, "so_kernels.cuh"), os.path.join(CSRC, "so_step_tma.cuh"), os.path.join(CSRC, "so_types.h"), os.path.join(CSRC, "so_pack.cuh"),
                   os.path.join(INCLUDE, "superoffload.h")]


def _nvcc() -> str:
    for cand in (shutil.which("nvcc"), "/usr/local/cuda/bin/nvcc"):
        if cand and os.path.exists(cand):
            return cand
    raise RuntimeError("nvcc not found: the CUDA library cannot be built")


def is_stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    built = os.path.getmtime(LIB_PATH)
    return any(os.path.getmtime(p) > built for p in _DEPS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile ``libsuperoffload.so`` (sm_100a only) next to this file."""
    if not force and not is_stale():
        return LIB_PATH
    tmp = LIB_PATH + f".tmp{os.getpid()}"
    cmd = [_nvcc(), "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3",
           "-std=c++17", "--fmad=false", "-Xcompiler", "-fPIC,-O2,-Wall", "-shared",
           "-I", INCLUDE, "-I", CSRC, "-o", tmp] + SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, LIB_PATH)
    if verbose:
        print(res.stderr)
    return LIB_PATH


if __name__ == "__main__":
    print(build_library(force=True, verbose=True))
