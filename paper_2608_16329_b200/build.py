"""Compile the CUDA library in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
CSRC = os.path.join(_PKG, "csrc")
LIB_PATH = os.path.join(_PKG, "libmlip_b200.so")


def sources() -> list[str]:
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def needs_build() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = sources() + glob.glob(os.path.join(CSRC, "*.cuh")) + glob.glob(os.path.join(_ROOT, "include", "*.h"))
    return any(os.path.getmtime(d) > t for d in deps)


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False) -> str:
    """debug_bounds: the range-checked build (-DMLIP_DEBUG_BOUNDS) as libmlip_b200_bounds.so next to the library; load it
    through the MLIP_B200_LIB environment variable."""
    if debug_bounds:
        return _compile(os.path.join(_PKG, "libmlip_b200_bounds.so"), ["-DMLIP_DEBUG_BOUNDS"], verbose)
    if not force and not needs_build():
        return LIB_PATH
    return _compile(LIB_PATH, [], verbose)


def _compile(target: str, defines: list[str], verbose: bool) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--threads", "0", "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
           "-o", target] + defines + sources()
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    subprocess.check_call(cmd)
    return target
