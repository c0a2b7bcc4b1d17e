"""Build libspx.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "libspx.so")
_SOURCES = [os.path.join(_PKG, "csrc", "spx_api.cu")]


def _newest_source_mtime() -> float:
    newest = 0.0
    for d in (os.path.join(_PKG, "csrc"), os.path.join(_ROOT, "include")):
        for name in os.listdir(d):
            newest = max(newest, os.path.getmtime(os.path.join(d, name)))
    return newest


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source into paper_2609_34370_b200/libspx.so; returns its path."""
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC", "-cudart", "static",
           "-I", os.path.join(_ROOT, "include"), "-I", os.path.join(_PKG, "csrc"),
           "-o", LIB_PATH] + _SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
