"""Build libspx.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
LIB_PATH = os.path.join(_PKG, "libspx.so")
TIMELINE_LIB_PATH = os.path.join(_PKG, "libspx_timeline.so")
WAIT_TEST_LIB_PATH = os.path.join(_PKG, "libspx_waittest.so")
_SOURCES = [os.path.join(_PKG, "csrc", "spx_api.cu")]


def _newest_source_mtime() -> float:
    newest = 0.0
    for d in (os.path.join(_PKG, "csrc"), os.path.join(_ROOT, "include")):
        for name in os.listdir(d):
            newest = max(newest, os.path.getmtime(os.path.join(d, name)))
    return newest


def _compile(out_path: str, defines=(), verbose: bool = False) -> str:
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "--shared", "-Xcompiler", "-fPIC", "-cudart", "static",
           "-I", os.path.join(_ROOT, "include"), "-I", os.path.join(_PKG, "csrc")]
    cmd += ["-D" + d for d in defines]
    cmd += ["-o", out_path] + _SOURCES
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    return out_path


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile every CUDA source into paper_2609_34370_b200/libspx.so; returns its path."""
    if not force and os.path.exists(LIB_PATH) and os.path.getmtime(LIB_PATH) >= _newest_source_mtime():
        return LIB_PATH
    return _compile(LIB_PATH, verbose=verbose)


def build_timeline(force: bool = False) -> str:
    """The same sources with per-CTA timestamps compiled in (libspx_timeline.so; see
    spx_debug_timeline).  Used by `bench.py --timeline` only."""
    if not force and os.path.exists(TIMELINE_LIB_PATH) and os.path.getmtime(TIMELINE_LIB_PATH) >= _newest_source_mtime():
        return TIMELINE_LIB_PATH
    return _compile(TIMELINE_LIB_PATH, defines=("SPX_TIMELINE=1",))


def build_wait_test(force: bool = False) -> str:
    """The same sources with every bounded wait limited to 100k cycles (about 50 us) and the kernel
    behind spx_debug_wait_expiry compiled in (libspx_waittest.so).  Used by the timeout test only:
    its production kernels would give up on ordinary memory latency."""
    if not force and os.path.exists(WAIT_TEST_LIB_PATH) and os.path.getmtime(WAIT_TEST_LIB_PATH) >= _newest_source_mtime():
        return WAIT_TEST_LIB_PATH
    return _compile(WAIT_TEST_LIB_PATH, defines=("SPX_WAIT_TEST=1", "SPX_WAIT_LIMIT_CYCLES=100000"))


if __name__ == "__main__":
    print(build(force=True, verbose=True))
