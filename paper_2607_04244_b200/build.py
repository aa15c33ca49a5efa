"""Builds libqlinear_w4a16.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

PKG_DIR = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(PKG_DIR, "csrc")
LIB_PATH = os.path.join(PKG_DIR, "libqlinear_w4a16.so")
LIB_PATH_TIMELINE = os.path.join(PKG_DIR, "libqlinear_w4a16_timeline.so")   # same library built with -DQL_TIMELINE
SOURCES = ["api.cu", "qpack.cu", "glue.cu", "qlinear_mma.cu", "qlinear_tc5.cu", "qstack_tc5.cu", "qlinear_static.cu", "qattn_swa.cu"]
HEADERS = ["ql_device.cuh", "ql_params.h", os.path.join("..", "..", "include", "qlinear_w4a16.h")]
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "--shared", "-Xcompiler", "-fPIC"]


def _stale(lib_path: str = LIB_PATH) -> bool:
    if not os.path.exists(lib_path):
        return True
    t = os.path.getmtime(lib_path)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps)


def build_library(force: bool = False, verbose: bool = False, timeline: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; returns its path.
    timeline=True builds the instrumented twin (the stack kernel stamps its phases with globaltimer)."""
    lib_path = LIB_PATH_TIMELINE if timeline else LIB_PATH
    if not force and not _stale(lib_path):
        return lib_path
    nvcc = os.environ.get("NVCC", "nvcc")
    cmd = [nvcc] + NVCC_FLAGS + (["-DQL_TIMELINE"] if timeline else []) + (["-Xptxas", "-v"] if verbose else []) + \
          ["-o", lib_path] + [os.path.join(CSRC, s) for s in SOURCES]
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    return lib_path


if __name__ == "__main__":
    print(build_library(force="--force" in sys.argv, verbose="-v" in sys.argv, timeline="--timeline" in sys.argv))
