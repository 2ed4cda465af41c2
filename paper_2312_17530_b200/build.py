"""Builds the CUDA library in-tree with nvcc for sm_100a (no JIT cache, no torch extension)."""
from __future__ import annotations

import os
import subprocess
import sys

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "librsdgc_b200.so")
SOURCES = ["plan.cu", "accumulate_nsi.cu", "compress.cu", "ratio.cu", "decompress.cu", "ratio_noalloc.cu", "coo.cu", "tail.cu"]
HEADERS = ["rsdgc_internal.cuh", "device_utils.cuh", "ratio_common.cuh"]


def _stale() -> bool:
    if not os.path.exists(LIB_PATH):
        return True
    t = os.path.getmtime(LIB_PATH)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS] + [os.path.join(_ROOT, "include", "rsdgc.h")]
    return any(os.path.getmtime(d) > t for d in deps)


DEBUG_LIB_PATH = os.path.join(_HERE, "librsdgc_b200_debug.so")


def build_library(force: bool = False, verbose: bool = False, debug: bool = False) -> str:
    """nvcc -> librsdgc_b200.so next to this file; returns its path.  ``debug``: the bounds-checked
    build (-DRSDGC_DEBUG: every index the kernels form is tested against the plan's extents, failures
    raise RSDGC_STATUS_BOUNDS and skip the access) -> librsdgc_b200_debug.so; load it by pointing the
    environment variable RSDGC_LIBRARY at it."""
    if debug:
        return _compile(DEBUG_LIB_PATH, verbose, ["-DRSDGC_DEBUG"])
    if not force and not _stale():
        return LIB_PATH
    return _compile(LIB_PATH, verbose, [])


def _compile(out_path: str, verbose: bool, extra) -> str:
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    tmp = out_path + ".tmp.%d" % os.getpid()
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC,-Wall", "-shared", "-I", os.path.join(_ROOT, "include"), "-I", CSRC,
           "-o", tmp] + list(extra) + [os.path.join(CSRC, s) for s in SOURCES]
    # NVTX ranges around the entry points (header-only NVTX 3; RSDGC_NVTX=0 compiles them out)
    if os.environ.get("RSDGC_NVTX", "1") != "0":
        cmd[1:1] = ["-DRSDGC_NVTX"]
        cmd += ["-ldl"]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if verbose:
        sys.stderr.write(res.stderr)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    os.replace(tmp, out_path)
    return out_path


if __name__ == "__main__":
    print(build_library(force=True, verbose="-v" in sys.argv, debug="--debug" in sys.argv))
