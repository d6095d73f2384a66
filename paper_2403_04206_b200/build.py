"""In-tree build of libgrawa.so (nvcc, sm_100a only)."""
from __future__ import annotations

import os
import shutil
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_HERE)
CSRC = os.path.join(_HERE, "csrc")
LIB_PATH = os.path.join(_HERE, "libgrawa.so")
DEBUG_LIB_PATH = os.path.join(_HERE, "libgrawa_debug_bounds.so")
TRACE_LIB_PATH = os.path.join(_HERE, "libgrawa_trace.so")
SOURCES = [os.path.join(CSRC, "grawa.cu")]
HEADERS = [os.path.join(CSRC, "kernels.cuh"), os.path.join(CSRC, "center_pull_bulk.cuh"), os.path.join(CSRC, "kernels_16bit.cuh"), os.path.join(CSRC, "center_pull_staged_any.cuh"),
           os.path.join(_ROOT, "include", "grawa.h")]

# IEEE arithmetic throughout: no fast-math.
NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def _nvcc() -> str:
    exe = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    if not os.path.exists(exe):
        raise RuntimeError("nvcc not found: libgrawa.so cannot be built and there is no fallback path")
    return exe


def is_stale(path: str = LIB_PATH) -> bool:
    if not os.path.exists(path):
        return True
    t = os.path.getmtime(path)
    return any(os.path.getmtime(p) > t for p in SOURCES + HEADERS)


def _build_variant(path: str, define: str, force: bool) -> str:
    if force or is_stale(path):
        tmp = path + f".tmp{os.getpid()}"
        cmd = [_nvcc()] + NVCC_FLAGS + [define, "-o", tmp] + SOURCES
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
        os.replace(tmp, path)
    return path


def build(force: bool = False, verbose: bool = False, debug_bounds: bool = False, trace: bool = False) -> str:
    """Compile the CUDA library when missing or older than its sources; returns its path.
    debug_bounds: the variant whose kernels check their global accesses against the plan;
    trace: the variant whose kernels stamp the device timer (see grawa_trace_read)."""
    if debug_bounds:
        return _build_variant(DEBUG_LIB_PATH, "-DGRAWA_DEBUG_BOUNDS", force)
    if trace:
        return _build_variant(TRACE_LIB_PATH, "-DGRAWA_TRACE", force)
    if force or is_stale():
        tmp = LIB_PATH + f".tmp{os.getpid()}"
        cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + ["-o", tmp] + SOURCES
        res = subprocess.run(cmd, capture_output=True, text=True)
        if res.returncode != 0:
            raise RuntimeError("nvcc failed:\n" + " ".join(cmd) + "\n" + res.stdout + res.stderr)
        if verbose:
            print(res.stderr)
        os.replace(tmp, LIB_PATH)
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
