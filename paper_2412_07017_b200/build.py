"""Builds libasynclm.so (CUDA kernels + host planner + C ABI) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import glob
import os
import shutil
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
INCLUDE = os.path.join(os.path.dirname(HERE), "include")
LIB = os.path.join(CSRC, "libasynclm.so")
# A second build with per-CTA time stamps compiled in (-DASYNCLM_TRACE, asynclm_trace_read): for
# performance work only; the binding loads it when ASYNCLM_LIBRARY points at it.
TRACE_LIB = os.path.join(CSRC, "libasynclm_trace.so")
# A third build with device-side checks of every page id a kernel turns into an address (-DASYNCLM_DEBUG):
# a bad id sets the plan's status word and the access is left out.  For bringing up a new caller.
DEBUG_LIB = os.path.join(CSRC, "libasynclm_debug.so")

NVCC_FLAGS = [
    "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
    "--use_fast_math", "-Xcompiler", "-fPIC", "-shared", "--threads", "0",
]


def sources():
    return sorted(glob.glob(os.path.join(CSRC, "*.cu")))


def _inputs():
    return sources() + glob.glob(os.path.join(CSRC, "*.h")) + glob.glob(os.path.join(CSRC, "*.cuh")) \
        + glob.glob(os.path.join(INCLUDE, "*.h")) + [os.path.abspath(__file__)]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in _inputs())


def find_nvcc():
    nvcc = shutil.which("nvcc") or "/usr/local/cuda/bin/nvcc"
    return nvcc if os.path.exists(nvcc) else None


def build(force: bool = False, verbose: bool = False, trace: bool = False, debug: bool = False) -> str:
    lib = TRACE_LIB if trace else DEBUG_LIB if debug else LIB
    if not force and not trace and not debug and not is_stale():
        return lib
    nvcc = find_nvcc()
    if nvcc is None:
        raise RuntimeError("nvcc not found; cannot build libasynclm.so")
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [nvcc] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + \
        (["-DASYNCLM_TRACE"] if trace else []) + (["-DASYNCLM_DEBUG"] if debug else []) + ["-I", INCLUDE, "-I", CSRC, "-o", tmp] + sources()
    proc = subprocess.run(cmd, capture_output=True, text=True)
    if proc.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + proc.stdout + proc.stderr)
    if verbose:
        sys.stderr.write(proc.stderr)
    os.replace(tmp, lib)
    return lib


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv, trace="--trace" in sys.argv, debug="--debug" in sys.argv))
