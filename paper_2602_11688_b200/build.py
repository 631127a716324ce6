"""Builds ``libgorgo_b200.so`` in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libgorgo_b200.so")
LIB_PROF = os.path.join(HERE, "libgorgo_b200_prof.so")
SOURCES = ["gorgo_kernels.cu", "gorgo_host.cu"]
HEADERS = ["gorgo_internal.h", os.path.join("..", "..", "include", "gorgo.h")]

NVCC_FLAGS = [
    "-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
    "-fmad=false",               # cost/time arithmetic must not be contracted into FMAs
    "--shared", "-Xcompiler", "-fPIC", "-Xcompiler", "-O2", "-cudart", "shared",
    "-Xcompiler", "-ffp-contract=off",   # host side too (Eq. 4 of the tuner): no fused multiply-add
]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def up_to_date(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return False
    t = os.path.getmtime(lib)
    deps = [os.path.join(CSRC, s) for s in SOURCES + HEADERS] + [os.path.abspath(__file__)]
    return all(os.path.getmtime(d) <= t for d in deps)


def _compile(lib: str, extra, verbose: bool) -> str:
    tmp = lib + f".tmp{os.getpid()}"
    cmd = [_nvcc()] + NVCC_FLAGS + list(extra) + (["-Xptxas", "-v"] if verbose else []) + \
          [os.path.join(CSRC, s) for s in SOURCES] + ["-o", tmp]
    subprocess.check_call(cmd)
    os.replace(tmp, lib)
    return lib


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and up_to_date():
        return LIB
    return _compile(LIB, [], verbose)


def build_phase_profile(force: bool = False, verbose: bool = False) -> str:
    """Second library with cycle accounting compiled into the replay kernel (-DGORGO_PROF);
    used only by ``phase_profile.py``, never by the product path."""
    if not force and up_to_date(LIB_PROF):
        return LIB_PROF
    return _compile(LIB_PROF, ["-DGORGO_PROF"], verbose)


if __name__ == "__main__":
    if "--phase-profile" in sys.argv:
        print(build_phase_profile(force="--force" in sys.argv, verbose="-v" in sys.argv))
    else:
        print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
