"""Builds the C-ABI shared library (libwg.so) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess
import sys

PKG = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(PKG)
CSRC = os.path.join(PKG, "csrc")
LIB = os.path.join(PKG, "libwg.so")
SOURCES = ["wg_api.cu", "wg_lower.cpp", "wg_regex.cpp", "wg_template.cpp"]
HEADERS = [os.path.join(CSRC, "wg_kernels.cuh"), os.path.join(CSRC, "wg_internal.h"),
           os.path.join(ROOT, "include", "wg.h")]
NVCC_FLAGS = ["-O3", "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo",
              "-Xcompiler", "-fPIC", "-shared", "-cudart", "shared", "-ldl"]


def _nvcc() -> str:
    cand = os.path.join(os.environ.get("CUDA_HOME", "/usr/local/cuda"), "bin", "nvcc")
    return cand if os.path.exists(cand) else "nvcc"


def needs_build() -> bool:
    if not os.path.exists(LIB):
        return True
    built = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, s) for s in SOURCES] + HEADERS
    return any(os.path.getmtime(d) > built for d in deps)


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not needs_build():
        return LIB
    tmp = LIB + f".tmp{os.getpid()}"
    cmd = [_nvcc()] + NVCC_FLAGS + (["-Xptxas", "-v"] if verbose else []) + [
        "-I", os.path.join(ROOT, "include"), "-I", CSRC, "-o", tmp] + [
        os.path.join(CSRC, s) for s in SOURCES]
    subprocess.check_call(cmd)
    os.replace(tmp, LIB)
    return LIB


def ensure() -> str:
    """The library, built if it is missing; a library that only looks older than its sources
    (file times change when a tree is copied) is rebuilt when nvcc is there and kept otherwise."""
    if not os.path.exists(LIB):
        return build(force=True)
    if needs_build():
        try:
            return build(force=True)
        except (OSError, subprocess.CalledProcessError):
            pass
    return LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
