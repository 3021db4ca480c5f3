"""Builds libhap.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(_DIR, "libhap.so")
SOURCES = [os.path.join(_DIR, "csrc", "hap_api.cu")]
HEADERS = [os.path.join(_DIR, "csrc", "hap_device.cuh"), os.path.join(_DIR, "csrc", "hap_trie.cuh"), os.path.join(os.path.dirname(_DIR), "include", "hap.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "--fmad=false", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def is_stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build_library(force: bool = False, verbose: bool = False) -> str:
    """Compile the library if it is missing or older than its sources; returns its path."""
    if force or is_stale():
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc, *NVCC_FLAGS, *( ["-Xptxas", "-v"] if verbose else []), "-o", LIB, *SOURCES]
        subprocess.run(cmd, check=True)
    return LIB
