"""Builds libhap.so (the C-ABI CUDA library) in-tree with nvcc for sm_100a."""
from __future__ import annotations

import os
import subprocess

_DIR = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(_DIR, "libhap.so")
LIB_CHECKED = os.path.join(_DIR, "libhap_checked.so")      # the same sources with -DHAP_CHECKED (self-checking kernels)
SOURCES = [os.path.join(_DIR, "csrc", "hap_api.cu")]
HEADERS = [os.path.join(_DIR, "csrc", "hap_device.cuh"), os.path.join(_DIR, "csrc", "hap_trie.cuh"), os.path.join(os.path.dirname(_DIR), "include", "hap.h")]

NVCC_FLAGS = ["-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "--fmad=false", "-std=c++17",
              "-shared", "-Xcompiler", "-fPIC"]


def is_stale(lib: str = LIB) -> bool:
    if not os.path.exists(lib):
        return True
    t = os.path.getmtime(lib)
    return any(os.path.getmtime(f) > t for f in SOURCES + HEADERS)


def build_library(force: bool = False, verbose: bool = False, checked: bool = False) -> str:
    """Compile the library (or its self-checking variant) if it is missing or older than its sources; returns its path."""
    lib = LIB_CHECKED if checked else LIB
    if force or is_stale(lib):
        nvcc = os.environ.get("NVCC", "nvcc")
        cmd = [nvcc, *NVCC_FLAGS, *(["-DHAP_CHECKED"] if checked else []), *(["-Xptxas", "-v"] if verbose else []), "-o", lib, *SOURCES]
        subprocess.run(cmd, check=True)
    return lib
