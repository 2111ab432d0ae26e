"""Builds and loads the small CUDA helpers that only the tests use (tests/csrc)."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "csrc", "early_trigger.cu")
LIB = os.path.join(HERE, "libst3_testkernels.so")


def build(force: bool = False) -> str:
    if force or not os.path.exists(LIB) or os.path.getmtime(SRC) > os.path.getmtime(LIB):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-shared", "-Xcompiler",
                        "-fPIC", "-o", LIB, SRC], check=True)
    return LIB


def load():
    lib = C.CDLL(build())
    lib.st3_test_early_trigger_copy.argtypes = [C.c_void_p, C.c_void_p, C.c_size_t, C.c_int, C.c_void_p]
    lib.st3_test_early_trigger_copy.restype = C.c_int
    return lib
