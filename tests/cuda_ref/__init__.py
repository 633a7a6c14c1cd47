"""Test-only naive FP64 GPU matmul (tests/cuda_ref/naive_gemm.cu): built with nvcc next to its source and loaded
with ctypes.  Not part of the library and not used by it."""
import ctypes
import os
import subprocess

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "naive_gemm.cu")
LIB = os.path.join(HERE, "libnaive_gemm.so")


def build(force=False):
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(SRC):
        nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
        subprocess.run([nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O2", "-shared", "-Xcompiler", "-fPIC", SRC, "-o", LIB], check=True)
    return LIB


def load():
    lib = ctypes.CDLL(build())
    lib.naive_gemm_f64.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64]
    lib.naive_gemm_f64.restype = ctypes.c_int
    return lib
