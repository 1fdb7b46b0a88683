"""ctypes wrapper of the vectorised CPU codec (a host baseline for the benchmark; not used by the CUDA library).

`build()` compiles enec_cpu.cpp with g++ (-mavx2 -mbmi2); `available()` says whether this machine can run it.
"""
import ctypes as C
import os
import subprocess

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(HERE, "enec_cpu.cpp")
LIB = os.path.join(HERE, "libenec_cpu.so")
_lib = None


def available() -> bool:
    try:
        flags = open("/proc/cpuinfo").read()
    except OSError:
        return False
    return " avx2" in flags and " bmi2" in flags


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    subprocess.run(["g++", "-std=c++17", "-O3", "-mavx2", "-mbmi2", "-ffp-contract=off", "-fPIC", "-shared", "-pthread",
                    "-Wall", "-o", LIB, SRC], check=True)
    return LIB


def lib():
    global _lib
    if _lib is None:
        if not available():
            raise RuntimeError("this CPU has no AVX2/BMI2")
        L = C.CDLL(build())
        L.enec_cpu_max_compressed_size.argtypes = [C.c_int, C.c_size_t]
        L.enec_cpu_max_compressed_size.restype = C.c_size_t
        L.enec_cpu_compress.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_void_p, C.c_size_t, C.c_int]
        L.enec_cpu_compress.restype = C.c_size_t
        L.enec_cpu_decompress.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_size_t, C.c_void_p, C.c_int]
        L.enec_cpu_decompress.restype = C.c_int
        _lib = L
    return _lib


def compress(words: np.ndarray, dtype: int, threads: int = 0) -> np.ndarray:
    """words: raw bit patterns (uint16 for bf16/fp16, uint32 for fp32). Returns the stream as uint8."""
    words = np.ascontiguousarray(words)
    cap = lib().enec_cpu_max_compressed_size(dtype, words.size)
    out = np.empty(cap, dtype=np.uint8)
    n = lib().enec_cpu_compress(words.ctypes.data, dtype, words.size, out.ctypes.data, cap, threads)
    if n == 0:
        raise ValueError("enec_cpu_compress: bad arguments")
    return out[:n]


def decompress(stream: np.ndarray, dtype: int, count: int, threads: int = 0) -> np.ndarray:
    stream = np.ascontiguousarray(stream)
    out = np.empty(count, dtype=np.uint32 if dtype == 2 else np.uint16)
    if lib().enec_cpu_decompress(stream.ctypes.data, stream.size, dtype, count, out.ctypes.data, threads) != 0:
        raise ValueError("enec_cpu_decompress: bad stream")
    return out


def compress_into(words: np.ndarray, dtype: int, out: np.ndarray, threads: int = 0) -> int:
    """Compresses into a caller's uint8 buffer (at least max size); returns the stream length."""
    n = lib().enec_cpu_compress(words.ctypes.data, dtype, words.size, out.ctypes.data, out.size, threads)
    if n == 0:
        raise ValueError("enec_cpu_compress: bad arguments")
    return n


def decompress_into(stream: np.ndarray, nbytes: int, dtype: int, out: np.ndarray, threads: int = 0) -> None:
    if lib().enec_cpu_decompress(stream.ctypes.data, nbytes, dtype, out.size, out.ctypes.data, threads) != 0:
        raise ValueError("enec_cpu_decompress: bad stream")


def max_compressed_size(dtype: int, count: int) -> int:
    return lib().enec_cpu_max_compressed_size(dtype, count)
