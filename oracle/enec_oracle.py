"""ctypes binding of the ENEC oracle (TEST INFRASTRUCTURE, NOT THE PRODUCT).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this module. It loads
``oracle/libenec_oracle.so`` (built from ``enec_oracle.cpp`` by ``oracle/build.py``) and marshals numpy
arrays; every step of the codec runs in the C++ oracle.
"""
import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = None

BF16, FP16, FP32 = 0, 1, 2


def lib():
    global _LIB
    if _LIB is None:
        import importlib.util
        spec = importlib.util.spec_from_file_location("_enec_oracle_build", os.path.join(_HERE, "build.py"))
        mod = importlib.util.module_from_spec(spec)
        spec.loader.exec_module(mod)
        L = C.CDLL(mod.build())
        L.enec_oracle_split.argtypes = [C.c_uint32, C.c_int, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
        L.enec_oracle_split.restype = None
        L.enec_oracle_join.argtypes = [C.c_uint32, C.c_uint32, C.c_int]
        L.enec_oracle_join.restype = C.c_uint32
        L.enec_oracle_width_eq1.argtypes = [C.c_int] * 4
        L.enec_oracle_width_eq1.restype = C.c_int
        L.enec_oracle_transform.argtypes = [C.c_uint32, C.c_int, C.c_int]
        L.enec_oracle_transform.restype = C.c_uint32
        L.enec_oracle_inverse_transform.argtypes = [C.c_uint32, C.c_int, C.c_int, C.c_int]
        L.enec_oracle_inverse_transform.restype = C.c_uint32
        L.enec_oracle_param_search.argtypes = [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int),
                                               C.POINTER(C.c_int), C.c_void_p, C.c_void_p]
        L.enec_oracle_param_search.restype = None
        L.enec_oracle_alg2_pack.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_void_p]
        L.enec_oracle_alg2_pack.restype = C.c_size_t
        L.enec_oracle_alg2_unpack.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_void_p]
        L.enec_oracle_alg2_unpack.restype = None
        L.enec_oracle_max_compressed_size.argtypes = [C.c_int, C.c_size_t]
        L.enec_oracle_max_compressed_size.restype = C.c_size_t
        L.enec_oracle_max_compressed_size_ranked.argtypes = [C.c_int, C.c_size_t]
        L.enec_oracle_max_compressed_size_ranked.restype = C.c_size_t
        L.enec_oracle_compress_ranked.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_void_p, C.c_size_t,
                                                  C.POINTER(C.c_size_t)]
        L.enec_oracle_compress_ranked.restype = C.c_int
        L.enec_oracle_compress.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_void_p, C.c_size_t,
                                           C.POINTER(C.c_size_t)]
        L.enec_oracle_compress.restype = C.c_int
        L.enec_oracle_max_compressed_size_blockwise.argtypes = [C.c_int, C.c_size_t]
        L.enec_oracle_max_compressed_size_blockwise.restype = C.c_size_t
        L.enec_oracle_compress_blockwise.argtypes = L.enec_oracle_compress.argtypes
        L.enec_oracle_compress_blockwise.restype = C.c_int
        L.enec_oracle_compress_with_params.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_int,
                                                       C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t)]
        L.enec_oracle_compress_with_params.restype = C.c_int
        L.enec_oracle_decompress.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_size_t, C.c_void_p]
        L.enec_oracle_decompress.restype = C.c_int
        _LIB = L
    return _LIB


class OracleError(RuntimeError):
    def __init__(self, status):
        super().__init__(f"oracle status {status}")
        self.status = status


def split(w, dtype):
    x, sm = C.c_uint32(), C.c_uint32()
    lib().enec_oracle_split(int(w), dtype, C.byref(x), C.byref(sm))
    return x.value, sm.value


def join(x, sm, dtype):
    return lib().enec_oracle_join(int(x), int(sm), dtype)


def width_eq1(b, l, h, E):
    return lib().enec_oracle_width_eq1(b, l, h, E)


def transform(x, b, n):
    return lib().enec_oracle_transform(int(x), b, n)


def inverse_transform(y, b, n, E):
    return lib().enec_oracle_inverse_transform(int(y), b, n, E)


def param_search(hist, E):
    """Returns (b, n, m, cost[2^E], bexp[9])."""
    hist = np.ascontiguousarray(hist, dtype=np.uint64)
    assert hist.size == 1 << E
    cost = np.empty(1 << E, dtype=np.uint64)
    bexp = np.empty(9, dtype=np.float64)
    b, n, m = C.c_int(), C.c_int(), C.c_int()
    lib().enec_oracle_param_search(hist.ctypes.data, E, C.byref(b), C.byref(n), C.byref(m),
                                   cost.ctypes.data, bexp.ctypes.data)
    return b.value, n.value, m.value, cost, bexp


def alg2_pack(data, a):
    data = np.ascontiguousarray(data, dtype=np.uint16)
    out = np.zeros(data.size * 2 + 2, dtype=np.uint8)
    nbytes = lib().enec_oracle_alg2_pack(data.ctypes.data, data.size, a, out.ctypes.data)
    return out[:nbytes].copy()


def alg2_unpack(stream, N, a):
    stream = np.ascontiguousarray(stream, dtype=np.uint8)
    out = np.empty(N, dtype=np.uint16)
    lib().enec_oracle_alg2_unpack(stream.ctypes.data, N, a, out.ctypes.data)
    return out


def max_compressed_size(dtype, count):
    return lib().enec_oracle_max_compressed_size(dtype, count)


def compress(words, dtype, params=None):
    """words: numpy array of raw bit patterns (uint16 for bf16/fp16, uint32 for fp32). Returns the stream as a
    uint8 array."""
    words = np.ascontiguousarray(words, dtype=np.uint32 if dtype == FP32 else np.uint16).reshape(-1)
    cap = max_compressed_size(dtype, words.size)
    out = np.empty(cap, dtype=np.uint8)
    size = C.c_size_t(0)
    if params is None:
        st = lib().enec_oracle_compress(words.ctypes.data, dtype, words.size, out.ctypes.data, cap, C.byref(size))
    else:
        b, n, m = params
        st = lib().enec_oracle_compress_with_params(words.ctypes.data, dtype, words.size, b, n, m,
                                                    out.ctypes.data, cap, C.byref(size))
    if st != 0:
        raise OracleError(st)
    return out[:size.value].copy()


def compress_ranked(words, dtype):
    """The frequency-rank variant of compress(): same stream sections plus the rank -> exponent table."""
    words = np.ascontiguousarray(words, dtype=np.uint32 if dtype == FP32 else np.uint16).reshape(-1)
    cap = lib().enec_oracle_max_compressed_size_ranked(dtype, words.size)
    out = np.empty(cap, dtype=np.uint8)
    size = C.c_size_t(0)
    st = lib().enec_oracle_compress_ranked(words.ctypes.data, dtype, words.size, out.ctypes.data, cap, C.byref(size))
    if st != 0:
        raise OracleError(st)
    return out[:size.value].copy()


def max_compressed_size_blockwise(dtype, count):
    return lib().enec_oracle_max_compressed_size_blockwise(dtype, count)


def compress_blockwise(words, dtype):
    """The block-wise variant of compress(): every block chooses its own (b, n, m)."""
    words = np.ascontiguousarray(words, dtype=np.uint32 if dtype == FP32 else np.uint16).reshape(-1)
    cap = max_compressed_size_blockwise(dtype, words.size)
    out = np.empty(cap, dtype=np.uint8)
    size = C.c_size_t(0)
    st = lib().enec_oracle_compress_blockwise(words.ctypes.data, dtype, words.size, out.ctypes.data, cap, C.byref(size))
    if st != 0:
        raise OracleError(st)
    return out[:size.value].copy()


def decompress(stream, dtype, count):
    stream = np.ascontiguousarray(stream, dtype=np.uint8)
    out = np.empty(count, dtype=np.uint32 if dtype == FP32 else np.uint16)
    st = lib().enec_oracle_decompress(stream.ctypes.data, stream.size, dtype, count, out.ctypes.data)
    if st != 0:
        raise OracleError(st)
    return out
