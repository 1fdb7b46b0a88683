"""ctypes binding of libenec.so. Argument marshalling only."""
import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libenec.so")
_LIB = None

BF16, FP16, FP32 = 0, 1, 2
_DT = {torch.bfloat16: BF16, torch.float16: FP16, torch.float32: FP32}

STATUS_NAMES = {0: "ENEC_OK", -1: "ENEC_ERR_INVALID_ARG", -2: "ENEC_ERR_UNSUPPORTED_DTYPE",
                -3: "ENEC_ERR_BUFFER_TOO_SMALL", -4: "ENEC_ERR_BAD_STREAM",
                -5: "ENEC_ERR_PARAMS_NOT_LOSSLESS", -6: "ENEC_ERR_TIMEOUT", -7: "ENEC_ERR_CUDA",
                -8: "ENEC_ERR_TOO_LARGE"}


class EnecError(RuntimeError):
    def __init__(self, status, where=""):
        super().__init__(f"{where}: {STATUS_NAMES.get(status, status)}")
        self.status = status


class BatchItem(C.Structure):
    _fields_ = [("d_in", C.c_void_p), ("d_out", C.c_void_p), ("count", C.c_size_t), ("size", C.c_size_t)]


def lib():
    """Loads libenec.so (built in-tree by ``build.py``). Raises if it is missing: there is no fallback."""
    global _LIB
    if _LIB is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} not found: build it with `python -m paper_2604_03298_b200.build` "
                               "(no CPU fallback exists)")
        L = C.CDLL(_LIB_PATH)
        L.enec_max_compressed_size.argtypes = [C.c_int, C.c_size_t]
        L.enec_max_compressed_size.restype = C.c_size_t
        L.enec_compress.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p,
                                    C.c_void_p, C.c_void_p]
        L.enec_compress.restype = C.c_int
        L.enec_compress_noalloc.argtypes = L.enec_compress.argtypes
        L.enec_compress_noalloc.restype = C.c_int
        L.enec_compress_ranked.argtypes = L.enec_compress.argtypes
        L.enec_compress_ranked.restype = C.c_int
        L.enec_max_compressed_size_ranked.argtypes = [C.c_int, C.c_size_t]
        L.enec_max_compressed_size_ranked.restype = C.c_size_t
        L.enec_compress_blockwise.argtypes = L.enec_compress.argtypes
        L.enec_compress_blockwise.restype = C.c_int
        L.enec_max_compressed_size_blockwise.argtypes = [C.c_int, C.c_size_t]
        L.enec_max_compressed_size_blockwise.restype = C.c_size_t
        L.enec_compress_with_params.argtypes = [C.c_void_p, C.c_int, C.c_size_t, C.c_int, C.c_int, C.c_int,
                                                C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p, C.c_void_p]
        L.enec_compress_with_params.restype = C.c_int
        L.enec_decompress.argtypes = [C.c_void_p, C.c_size_t, C.c_int, C.c_size_t, C.c_void_p, C.c_void_p,
                                      C.c_void_p]
        L.enec_decompress.restype = C.c_int
        L.enec_decompress_ranked.argtypes = L.enec_decompress.argtypes
        L.enec_decompress_ranked.restype = C.c_int
        L.enec_decompress_blockwise.argtypes = L.enec_decompress.argtypes
        L.enec_decompress_blockwise.restype = C.c_int
        L.enec_decompress_batched.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.enec_decompress_batched.restype = C.c_int
        L.enec_compress_batched.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.enec_compress_batched.restype = C.c_int
        L.enec_launch_count.argtypes = []
        L.enec_launch_count.restype = C.c_uint64
        L.enec_allocation_count.argtypes = []
        L.enec_allocation_count.restype = C.c_uint64
        L.enec_version.argtypes = []
        L.enec_version.restype = C.c_int
        _LIB = L
    return _LIB


def _stream():
    # raw handle of torch's current stream on the current device (an integer; 0 is the legacy default stream)
    return torch._C._cuda_getCurrentRawStream(torch.cuda.current_device())


def _ptr(t):
    return t.data_ptr() if t is not None else None


def enec_max_compressed_size(dt: int, count: int) -> int:
    return lib().enec_max_compressed_size(dt, count)


def enec_compress(d_in, dt, count, d_out, out_capacity, d_out_size=None, d_status=None) -> int:
    """d_in/d_out/d_out_size/d_status: CUDA tensors (or None). Enqueues on the current stream; returns status."""
    return lib().enec_compress(_ptr(d_in), dt, count, _ptr(d_out), out_capacity, _ptr(d_out_size),
                               _ptr(d_status), _stream())


def enec_compress_noalloc(d_in, dt, count, d_out, out_capacity, d_out_size=None, d_status=None) -> int:
    """enec_compress with the library's built-in scratch array instead of allocated scratch: for callers that
    must not allocate device memory. At most 2^30 values; calls that overlap on the GPU must not share a device."""
    return lib().enec_compress_noalloc(_ptr(d_in), dt, count, _ptr(d_out), out_capacity, _ptr(d_out_size),
                                       _ptr(d_status), _stream())


def enec_max_compressed_size_ranked(dt: int, count: int) -> int:
    return lib().enec_max_compressed_size_ranked(dt, count)


def enec_compress_ranked(d_in, dt, count, d_out, out_capacity, d_out_size=None, d_status=None) -> int:
    """The frequency-rank variant of enec_compress (ablation): same arguments, 256 bytes more capacity."""
    return lib().enec_compress_ranked(_ptr(d_in), dt, count, _ptr(d_out), out_capacity, _ptr(d_out_size),
                                      _ptr(d_status), _stream())


def enec_max_compressed_size_blockwise(dt: int, count: int) -> int:
    return lib().enec_max_compressed_size_blockwise(dt, count)


def enec_compress_blockwise(d_in, dt, count, d_out, out_capacity, d_out_size=None, d_status=None) -> int:
    """The block-wise variant of enec_compress (ablation): every 16384-element block gets its own (b, n, m)."""
    return lib().enec_compress_blockwise(_ptr(d_in), dt, count, _ptr(d_out), out_capacity, _ptr(d_out_size),
                                         _ptr(d_status), _stream())


def enec_decompress_blockwise(d_in, in_size, dt, count, d_out, d_status=None) -> int:
    """Decompresses a stream written by enec_compress_blockwise."""
    return lib().enec_decompress_blockwise(_ptr(d_in), in_size, dt, count, _ptr(d_out), _ptr(d_status), _stream())


def enec_compress_with_params(d_in, dt, count, b, n, m, d_out, out_capacity, d_out_size=None, d_status=None) -> int:
    return lib().enec_compress_with_params(_ptr(d_in), dt, count, b, n, m, _ptr(d_out), out_capacity,
                                           _ptr(d_out_size), _ptr(d_status), _stream())


def enec_decompress(d_in, in_size, dt, count, d_out, d_status=None) -> int:
    return lib().enec_decompress(_ptr(d_in), in_size, dt, count, _ptr(d_out), _ptr(d_status), _stream())


def make_batch(items):
    """The C array of enec_batch_item for a list of (in_tensor, out_tensor, count, size) tuples. A caller that
    repeats a batched call on the same buffers can build it once and pass it instead of the list."""
    arr = (BatchItem * len(items))()
    for i, (src, dst, count, size) in enumerate(items):
        arr[i].d_in, arr[i].d_out, arr[i].count, arr[i].size = src.data_ptr(), dst.data_ptr(), count, size
    return arr


def enec_decompress_ranked(d_in, in_size, dt, count, d_out, d_status=None) -> int:
    """Decompresses a stream written by enec_compress_ranked."""
    return lib().enec_decompress_ranked(_ptr(d_in), in_size, dt, count, _ptr(d_out), _ptr(d_status), _stream())


def enec_decompress_batched(items, dt, d_status=None) -> int:
    """items: list of (stream_tensor, stream_bytes, out_tensor, count), or a make_batch() array."""
    arr = items if isinstance(items, C.Array) else make_batch([(src, dst, count, nbytes) for src, nbytes, dst, count in items])
    return lib().enec_decompress_batched(C.cast(arr, C.c_void_p), len(arr), dt, _ptr(d_status), _stream())


def enec_compress_batched(items, dt, d_out_sizes=None, d_status=None) -> int:
    """items: list of (tensor, stream_buffer, count, capacity), or a make_batch() array; d_out_sizes: int64 CUDA
    tensor [len(items)] or None."""
    arr = items if isinstance(items, C.Array) else make_batch(items)
    return lib().enec_compress_batched(C.cast(arr, C.c_void_p), len(arr), dt, _ptr(d_out_sizes), _ptr(d_status),
                                       _stream())


def enec_launch_count() -> int:
    return lib().enec_launch_count()


def enec_allocation_count() -> int:
    return lib().enec_allocation_count()


# ---- convenience wrappers (allocation with torch, status check) --------------------------------------
def compress_tensor(t: torch.Tensor, params=None) -> torch.Tensor:
    """Compresses a CUDA bf16/fp16/fp32 tensor; returns the stream as a uint8 CUDA tensor (synchronises once to
    read the stream length)."""
    dt = _DT[t.dtype]
    t = t.contiguous()
    count = t.numel()
    cap = enec_max_compressed_size(dt, count)
    out = torch.empty(cap, dtype=torch.uint8, device=t.device)
    meta = torch.zeros(2, dtype=torch.int64, device=t.device)   # [0] = size, [1] = status
    status = meta[1:].view(torch.int32)
    if params is None:
        st = enec_compress(t, dt, count, out, cap, meta, status)
    else:
        st = enec_compress_with_params(t, dt, count, *params, out, cap, meta, status)
    if st != 0:
        raise EnecError(st, "enec_compress")
    size, dev_status = meta.tolist()
    dev_status = dev_status & 0xFFFFFFFF
    dev_status = dev_status - (1 << 32) if dev_status & 0x80000000 else dev_status
    if dev_status != 0:
        raise EnecError(dev_status, "enec_compress (device)")
    return out[:size]


def decompress_tensor(stream: torch.Tensor, dtype: torch.dtype, shape) -> torch.Tensor:
    dt = _DT[dtype]
    out = torch.empty(shape, dtype=dtype, device=stream.device)
    status = torch.zeros(1, dtype=torch.int32, device=stream.device)
    st = enec_decompress(stream, stream.numel(), dt, out.numel(), out, status)
    if st != 0:
        raise EnecError(st, "enec_decompress")
    dev_status = int(status.item())
    if dev_status != 0:
        raise EnecError(dev_status, "enec_decompress (device)")
    return out
