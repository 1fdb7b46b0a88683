"""B200-native ENEC codec: thin Python binding over the C-ABI CUDA library ``libenec.so``.

The functions here have the names of the C entry points declared in ``include/enec.h`` and only marshal
arguments (device pointers of torch tensors, sizes, the current CUDA stream). Every step of the codec
runs in the library's CUDA kernels. There is no CPU fallback: importing works without a GPU, but any call
raises if the library is missing.
"""
from .binding import (  # noqa: F401
    BF16, FP16, FP32, EnecError, lib, make_batch, enec_max_compressed_size, enec_compress, enec_compress_with_params, enec_compress_noalloc,
    enec_compress_batched, enec_compress_ranked, enec_max_compressed_size_ranked,
    enec_compress_blockwise, enec_max_compressed_size_blockwise, enec_decompress_blockwise, enec_decompress, enec_decompress_ranked, enec_decompress_batched, enec_launch_count, enec_allocation_count, compress_tensor, decompress_tensor,
)
