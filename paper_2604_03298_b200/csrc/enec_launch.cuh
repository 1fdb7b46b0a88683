// Host-side launch helpers shared by the library's translation units.
#pragma once

#include <atomic>
#include <cuda_runtime.h>
#include <stdint.h>

#include "enec.h"

namespace enec {

extern std::atomic<uint64_t> g_launches;  // kernels launched by the library (enec_launch_count)
constexpr int kMaxDevices = 64;  // device ordinals the per-device tables cover; calls on others fail with ENEC_ERR_CUDA

struct DecodeBatch;
// Launches the decode kernel instance for dt (and for the frequency-rank variant when ranked) over `batch`.
// ticketed: 1 = the batch's device arrays carry a ticket word and the chunk table, 2 = one tensor with a ticket word
// of the library's scratch (see DecodeBatch and enec_decode_kernel), 0 = fixed shares of the blocks.
enec_status launch_decode_any(int dt, const DecodeBatch& batch, int* d_status, cudaStream_t stream, bool ranked,
                              int ticketed = 0);

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor in the
// stream drains; it waits for the predecessor's completion itself (pdl_wait) before touching memory.
template <class... KernelArgs, class... Args>
inline cudaError_t launch_pdl(void (*kernel)(KernelArgs...), uint32_t grid, uint32_t threads, size_t smem,
                              cudaStream_t stream, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(threads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KernelArgs(args)...);
}

}  // namespace enec
