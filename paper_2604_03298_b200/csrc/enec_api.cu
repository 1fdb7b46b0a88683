// C-ABI entry points of libenec (see include/enec.h). Host-side validation and kernel launches only.
#include <atomic>
#include <mutex>

#include "enec_decode.cuh"

namespace enec {

std::atomic<uint64_t> g_launches{0};

struct DeviceInfo {
    int sms = 0;
    bool decode_attr_set[2] = {false, false};
};

static DeviceInfo& device_info(int dev) {
    static std::mutex mu;
    static DeviceInfo infos[64];
    std::lock_guard<std::mutex> lock(mu);
    DeviceInfo& d = infos[dev & 63];
    if (d.sms == 0) cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    return d;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

template <int DT>
static enec_status launch_decode(const DecodeJob& job, uint32_t nblocks, int* d_status, cudaStream_t stream) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
    DeviceInfo& info = device_info(dev);
    if (!info.decode_attr_set[DT]) {
        if (cudaFuncSetAttribute(enec_decode_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kDecodeSmemBytes)) != cudaSuccess)
            return ENEC_ERR_CUDA;
        info.decode_attr_set[DT] = true;
    }
    uint32_t grid = uint32_t(info.sms) * 3;
    if (grid > nblocks) grid = nblocks;
    if (grid == 0) grid = 1;
    enec_decode_kernel<DT><<<grid, kDecodeThreads, kDecodeSmemBytes, stream>>>(job, d_status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? ENEC_OK : ENEC_ERR_CUDA;
}

}  // namespace enec

using namespace enec;

extern "C" {

size_t enec_max_compressed_size(enec_dtype dt, size_t count) {
    if ((dt != ENEC_BF16 && dt != ENEC_FP16) || (uint64_t(count) >> 36)) return 0;
    const int E = exp_bits(dt);
    const Geometry g = make_geometry(count);
    uint64_t worst = 0;
    for (int m = 1; m <= E; ++m) {
        const uint64_t t = make_sections(dt, count, g, E, m, g.total_groups).total;
        if (t > worst) worst = t;
    }
    return size_t(worst);
}

enec_status enec_decompress(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                            int* d_status, enec_stream_t stream) {
    if (dt != ENEC_BF16 && dt != ENEC_FP16) return ENEC_ERR_UNSUPPORTED_DTYPE;
    if (!d_in || (!d_out && count) || (uint64_t(count) >> 36) || !aligned16(d_in) || !aligned16(d_out))
        return ENEC_ERR_INVALID_ARG;
    if (in_size < kHeaderBytes + 16) return ENEC_ERR_BAD_STREAM;
    DecodeJob job{static_cast<const uint8_t*>(d_in), static_cast<uint16_t*>(d_out), uint64_t(count), uint64_t(in_size)};
    const Geometry g = make_geometry(count);
    return dt == ENEC_BF16 ? launch_decode<ENEC_BF16>(job, g.nblocks, d_status, stream)
                           : launch_decode<ENEC_FP16>(job, g.nblocks, d_status, stream);
}

enec_status enec_compress(const void*, enec_dtype, size_t, void*, size_t, size_t*, int*, enec_stream_t) {
    return ENEC_ERR_CUDA;  // TEMP
}
enec_status enec_compress_with_params(const void*, enec_dtype, size_t, int, int, int, void*, size_t, size_t*, int*,
                                      enec_stream_t) {
    return ENEC_ERR_CUDA;  // TEMP
}
enec_status enec_decompress_batched(const enec_batch_item*, int, enec_dtype, int*, enec_stream_t) {
    return ENEC_ERR_CUDA;  // TEMP
}

uint64_t enec_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int enec_version(void) { return 100; }

}  // extern "C"
