// The launch of a decode kernel instance, shared by the per-dtype translation units (the decode kernels'
// instances are most of the library's compile time, so each dtype is compiled on its own).
#pragma once

#include <mutex>

#include "enec_decode.cuh"
#include "enec_launch.cuh"

namespace enec {

struct DecodeDevice {
    int sms = 0;
    bool attr_set[3] = {false, false, false};
};
inline DecodeDevice* decode_device(int dev) {
    static std::mutex mu;
    static DecodeDevice infos[kMaxDevices];
    if (dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    DecodeDevice& d = infos[dev];
    if (d.sms == 0) cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    return &d;
}

template <int DT>
inline enec_status launch_decode(const DecodeBatch& batch, int* d_status, cudaStream_t stream, bool ranked = false,
                                 int ticketed = 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
    DecodeDevice* found = decode_device(dev);
    if (!found) return ENEC_ERR_CUDA;
    DecodeDevice& info = *found;
    if (!info.attr_set[DT]) {
        if (cudaFuncSetAttribute(enec_decode_kernel<DT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kDecodeSmemBytes)) != cudaSuccess ||
            cudaFuncSetAttribute(enec_decode_kernel<DT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kDecodeSmemBytes)) != cudaSuccess ||
            cudaFuncSetAttribute(enec_decode_kernel<DT, false, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kDecodeSmemBytes)) != cudaSuccess ||
            cudaFuncSetAttribute(enec_decode_kernel<DT, false, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kDecodeSmemBytes)) != cudaSuccess)
            return ENEC_ERR_CUDA;
        info.attr_set[DT] = true;
    }
    uint32_t grid = uint32_t(info.sms) * 3;  // three resident CTAs per SM
    if (grid > batch.total_blocks) grid = batch.total_blocks;
    if (grid == 0) grid = 1;
    const cudaError_t err =
        ranked         ? launch_pdl(enec_decode_kernel<DT, true>, grid, kDecodeThreads, kDecodeSmemBytes, stream, batch, d_status)
        : ticketed == 1 ? launch_pdl(enec_decode_kernel<DT, false, 1>, grid, kDecodeThreads, kDecodeSmemBytes, stream, batch,
                                     d_status)
        : ticketed == 2 ? launch_pdl(enec_decode_kernel<DT, false, 2>, grid, kDecodeThreads, kDecodeSmemBytes, stream, batch,
                                     d_status)
                       : launch_pdl(enec_decode_kernel<DT, false>, grid, kDecodeThreads, kDecodeSmemBytes, stream, batch, d_status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return err == cudaSuccess ? ENEC_OK : ENEC_ERR_CUDA;
}


enec_status launch_decode_bf16(const DecodeBatch& batch, int* d_status, cudaStream_t stream, bool ranked, int ticketed);
enec_status launch_decode_fp16(const DecodeBatch& batch, int* d_status, cudaStream_t stream, bool ranked, int ticketed);
enec_status launch_decode_fp32(const DecodeBatch& batch, int* d_status, cudaStream_t stream, bool ranked, int ticketed);

}  // namespace enec
