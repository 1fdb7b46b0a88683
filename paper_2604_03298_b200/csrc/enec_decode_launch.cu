// Picks the decode kernels of a dtype; the instances themselves are compiled per dtype (enec_decode_<dtype>.cu).
#include "enec_decode_launch.cuh"

namespace enec {

enec_status launch_decode_any(int dt, const DecodeBatch& batch, int* d_status, cudaStream_t stream, bool ranked,
                              int ticketed) {
    return dt == ENEC_BF16   ? launch_decode_bf16(batch, d_status, stream, ranked, ticketed)
           : dt == ENEC_FP16 ? launch_decode_fp16(batch, d_status, stream, ranked, ticketed)
                             : launch_decode_fp32(batch, d_status, stream, ranked, ticketed);
}

}  // namespace enec
