// The decode kernel instances for bf16 streams.
#include "enec_decode_launch.cuh"

namespace enec {

enec_status launch_decode_bf16(const DecodeBatch& batch, int* d_status, cudaStream_t stream, bool ranked, int ticketed) {
    return launch_decode<ENEC_BF16>(batch, d_status, stream, ranked, ticketed);
}

}  // namespace enec
