// C-ABI entry points of libenec (see include/enec.h). Host-side validation and kernel launches only.
#include <atomic>
#include <map>
#include <mutex>
#include <utility>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "enec_decode.cuh"
#include "enec_encode.cuh"
#include "enec_blockwise.cuh"
#include "enec_launch.cuh"

namespace enec {

std::atomic<uint64_t> g_launches{0};

struct DeviceInfo {
    int sms = 0;
    bool hist_attr_set[3] = {false, false, false};
    bool encode_attr_set[3] = {false, false, false};
    bool batch_attr_set[3] = {false, false, false};
    bool blockwise_attr_set[3] = {false, false, false};
    bool split_attr_set[3] = {false, false, false};
};

// Per-device facts, for device ordinals below kMaxDevices (null beyond: the caller fails with ENEC_ERR_CUDA).
static DeviceInfo* device_info(int dev) {
    static std::mutex mu;
    static DeviceInfo infos[kMaxDevices];
    if (dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    DeviceInfo& d = infos[dev];
    if (d.sms == 0) cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev);
    return &d;
}

std::atomic<uint64_t> g_allocations{0};  // cudaMalloc calls the library has made (enec_allocation_count)

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// Device scratch, one area per (device, stream, purpose): for the compressor control words and one state
// word per block, for a batched call the tensor descriptors. Grown when a larger request arrives;
// outgrown areas are kept until exit because work that uses them may still be queued.
struct ScratchArea {
    uint8_t* ptr = nullptr;
    size_t bytes = 0;
    uint32_t epoch = 0;       // compressor areas: number of the last call
    bool needs_clear = true;  // compressor areas: fresh memory, a wrapped epoch or a launch that failed
};

enum ScratchKind { kScratchCompress = 0, kScratchBatch = 1, kScratchCompressBatch = 2, kScratchBlockwise = 3, kScratchDecodeTicket = 4 };

static std::mutex g_scratch_mu;
static ScratchArea& scratch_area(int dev, cudaStream_t stream, ScratchKind kind) {
    static std::map<std::pair<std::pair<int, int>, cudaStream_t>, ScratchArea> areas;
    return areas[std::make_pair(std::make_pair(dev, int(kind)), stream)];
}

static enec_status grow(ScratchArea& a, size_t need) {
    if (a.bytes >= need) return ENEC_OK;
    size_t bytes = a.bytes ? a.bytes : size_t(64) << 10;
    while (bytes < need) bytes *= 2;
    void* p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) return ENEC_ERR_CUDA;
    g_allocations.fetch_add(1, std::memory_order_relaxed);
    a.ptr = static_cast<uint8_t*>(p);
    a.bytes = bytes;
    a.needs_clear = true;
    return ENEC_OK;
}

static enec_status get_scratch(int dev, cudaStream_t stream, ScratchKind kind, size_t need, uint8_t** out) {
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    ScratchArea& a = scratch_area(dev, stream, kind);
    const enec_status st = grow(a, need);
    *out = a.ptr;
    return st;
}

// Scratch of one compress call and the call's number on it. The area is cleared (on `stream`) only when it
// is new, when the numbers have run out or after a call on it failed to launch; otherwise the kernels keep
// it usable from call to call (see EncodeControl).
static enec_status lease_compress_scratch(int dev, cudaStream_t stream, size_t need, uint8_t** out, uint32_t* epoch) {
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    ScratchArea& a = scratch_area(dev, stream, kScratchCompress);
    const enec_status st = grow(a, need);
    if (st != ENEC_OK) return st;
    if (a.needs_clear || a.epoch >= kEpochMax) {
        if (cudaMemsetAsync(a.ptr, 0, a.bytes, stream) != cudaSuccess) return ENEC_ERR_CUDA;
        a.needs_clear = false;
        a.epoch = 0;
    }
    *out = a.ptr;
    *epoch = ++a.epoch;
    return ENEC_OK;
}

static void mark_compress_scratch_unclean(int dev, cudaStream_t stream) {
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    scratch_area(dev, stream, kScratchCompress).needs_clear = true;
}

// The job's pointers into a scratch area for call number `epoch`.
static void place_job(EncodeJob& job, uint8_t* scratch, uint32_t epoch) {
    job.ctl = reinterpret_cast<EncodeControl*>(scratch + (epoch & 1) * kControlSlotBytes);
    job.ctl_next = reinterpret_cast<EncodeControl*>(scratch + ((epoch & 1) ^ 1) * kControlSlotBytes);
    job.state = reinterpret_cast<unsigned long long*>(scratch + kControlBytes);
    job.epoch = epoch;
}

// Tensors of split_min_blocks() .. split_max_blocks() - 1 blocks are compressed in the split form (pack kernel, then
// the kernel that places the records). Below that range the third launch costs more than the look-back it replaces;
// there is no upper bound by default. ENEC_SPLIT_MIN_BLOCKS and ENEC_SPLIT_MAX_BLOCKS in the environment override
// the bounds (read once; for measurements and tests).
static uint32_t env_blocks(const char* name, uint32_t fallback) {
    const char* e = getenv(name);
    return e && *e ? uint32_t(strtoul(e, nullptr, 10)) : fallback;
}
static uint32_t split_min_blocks() {
    static const uint32_t value = env_blocks("ENEC_SPLIT_MIN_BLOCKS", 2048u);
    return value;
}
static uint32_t split_max_blocks() {
    static const uint32_t value = env_blocks("ENEC_SPLIT_MAX_BLOCKS", 0xFFFFFFFFu);
    return value;
}

template <int DT>
static enec_status launch_split(const EncodeJob& job, uint32_t nblocks, int* d_status, DeviceInfo& info,
                                cudaStream_t stream) {
    if (!info.split_attr_set[DT]) {
        if (cudaFuncSetAttribute(enec_pack_tensor_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kPackSmemBytes)) != cudaSuccess ||
            cudaFuncSetAttribute(enec_place_records_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kPlaceSmemBytes)) != cudaSuccess)
            return ENEC_ERR_CUDA;
        info.split_attr_set[DT] = true;
    }
    uint32_t grid = uint32_t(info.sms) * 4;
    if (grid > nblocks) grid = nblocks;
    if (launch_pdl(enec_pack_tensor_kernel<DT>, grid, kPackThreads, kPackSmemBytes, stream, job, d_status) != cudaSuccess)
        return ENEC_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    grid = uint32_t(info.sms) * 2;
    if (grid > nblocks) grid = nblocks;
    if (grid > kPlaceMaxCtas) grid = kPlaceMaxCtas;
    if (launch_pdl(enec_place_records_kernel<DT>, grid, kPlaceThreads, kPlaceSmemBytes, stream, job, d_status) != cudaSuccess)
        return ENEC_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ENEC_OK;
}

template <int DT>
static enec_status launch_encode(const EncodeJob& job, uint32_t nblocks, bool search, int* d_status, DeviceInfo& info,
                                 cudaStream_t stream, bool may_split = false) {
    if (search) {
        const uint32_t smem = HistShape<DT>::kBytes;
        if (!info.hist_attr_set[DT]) {
            if (cudaFuncSetAttribute(enec_histogram_kernel<DT, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     int(smem)) != cudaSuccess ||
                cudaFuncSetAttribute(enec_histogram_kernel<DT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     int(smem)) != cudaSuccess)
                return ENEC_ERR_CUDA;
            info.hist_attr_set[DT] = true;
        }
        const uint64_t chunks = (job.count * uint64_t(elem_bytes(DT))) >> 4;  // 16-byte loads
        uint64_t grid = (chunks + kHistThreads - 1) / kHistThreads;
        if (grid > uint64_t(info.sms) * 3) grid = uint64_t(info.sms) * 3;
        if (grid == 0) grid = 1;
        const cudaError_t herr =
            job.ranked ? launch_pdl(enec_histogram_kernel<DT, true>, uint32_t(grid), kHistThreads, smem, stream, job.in,
                                    job.count, job.ctl)
                       : launch_pdl(enec_histogram_kernel<DT, false>, uint32_t(grid), kHistThreads, smem, stream, job.in,
                                    job.count, job.ctl);
        if (herr != cudaSuccess) return ENEC_ERR_CUDA;
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (may_split && !job.ranked && nblocks >= split_min_blocks() && nblocks < split_max_blocks()) return launch_split<DT>(job, nblocks, d_status, info, stream);
    }
    if (!info.encode_attr_set[DT]) {
        if (cudaFuncSetAttribute(enec_encode_kernel<DT, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(EncodeSmem<DT>::kBytes)) != cudaSuccess ||
            cudaFuncSetAttribute(enec_encode_kernel<DT, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(EncodeSmem<DT>::kBytes)) != cudaSuccess)
            return ENEC_ERR_CUDA;
        info.encode_attr_set[DT] = true;
    }
    uint32_t grid = uint32_t(info.sms) * 4;  // four resident CTAs per SM, each takes block after block
    if (grid > nblocks) grid = nblocks;
    const cudaError_t err =
        job.ranked ? launch_pdl(enec_encode_kernel<DT, false, true>, grid, kEncodeThreads, EncodeSmem<DT>::kBytes, stream,
                                job, EncodeBatch{}, d_status)
                   : launch_pdl(enec_encode_kernel<DT, false, false>, grid, kEncodeThreads, EncodeSmem<DT>::kBytes, stream,
                                job, EncodeBatch{}, d_status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return err == cudaSuccess ? ENEC_OK : ENEC_ERR_CUDA;
}

// The two launches of a batched compress call: histograms and parameter search of every tensor, then the
// encode of all their blocks.
template <int DT>
static enec_status launch_encode_batched(const EncodeJob* d_jobs, const HistUnit* d_units, uint32_t n_units,
                                         const EncodeBatch& batch, int* d_status, DeviceInfo& info, cudaStream_t stream) {
    const uint32_t hist_smem = HistShape<DT>::kBytes;
    if (!info.batch_attr_set[DT]) {
        if (cudaFuncSetAttribute(enec_histogram_batched_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(hist_smem)) != cudaSuccess ||
            cudaFuncSetAttribute(enec_encode_kernel<DT, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(EncodeSmem<DT>::kBytes)) != cudaSuccess)
            return ENEC_ERR_CUDA;
        info.batch_attr_set[DT] = true;
    }
    uint32_t grid = uint32_t(info.sms) * 3;
    if (grid > n_units) grid = n_units;
    // the second word of the call's ticket area hands out the histogram units (the first one the blocks of the encode)
    if (launch_pdl(enec_histogram_batched_kernel<DT>, grid, kHistThreads, hist_smem, stream, d_jobs, d_units, n_units,
                   batch.ticket + 4) != cudaSuccess)
        return ENEC_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    grid = uint32_t(info.sms) * 4;
    if (grid > batch.total_blocks) grid = batch.total_blocks;
    const cudaError_t err = launch_pdl(enec_encode_kernel<DT, true>, grid, kEncodeThreads, EncodeSmem<DT>::kBytes, stream,
                                       EncodeJob{}, batch, d_status);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return err == cudaSuccess ? ENEC_OK : ENEC_ERR_CUDA;
}

static enec_status compress_common(const void* d_in, enec_dtype dt, size_t count, bool with_params, int b, int n,
                                   int m, void* d_out, size_t out_capacity, size_t* d_out_size, int* d_status,
                                   cudaStream_t stream, bool ranked = false) {
    if (!known_dtype(dt)) return ENEC_ERR_UNSUPPORTED_DTYPE;
    if ((!d_in && count) || !d_out || (uint64_t(count) >> 36) || !aligned16(d_in) || !aligned16(d_out) ||
        (reinterpret_cast<uintptr_t>(d_out_size) & 7))
        return ENEC_ERR_INVALID_ARG;
    const int E = exp_bits(dt);
    if (with_params && (n < 1 || n > E || m < 1 || m > n || b < 0 || b >= (1 << E))) return ENEC_ERR_INVALID_ARG;
    if (out_capacity < (ranked ? enec_max_compressed_size_ranked(dt, count) : enec_max_compressed_size(dt, count)))
        return ENEC_ERR_BUFFER_TOO_SMALL;
    unsigned long long* out_size = reinterpret_cast<unsigned long long*>(d_out_size);
    if (count == 0) {
        // no exponent occurs: the search of Sec. 5.5 has nothing to minimise and keeps (0, 1, 1)
        enec_encode_empty_kernel<<<1, 32, 0, stream>>>(static_cast<uint8_t*>(d_out), int(dt), with_params ? b : 0,
                                                      with_params ? n : 1, with_params ? m : 1, out_size, ranked ? 1 : 0);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return cudaGetLastError() == cudaSuccess ? ENEC_OK : ENEC_ERR_CUDA;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
    DeviceInfo* found = device_info(dev);
    if (!found) return ENEC_ERR_CUDA;
    DeviceInfo& info = *found;
    const Geometry g = make_geometry(count);
    // control words, a state word per block, and the progress words of the kernel that places the records
    const size_t need = kControlBytes + (size_t(g.nblocks) + kPlaceMaxCtas) * sizeof(unsigned long long);
    // the scratch area carries state from call to call, which a replayed recording would not see
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return ENEC_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) return ENEC_ERR_INVALID_ARG;
    uint8_t* scratch = nullptr;
    uint32_t epoch = 0;
    enec_status st = lease_compress_scratch(dev, stream, need, &scratch, &epoch);
    if (st != ENEC_OK) return st;
    EncodeJob job;
    job.in = static_cast<const uint16_t*>(d_in);
    job.out = static_cast<uint8_t*>(d_out);
    job.count = count;
    place_job(job, scratch, epoch);
    job.out_size = out_size;
    job.b = b; job.n = n; job.m = m;
    job.from_search = with_params ? 0 : 1;
    job.check = with_params ? 1 : 0;
    job.ranked = ranked ? 1 : 0;
    st = dt == ENEC_BF16   ? launch_encode<ENEC_BF16>(job, g.nblocks, !with_params, d_status, info, stream, true)
         : dt == ENEC_FP16 ? launch_encode<ENEC_FP16>(job, g.nblocks, !with_params, d_status, info, stream, true)
                           : launch_encode<ENEC_FP32>(job, g.nblocks, !with_params, d_status, info, stream, true);
    if (st != ENEC_OK) mark_compress_scratch_unclean(dev, stream);  // a kernel of the call may not have run
    return st;
}

// ---- compression without any allocation ------------------------------------------------------------
// Scratch of enec_compress_noalloc: the compressor's control words and one look-back state word per
// block, for tensors of up to kNoAllocMaxCount values, held in the library image on every GPU that loads
// it. In host code `g_noalloc_scratch` is only a handle for cudaGetSymbolAddress, never an address to
// hand to a kernel.
constexpr uint64_t kNoAllocMaxCount = uint64_t(1) << 30;
constexpr size_t kNoAllocScratchBytes = kControlBytes + size_t(kNoAllocMaxCount / kBlockElems) * sizeof(unsigned long long);
static __device__ __align__(256) uint8_t g_noalloc_scratch[kNoAllocScratchBytes];
static_assert(kNoAllocScratchBytes == ENEC_NOALLOC_SCRATCH_BYTES, "the header states the size of the built-in scratch");

// Device address of the scratch on the current device, looked up once per device.
static enec_status noalloc_scratch(int dev, uint8_t** out) {
    static std::mutex mu;
    static uint8_t* addr[kMaxDevices] = {};
    if (dev < 0 || dev >= kMaxDevices) return ENEC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return ENEC_ERR_CUDA;
        addr[dev] = static_cast<uint8_t*>(p);
    }
    *out = addr[dev];
    return ENEC_OK;
}

// ---- the block-wise variant ------------------------------------------------------------------------

// The counter of finished blocks: zeroed when the area is new or after a call on it failed to launch; the
// kernel that uses it leaves it at zero.
static enec_status lease_blockwise_counter(int dev, cudaStream_t stream, uint32_t** out) {
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    ScratchArea& a = scratch_area(dev, stream, kScratchBlockwise);
    const enec_status st = grow(a, 256);
    if (st != ENEC_OK) return st;
    if (a.needs_clear) {
        if (cudaMemsetAsync(a.ptr, 0, 256, stream) != cudaSuccess) return ENEC_ERR_CUDA;
        a.needs_clear = false;
    }
    *out = reinterpret_cast<uint32_t*>(a.ptr);
    return ENEC_OK;
}

template <int DT>
static enec_status launch_blockwise(const BlockwiseJob& job, uint32_t nblocks, int* d_status, DeviceInfo& info,
                                    cudaStream_t stream) {
    if (!info.blockwise_attr_set[DT]) {
        if (cudaFuncSetAttribute(enec_block_params_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(HistShape<DT>::kBytes)) != cudaSuccess ||
            cudaFuncSetAttribute(enec_pack_blocks_kernel<DT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 int(kPackSmemBytes)) != cudaSuccess)
            return ENEC_ERR_CUDA;
        info.blockwise_attr_set[DT] = true;
    }
    uint32_t grid = uint32_t(info.sms) * 3;
    if (grid > nblocks) grid = nblocks;
    cudaError_t err = launch_pdl(enec_block_params_kernel<DT>, grid, kBlockwiseThreads, HistShape<DT>::kBytes, stream, job,
                                 d_status);
    if (err != cudaSuccess) return ENEC_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    grid = uint32_t(info.sms) * 4;
    if (grid > nblocks) grid = nblocks;
    err = launch_pdl(enec_pack_blocks_kernel<DT>, grid, kBlockwiseThreads, kPackSmemBytes, stream, job, d_status);
    if (err != cudaSuccess) return ENEC_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ENEC_OK;
}

static size_t max_size_blockwise(enec_dtype dt, size_t count) {
    if (!known_dtype(dt) || (uint64_t(count) >> 36)) return 0;
    const int E = exp_bits(dt);
    const Geometry g = make_geometry(count);
    // a block's low plane and records together are largest when all its groups are wide with n = E; the two
    // variable sections each end in up to 15 bytes of padding
    uint64_t worst = 0;
    for (int m = 1; m <= E; ++m) {
        const uint64_t t = make_sections_blockwise(dt, count, g, g.padded_count * uint64_t(m) / 8,
                                                   uint64_t(g.total_groups) * 2 * uint64_t(E - m)).total;
        if (t > worst) worst = t;
    }
    return size_t(worst + 32);
}

static enec_status compress_blockwise(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                                      size_t* d_out_size, int* d_status, cudaStream_t stream) {
    if (!known_dtype(dt)) return ENEC_ERR_UNSUPPORTED_DTYPE;
    if ((!d_in && count) || !d_out || (uint64_t(count) >> 36) || !aligned16(d_in) || !aligned16(d_out) ||
        (reinterpret_cast<uintptr_t>(d_out_size) & 7))
        return ENEC_ERR_INVALID_ARG;
    if (out_capacity < max_size_blockwise(dt, count)) return ENEC_ERR_BUFFER_TOO_SMALL;
    unsigned long long* out_size = reinterpret_cast<unsigned long long*>(d_out_size);
    if (count == 0) {
        enec_encode_empty_kernel<<<1, 32, 0, stream>>>(static_cast<uint8_t*>(d_out), int(dt), 0, 0, 0, out_size, 2);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return cudaGetLastError() == cudaSuccess ? ENEC_OK : ENEC_ERR_CUDA;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
    DeviceInfo* found = device_info(dev);
    if (!found) return ENEC_ERR_CUDA;
    // the counter carries state from call to call, which a replayed recording would not see
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return ENEC_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) return ENEC_ERR_INVALID_ARG;
    BlockwiseJob job;
    job.in = static_cast<const uint16_t*>(d_in);
    job.out = static_cast<uint8_t*>(d_out);
    job.count = count;
    job.out_size = out_size;
    enec_status st = lease_blockwise_counter(dev, stream, &job.done);
    if (st != ENEC_OK) return st;
    const uint32_t nblocks = make_geometry(count).nblocks;
    st = dt == ENEC_BF16   ? launch_blockwise<ENEC_BF16>(job, nblocks, d_status, *found, stream)
         : dt == ENEC_FP16 ? launch_blockwise<ENEC_FP16>(job, nblocks, d_status, *found, stream)
                           : launch_blockwise<ENEC_FP32>(job, nblocks, d_status, *found, stream);
    if (st != ENEC_OK) {
        std::lock_guard<std::mutex> lock(g_scratch_mu);
        scratch_area(dev, stream, kScratchBlockwise).needs_clear = true;
    }
    return st;
}

}  // namespace enec

using namespace enec;

extern "C" {

size_t enec_max_compressed_size(enec_dtype dt, size_t count) {
    if (!known_dtype(dt) || (uint64_t(count) >> 36)) return 0;
    const int E = exp_bits(dt);
    const Geometry g = make_geometry(count);
    uint64_t worst = 0;
    for (int m = 1; m <= E; ++m) {
        const uint64_t t = make_sections(dt, count, g, E, m, g.total_groups).total;
        if (t > worst) worst = t;
    }
    return size_t(worst);
}

// The ticket word of a large tensor's decode launch and the number of the launch on it (see enec_decode_kernel,
// TICKET = 2). The word is cleared once, when its area is allocated; after that every launch finds the number of an
// earlier launch in it and starts it afresh.
static enec_status lease_decode_ticket(int dev, cudaStream_t stream, uint8_t** word, uint32_t* number) {
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    ScratchArea& a = scratch_area(dev, stream, kScratchDecodeTicket);
    const enec_status st = grow(a, 256);
    if (st != ENEC_OK) return st;
    if (a.needs_clear || a.epoch == 0xFFFFFFFFu) {
        if (cudaMemsetAsync(a.ptr, 0, 256, stream) != cudaSuccess) return ENEC_ERR_CUDA;
        a.needs_clear = false;
        a.epoch = 0;
    }
    *word = a.ptr;
    *number = ++a.epoch;
    return ENEC_OK;
}

// Tensors of at least this many blocks are decoded with their blocks handed out by a ticket (outside a stream
// capture: the ticket word carries the launch's number, which a replay would repeat). ENEC_DECODE_TICKET_MIN_BLOCKS
// in the environment overrides the bound (read once; for measurements and tests).
static uint32_t decode_ticket_min_blocks() {
    static const uint32_t value = env_blocks("ENEC_DECODE_TICKET_MIN_BLOCKS", 16384u);
    return value;
}

static enec_status decompress_one(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                                  int* d_status, cudaStream_t stream, bool ranked, bool blockwise = false) {
    if (!known_dtype(dt)) return ENEC_ERR_UNSUPPORTED_DTYPE;
    if (!d_in || (!d_out && count) || (uint64_t(count) >> 36) || !aligned16(d_in) || !aligned16(d_out))
        return ENEC_ERR_INVALID_ARG;
    if (in_size < kHeaderBytes + 16) return ENEC_ERR_BAD_STREAM;
    DecodeBatch batch;
    batch.jobs = nullptr;
    batch.prefix = nullptr;
    batch.n_jobs = 1;
    batch.blockwise = blockwise ? 1 : 0;
    batch.total_blocks = make_geometry(count).nblocks;
    batch.inline_jobs[0] = DecodeJob{static_cast<const uint8_t*>(d_in), static_cast<uint16_t*>(d_out), uint64_t(count),
                                     uint64_t(in_size)};
    batch.inline_prefix[0] = 0;
    batch.inline_prefix[1] = batch.total_blocks;
    int ticketed = 0;
    if (!ranked && !blockwise && batch.total_blocks >= decode_ticket_min_blocks()) {
        cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return ENEC_ERR_CUDA;
        if (capturing == cudaStreamCaptureStatusNone) {
            int dev = 0;
            if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
            uint8_t* word = nullptr;
            uint32_t number = 0;
            // without the word (no device memory to be had) the launch keeps fixed shares: slower, not wrong
            if (lease_decode_ticket(dev, stream, &word, &number) == ENEC_OK) {
                batch.inline_jobs[1] = DecodeJob{word, nullptr, uint64_t(number), 0};  // not a tensor: n_jobs stays 1
                ticketed = 2;
            }
        }
    }
    return launch_decode_any(dt, batch, d_status, stream, ranked, ticketed);
}

enec_status enec_decompress(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                            int* d_status, enec_stream_t stream) {
    return decompress_one(d_in, in_size, dt, count, d_out, d_status, stream, false);
}

enec_status enec_decompress_ranked(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                                   int* d_status, enec_stream_t stream) {
    return decompress_one(d_in, in_size, dt, count, d_out, d_status, stream, true);
}

enec_status enec_decompress_batched(const enec_batch_item* h_items, int n_items, enec_dtype dt, int* d_status,
                                    enec_stream_t stream) {
    if (!known_dtype(dt)) return ENEC_ERR_UNSUPPORTED_DTYPE;
    if (n_items < 0 || (n_items > 0 && !h_items)) return ENEC_ERR_INVALID_ARG;
    if (n_items == 0) return ENEC_OK;
    // descriptors and block prefix in one host buffer: [jobs | prefix]; long lists add [ticket | tensor of every chunk]
    const size_t jobs_bytes = size_t(n_items) * sizeof(DecodeJob);
    const size_t prefix_bytes = size_t(ticket_offset_behind_prefix(uint32_t(n_items)));
    std::vector<uint8_t> host(jobs_bytes + prefix_bytes);
    DecodeJob* jobs = reinterpret_cast<DecodeJob*>(host.data());
    uint32_t* prefix = reinterpret_cast<uint32_t*>(host.data() + jobs_bytes);
    uint64_t total = 0;
    for (int i = 0; i < n_items; ++i) {
        const enec_batch_item& it = h_items[i];
        if (!it.d_in || (!it.d_out && it.count) || (uint64_t(it.count) >> 36) || !aligned16(it.d_in) ||
            !aligned16(it.d_out))
            return ENEC_ERR_INVALID_ARG;
        if (it.size < kHeaderBytes + 16) return ENEC_ERR_BAD_STREAM;
        jobs[i] = DecodeJob{static_cast<const uint8_t*>(it.d_in), static_cast<uint16_t*>(it.d_out), uint64_t(it.count),
                            uint64_t(it.size)};
        prefix[i] = uint32_t(total);
        total += make_geometry(it.count).nblocks;
        if (total >> 31) return ENEC_ERR_INVALID_ARG;  // block indices are 32-bit
    }
    prefix[n_items] = uint32_t(total);
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return ENEC_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone && uint32_t(n_items) > kInlineJobs) {
        // A recording must hold neither a copy from this call's host memory nor the library's scratch: lists of
        // up to kInlineJobs tensors travel inside the launch parameters, so a longer list becomes several launches.
        for (int first = 0; first < n_items; first += int(kInlineJobs)) {
            const int n = n_items - first < int(kInlineJobs) ? n_items - first : int(kInlineJobs);
            DecodeBatch part;
            part.jobs = nullptr;
            part.prefix = nullptr;
            part.n_jobs = uint32_t(n);
            part.blockwise = 0;
            part.total_blocks = prefix[first + n] - prefix[first];
            for (int i = 0; i < n; ++i) part.inline_jobs[i] = jobs[first + i];
            for (int i = 0; i <= n; ++i) part.inline_prefix[i] = prefix[first + i] - prefix[first];
            const enec_status st = launch_decode_any(dt, part, d_status, stream, false);
            if (st != ENEC_OK) return st;
        }
        return ENEC_OK;
    }
    DecodeBatch batch;
    batch.n_jobs = uint32_t(n_items);
    batch.blockwise = 0;
    batch.total_blocks = uint32_t(total);
    bool ticketed = false;
    // A short list travels in the launch parameters: no copy, no scratch. Unless it has so many blocks that the
    // ticket of the long-list form (which needs a zeroed word, hence the copy) gains more than the copy costs.
    constexpr uint64_t kTicketWorthBlocks = 8192;
    if (uint32_t(n_items) <= kInlineJobs && (capturing != cudaStreamCaptureStatusNone || total < kTicketWorthBlocks)) {
        batch.jobs = nullptr;
        batch.prefix = nullptr;
        for (int i = 0; i < n_items; ++i) batch.inline_jobs[i] = jobs[i];
        for (int i = 0; i <= n_items; ++i) batch.inline_prefix[i] = prefix[i];
    } else {
        // the blocks of a long list are handed out in chunks: a zeroed ticket word and the tensor of every chunk's
        // first block travel with the descriptors
        const size_t ticket_at = host.size();
        const size_t n_chunks = size_t((total + kTicketChunk - 1) / kTicketChunk);
        host.resize(ticket_at + 16 + n_chunks * sizeof(uint32_t), 0);
        {
            const uint32_t* pre = reinterpret_cast<const uint32_t*>(host.data() + jobs_bytes);
            uint32_t* chunk_job = reinterpret_cast<uint32_t*>(host.data() + ticket_at + 16);
            uint32_t j = 0;
            for (size_t c = 0; c < n_chunks; ++c) {
                const uint64_t first = uint64_t(c) * kTicketChunk;
                while (pre[j + 1] <= first) ++j;  // tensors without blocks are skipped
                chunk_job[c] = j;
            }
        }
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
        uint8_t* scratch = nullptr;
        const enec_status st = get_scratch(dev, stream, kScratchBatch, host.size(), &scratch);
        if (st != ENEC_OK) return st;
        // pageable source: the call returns once the bytes are staged, so `host` may go out of scope
        if (cudaMemcpyAsync(scratch, host.data(), host.size(), cudaMemcpyHostToDevice, stream) != cudaSuccess)
            return ENEC_ERR_CUDA;
        batch.jobs = reinterpret_cast<const DecodeJob*>(scratch);
        batch.prefix = reinterpret_cast<const uint32_t*>(scratch + jobs_bytes);
        ticketed = n_chunks > 0;
    }
    return launch_decode_any(dt, batch, d_status, stream, false, ticketed);
}

enec_status enec_compress(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                          size_t* d_out_size, int* d_status, enec_stream_t stream) {
    return compress_common(d_in, dt, count, false, 0, 0, 0, d_out, out_capacity, d_out_size, d_status, stream);
}

enec_status enec_compress_with_params(const void* d_in, enec_dtype dt, size_t count, int b, int n, int m,
                                      void* d_out, size_t out_capacity, size_t* d_out_size, int* d_status,
                                      enec_stream_t stream) {
    return compress_common(d_in, dt, count, true, b, n, m, d_out, out_capacity, d_out_size, d_status, stream);
}


size_t enec_max_compressed_size_ranked(enec_dtype dt, size_t count) {
    const size_t base = enec_max_compressed_size(dt, count);
    return base ? base + kRankTableBytes : 0;
}

size_t enec_max_compressed_size_blockwise(enec_dtype dt, size_t count) { return max_size_blockwise(dt, count); }

enec_status enec_compress_blockwise(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                                    size_t* d_out_size, int* d_status, enec_stream_t stream) {
    return compress_blockwise(d_in, dt, count, d_out, out_capacity, d_out_size, d_status, stream);
}

enec_status enec_decompress_blockwise(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                                      int* d_status, enec_stream_t stream) {
    return decompress_one(d_in, in_size, dt, count, d_out, d_status, stream, false, true);
}

enec_status enec_compress_ranked(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                                 size_t* d_out_size, int* d_status, enec_stream_t stream) {
    return compress_common(d_in, dt, count, false, 0, 0, 0, d_out, out_capacity, d_out_size, d_status, stream, true);
}

enec_status enec_compress_batched(const enec_batch_item* h_items, int n_items, enec_dtype dt, size_t* d_out_sizes,
                                  int* d_status, enec_stream_t stream) {
    if (!known_dtype(dt)) return ENEC_ERR_UNSUPPORTED_DTYPE;
    if (n_items < 0 || (n_items > 0 && !h_items) || (reinterpret_cast<uintptr_t>(d_out_sizes) & 7))
        return ENEC_ERR_INVALID_ARG;
    if (n_items == 0) return ENEC_OK;
    for (int i = 0; i < n_items; ++i) {
        const enec_batch_item& it = h_items[i];
        if ((!it.d_in && it.count) || !it.d_out || (uint64_t(it.count) >> 36) || !aligned16(it.d_in) || !aligned16(it.d_out))
            return ENEC_ERR_INVALID_ARG;
        if (it.size < enec_max_compressed_size(dt, it.count)) return ENEC_ERR_BUFFER_TOO_SMALL;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
    DeviceInfo* found = device_info(dev);
    if (!found) return ENEC_ERR_CUDA;
    DeviceInfo& info = *found;
    // the call clears and fills scratch from host memory that does not outlive it: not something to record
    cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) return ENEC_ERR_CUDA;
    if (capturing != cudaStreamCaptureStatusNone) return ENEC_ERR_INVALID_ARG;
    unsigned long long* sizes = reinterpret_cast<unsigned long long*>(d_out_sizes);
    // device scratch of the call: [ticket | control words per tensor | state word per block | jobs | prefix | units];
    // everything in front of the tables is cleared, the tables are copied from the host
    constexpr size_t kCtlStride = (sizeof(EncodeControl) + 63) & ~size_t(63);
    std::vector<uint32_t> prefix(size_t(n_items) + 1);
    std::vector<HistUnit> units;
    uint64_t total_blocks = 0;
    for (int i = 0; i < n_items; ++i) {
        prefix[i] = uint32_t(total_blocks);
        const uint64_t count = h_items[i].count;
        if (count == 0) continue;  // written by a launch of its own below
        total_blocks += make_geometry(count).nblocks;
        const uint64_t chunks = (count * uint64_t(elem_bytes(dt))) >> 4;
        const uint32_t n = chunks ? uint32_t((chunks + kHistUnitChunks - 1) / kHistUnitChunks) : 1u;
        for (uint32_t u = 0; u < n; ++u) units.push_back(HistUnit{uint32_t(i), u, n, 0u});
    }
    if (total_blocks >> 32) return ENEC_ERR_INVALID_ARG;
    prefix[n_items] = uint32_t(total_blocks);
    const size_t off_ctl = 256;
    const size_t off_state = (off_ctl + size_t(n_items) * kCtlStride + 255) & ~size_t(255);
    const size_t off_jobs = (off_state + size_t(total_blocks) * sizeof(unsigned long long) + 255) & ~size_t(255);
    const size_t off_prefix = off_jobs + size_t(n_items) * sizeof(EncodeJob);
    const size_t off_units = (off_prefix + prefix.size() * sizeof(uint32_t) + 15) & ~size_t(15);
    const size_t need = off_units + units.size() * sizeof(HistUnit);
    uint8_t* scratch = nullptr;
    const enec_status st = get_scratch(dev, stream, kScratchCompressBatch, need, &scratch);
    if (st != ENEC_OK) return st;
    std::vector<uint8_t> host(need - off_jobs);
    EncodeJob* jobs = reinterpret_cast<EncodeJob*>(host.data());
    for (int i = 0; i < n_items; ++i) {
        EncodeJob& job = jobs[i];
        job.in = static_cast<const uint16_t*>(h_items[i].d_in);
        job.out = static_cast<uint8_t*>(h_items[i].d_out);
        job.count = h_items[i].count;
        job.ctl = reinterpret_cast<EncodeControl*>(scratch + off_ctl + size_t(i) * kCtlStride);
        job.ctl_next = nullptr;
        job.state = reinterpret_cast<unsigned long long*>(scratch + off_state) + prefix[i];
        job.epoch = 1;  // the area was just cleared
        job.out_size = sizes ? sizes + i : nullptr;
        job.b = 0; job.n = 0; job.m = 0;
        job.from_search = 1;
        job.check = 0;
        job.ranked = 0;
    }
    memcpy(host.data() + (off_prefix - off_jobs), prefix.data(), prefix.size() * sizeof(uint32_t));
    if (!units.empty()) memcpy(host.data() + (off_units - off_jobs), units.data(), units.size() * sizeof(HistUnit));
    for (int i = 0; i < n_items; ++i) {
        if (h_items[i].count != 0) continue;
        enec_encode_empty_kernel<<<1, 32, 0, stream>>>(static_cast<uint8_t*>(h_items[i].d_out), int(dt), 0, 1, 1,
                                                      sizes ? sizes + i : nullptr);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (cudaGetLastError() != cudaSuccess) return ENEC_ERR_CUDA;
    }
    if (total_blocks == 0) return ENEC_OK;
    if (cudaMemsetAsync(scratch, 0, off_jobs, stream) != cudaSuccess) return ENEC_ERR_CUDA;
    // pageable source: the call returns once the bytes are staged, so `host` may go out of scope
    if (cudaMemcpyAsync(scratch + off_jobs, host.data(), host.size(), cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return ENEC_ERR_CUDA;
    EncodeBatch batch;
    batch.jobs = reinterpret_cast<const EncodeJob*>(scratch + off_jobs);
    batch.prefix = reinterpret_cast<const uint32_t*>(scratch + off_prefix);
    batch.n_jobs = uint32_t(n_items);
    batch.total_blocks = uint32_t(total_blocks);
    batch.ticket = reinterpret_cast<uint32_t*>(scratch);
    const HistUnit* d_units = reinterpret_cast<const HistUnit*>(scratch + off_units);
    const uint32_t n_units = uint32_t(units.size());
    return dt == ENEC_BF16   ? launch_encode_batched<ENEC_BF16>(batch.jobs, d_units, n_units, batch, d_status, info, stream)
           : dt == ENEC_FP16 ? launch_encode_batched<ENEC_FP16>(batch.jobs, d_units, n_units, batch, d_status, info, stream)
                             : launch_encode_batched<ENEC_FP32>(batch.jobs, d_units, n_units, batch, d_status, info, stream);
}

enec_status enec_compress_noalloc(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                                  size_t* d_out_size, int* d_status, enec_stream_t stream) {
    if (!known_dtype(dt)) return ENEC_ERR_UNSUPPORTED_DTYPE;
    if (uint64_t(count) > kNoAllocMaxCount) return ENEC_ERR_TOO_LARGE;
    if ((!d_in && count) || !d_out || !aligned16(d_in) || !aligned16(d_out) ||
        (reinterpret_cast<uintptr_t>(d_out_size) & 7))
        return ENEC_ERR_INVALID_ARG;
    if (out_capacity < enec_max_compressed_size(dt, count)) return ENEC_ERR_BUFFER_TOO_SMALL;
    unsigned long long* out_size = reinterpret_cast<unsigned long long*>(d_out_size);
    if (count == 0) {
        enec_encode_empty_kernel<<<1, 32, 0, stream>>>(static_cast<uint8_t*>(d_out), int(dt), 0, 1, 1, out_size);
        g_launches.fetch_add(1, std::memory_order_relaxed);
        return cudaGetLastError() == cudaSuccess ? ENEC_OK : ENEC_ERR_CUDA;
    }
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return ENEC_ERR_CUDA;
    uint8_t* scratch = nullptr;
    const enec_status st = noalloc_scratch(dev, &scratch);
    if (st != ENEC_OK) return st;
    DeviceInfo* found = device_info(dev);
    if (!found) return ENEC_ERR_CUDA;
    DeviceInfo& info = *found;
    const Geometry g = make_geometry(count);
    // the area keeps the previous call's words: histogram, ticket, flags and state words start at zero
    const size_t used = kControlBytes + size_t(g.nblocks) * sizeof(unsigned long long);
    if (cudaMemsetAsync(scratch, 0, used, stream) != cudaSuccess) return ENEC_ERR_CUDA;
    EncodeJob job;
    job.in = static_cast<const uint16_t*>(d_in);
    job.out = static_cast<uint8_t*>(d_out);
    job.count = count;
    place_job(job, scratch, 1);  // everything was just cleared, so every call is call number 1
    job.out_size = out_size;
    job.b = 0; job.n = 0; job.m = 0;
    job.from_search = 1;
    job.check = 0;
    job.ranked = 0;
    return dt == ENEC_BF16   ? launch_encode<ENEC_BF16>(job, g.nblocks, true, d_status, info, stream)
           : dt == ENEC_FP16 ? launch_encode<ENEC_FP16>(job, g.nblocks, true, d_status, info, stream)
                             : launch_encode<ENEC_FP32>(job, g.nblocks, true, d_status, info, stream);
}

uint64_t enec_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

uint64_t enec_allocation_count(void) { return g_allocations.load(std::memory_order_relaxed); }

int enec_version(void) { return 100; }

}  // extern "C"
