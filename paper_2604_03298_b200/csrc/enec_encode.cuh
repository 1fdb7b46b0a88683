// Compression kernels (Sec. 5.1 compression flow).
//
//   enec_histogram_kernel  Sec. 5.5 phase 1 (exponent histogram of the whole tensor) with the search of
//                          phases 2 and 3 (Eq. 1, 3, 4) run by the last CTA to finish.
//   enec_encode_kernel     persistent CTAs, one 16384-element block at a time: split, transform (Eq. 2), group widths
//                          (Sec. 5.2), Algorithm 2 on packed bytes for the low plane and for the records
//                          of wide groups, and the block-offset prefix sum as a decoupled look-back over
//                          per-block state words, so the input is read once.
//   enec_encode_empty_kernel  the 80-byte stream of an empty tensor.
//
// Blocks are handed out by an atomic ticket, so a block's predecessors are always resident or finished
// and every look-back wait ends; the wait is bounded all the same and ends in ENEC_ERR_TIMEOUT.
#pragma once

#include "enec_common.cuh"

namespace enec {

constexpr int kEncodeThreads = 256;
constexpr int kHistThreads = 256;
constexpr uint32_t kControlSlotBytes = 4096;             // one set of control words
constexpr uint32_t kControlBytes = 2 * kControlSlotBytes;  // control area in front of the per-block state words

// Device scratch of a compressor: two sets of control words, then one 64-bit state word per block. Nothing
// is cleared between calls. Calls on the area are numbered (the epoch, 1 .. 2^29 - 1): call e uses control
// set e mod 2, which it finds zeroed, and its encode kernel zeroes the other set for call e + 1 (that set's
// last user, call e - 1, has finished before any kernel of call e reads or writes global memory). A state
// word carries the epoch of the call that wrote it and counts as empty in every other call.
struct alignas(16) EncodeControl {
    unsigned long long hist[256];  // exponent histogram (2^E bins used)
    uint32_t ticket;               // next block to hand out
    uint32_t hist_done;            // CTAs of the histogram kernel that have finished
    uint32_t reserved;             // ticket of the kernel that places the records (split form of the compressor)
    int b, n, m;                   // result of the parameter search
    uint8_t lut[256];              // frequency-rank variant: exponent -> rank
    uint8_t unmap[256];            // frequency-rank variant: rank -> exponent (goes into the stream)
};
static_assert(sizeof(EncodeControl) <= kControlSlotBytes, "a control set fits its slot");

// state word: bits 63..62 = kind, bit 61 = this block or one summed into the value saw parameters that lose
// exponents, bits 60..32 = epoch of the writing call, bits 31..0 = value. Failure travels inside the words, so
// no fence is needed around them.
constexpr unsigned long long kStateAggregate = 1ull << 62;  // value = wide groups in the block
constexpr unsigned long long kStatePrefix = 2ull << 62;     // value = wide groups up to and including the block
constexpr unsigned long long kStatePoison = 3ull << 62;     // a predecessor failed
constexpr unsigned long long kStateTaint = 1ull << 61;
constexpr uint32_t kEpochMax = (1u << 29) - 1;
__host__ __device__ constexpr unsigned long long epoch_bits(uint32_t epoch) { return (unsigned long long)epoch << 32; }
// The word as this call sees it: words of other calls are empty.
__device__ __forceinline__ unsigned long long state_of_epoch(unsigned long long word, uint32_t epoch) {
    return (uint32_t(word >> 32) & kEpochMax) == epoch ? word : 0ull;
}

struct EncodeJob {
    const uint16_t* in;
    uint8_t* out;
    uint64_t count;
    EncodeControl* ctl;            // this call's control set (zero when the call starts)
    EncodeControl* ctl_next;       // the other set: zeroed by this call's encode kernel
    unsigned long long* state;
    uint32_t epoch;                // number of this call on the scratch area
    unsigned long long* out_size;  // device, may be null
    int b, n, m;                   // used when from_search == 0
    int from_search;               // take (b, n, m) from ctl
    int check;                     // verify that (b, n) keeps every exponent
    int ranked;                    // frequency-rank variant: stored value = ctl->lut[exponent]
};

__device__ __forceinline__ unsigned long long ld_relaxed_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

// ---------------------------------------------------------------------------------------------------
// Sec. 5.5 phase 1: histogram of the exponent field.
//
// A CTA keeps 32 copies of the histogram in shared memory, one per lane number: bin x is a row of 32 counters
// (128 bytes) and lane l of every warp adds to counter l of the row, so the 32 adds of a warp instruction go
// to 32 different banks whatever the values are (weights concentrate in three or four exponents, the worst
// case for anything shared between lanes), and an instruction is one pass through shared memory. Warps share
// the rows: the adds are atomic. Counting is one `red.shared.add` per value: no read-modify-write chain in
// the thread, no overflow, nothing to fold until the end.
// ---------------------------------------------------------------------------------------------------
template <int DT>
struct HistShape {
    static constexpr int E = DT == ENEC_FP16 ? 5 : 8;
    static constexpr int kBins = 1 << E;
    static constexpr int kPerLoad = DT == ENEC_FP32 ? 4 : 8;  // values in a 16-byte load
    static constexpr int kCopies = 32;                   // copies of the histogram per CTA: one per lane number
    static constexpr int kRowBytes = kCopies * 4;
    static constexpr int kBytes = kBins * kRowBytes;
};

// One value counted: a fire-and-forget shared-memory add on the lane's counter of the value's row, addressed
// straight from the word's bits.
__device__ __forceinline__ void red_add_one(uint32_t addr) {
    asm volatile("red.shared.add.u32 [%0], %1;" ::"r"(addr), "r"(1u) : "memory");
}

template <int DT>
__device__ __forceinline__ void count_word_pair(uint32_t base, uint32_t w) {
    // two 16-bit values per 32-bit word (one fp32 value); bin x sits at byte x * 128 of the CTA's area
    if (DT == ENEC_FP32) {
        red_add_one(base + ((w >> 16) & 0x7F80u));   // x = bits 30..23
    } else if (DT == ENEC_BF16) {
        red_add_one(base + (w & 0x7F80u));           // x = bits 14..7: already in place
        red_add_one(base + ((w >> 16) & 0x7F80u));
    } else {
        red_add_one(base + ((w >> 3) & 0xF80u));     // x = bits 14..10
        red_add_one(base + ((w >> 19) & 0xF80u));
    }
}

__host__ __device__ inline int bit_width_u32(uint32_t v) {
    int w = 0;
    while (v) { ++w; v >>= 1; }
    return w;
}

// Eq. 1 with the logarithms of 0 and 1 read as 0 and the result kept inside 1..E.
__host__ __device__ inline int width_eq1(int b, int l, int h, int E) {
    const int pos = bit_width_u32(uint32_t(b - l));
    const int d = h - b;
    const int neg = d <= 1 ? 0 : bit_width_u32(uint32_t(d - 1));
    int n = (pos > neg ? pos : neg) + 1;
    if (n > E) n = E;
    return n;
}

// Eq. 4 at L = 16 for one m in 1..n, given the number of elements per bit width of the stored value. Plain IEEE
// double, one rounding per operation, no fused multiply-add.
__device__ __forceinline__ double expected_bits(const unsigned long long* width_count, int n, int m) {
    unsigned long long total = 0;
    for (int w = 0; w <= 8; ++w) total += width_count[w];
    unsigned long long cnt = 0;
    for (int w = 0; w <= m; ++w) cnt += width_count[w];
    const double p = __ddiv_rn(__ull2double_rn(cnt), __ull2double_rn(total));
    const double p2 = __dmul_rn(p, p);
    const double p4 = __dmul_rn(p2, p2);
    const double p8 = __dmul_rn(p4, p4);
    const double p16 = __dmul_rn(p8, p8);
    const double saving = __dmul_rn(double(m - n), p16);
    return __dadd_rn(__dadd_rn(double(n), 0.0625), saving);  // 1/L + n + (m - n) p^L
}

// Sec. 5.5 phases 2 and 3 on a finished histogram; threads 0..255 of one CTA, thread t bringing the count of
// exponent t (`mine`; zero beyond the field; at least one count is non-zero). All of them return with the same
// (b, n, m). Every thread of the CTA must call it (it synchronises the CTA).
template <int DT>
__device__ void parameter_search_counts(unsigned long long mine, int& out_b, int& out_n, int& out_m) {
    constexpr int E = HistShape<DT>::E;
    constexpr int kBins = 1 << E;
    __shared__ unsigned long long s_hist[256];
    __shared__ unsigned long long s_key[kHistThreads / 32];
    __shared__ unsigned long long s_width_count[9];
    __shared__ double s_bits[8];
    __shared__ int s_lo, s_hi, s_b, s_n, s_m;
    const uint32_t tid = threadIdx.x;
    s_hist[tid] = tid < uint32_t(kBins) ? mine : 0ull;
    if (tid < 9) s_width_count[tid] = 0;
    if (tid == 0) { s_lo = kBins; s_hi = -1; }
    __syncthreads();
    if (s_hist[tid]) { atomicMin(&s_lo, int(tid)); atomicMax(&s_hi, int(tid)); }
    __syncthreads();
    const int l = s_lo, h = s_hi;
    // phase 2: every candidate b in [l, h]; cost = sum c[x] * y (Eq. 3 times N); smallest (cost, n, b)
    unsigned long long key = ~0ull;
    if (int(tid) >= l && int(tid) <= h) {
        const int b = int(tid);
        const int n = width_eq1(b, l, h, E);
        const uint32_t nmask = (1u << n) - 1;
        unsigned long long cost = 0;
        for (int x = l; x <= h; ++x) cost += s_hist[x] * (unsigned long long)(uint32_t(b - x) & nmask);
        key = (cost << 12) | (unsigned long long)(n << 8) | (unsigned long long)b;  // cost < 2^44
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xFFFFFFFFu, key, d);
        key = o < key ? o : key;
    }
    if ((tid & 31) == 0) s_key[tid >> 5] = key;
    __syncthreads();
    if (tid == 0) {
        unsigned long long best = s_key[0];
        for (int i = 1; i < kHistThreads / 32; ++i) best = s_key[i] < best ? s_key[i] : best;
        s_b = int(best & 0xFF);
        s_n = int((best >> 8) & 0xF);
    }
    __syncthreads();
    const int b = s_b, n = s_n;
    // phase 3: elements per bit width of y, then Eq. 4 at L = 16 for every m
    if (int(tid) >= l && int(tid) <= h && s_hist[tid]) {
        const uint32_t y = uint32_t(b - int(tid)) & ((1u << n) - 1);
        atomicAdd(&s_width_count[bit_width_u32(y)], s_hist[tid]);
    }
    __syncthreads();
    // Eq. 4: thread m - 1 evaluates m (the double-precision chain is long, so the candidates run side by side);
    // thread 0 takes the smallest value, the smaller m on ties
    if (tid < uint32_t(n)) s_bits[tid] = expected_bits(s_width_count, n, int(tid) + 1);
    __syncthreads();
    if (tid == 0) {
        int best_m = 1;
        for (int m = 2; m <= n; ++m)
            if (s_bits[m - 1] < s_bits[best_m - 1]) best_m = m;
        s_m = best_m;
    }
    __syncthreads();
    out_b = b;
    out_n = n;
    out_m = s_m;
    __syncthreads();  // the shared words may be written again by the next call
}

// The search on a tensor's histogram in its control words; the result goes back there.
template <int DT>
__device__ void parameter_search(EncodeControl* ctl) {
    const uint32_t tid = threadIdx.x;
    int b, n, m;
    parameter_search_counts<DT>(tid < uint32_t(1 << HistShape<DT>::E) ? ld_relaxed_u64(&ctl->hist[tid]) : 0ull, b, n, m);
    if (tid == 0) {
        ctl->b = b;
        ctl->n = n;
        ctl->m = m;
    }
}

// The frequency-rank variant (Sec. 4.2, Algorithm 1): exponents sorted by falling count (ties: smaller exponent
// first) give the codes 0, 1, 2, ...; n = bits of the largest code, m by Eq. 4 over the codes' bit widths.
template <int DT>
__device__ void parameter_search_ranked(EncodeControl* ctl) {
    constexpr int kBins = 1 << HistShape<DT>::E;
    __shared__ unsigned long long s_hist[256];
    __shared__ unsigned long long s_width_count[9];
    __shared__ uint32_t s_occupied;
    const uint32_t tid = threadIdx.x;
    s_hist[tid] = tid < uint32_t(kBins) ? ld_relaxed_u64(&ctl->hist[tid]) : 0ull;
    if (tid < 9) s_width_count[tid] = 0;
    if (tid == 0) s_occupied = 0;
    ctl->unmap[tid] = 0;
    __syncthreads();
    const unsigned long long mine = s_hist[tid];
    uint32_t rank = 0;
    if (mine) {
        for (uint32_t u = 0; u < uint32_t(kBins); ++u) {
            const unsigned long long other = s_hist[u];
            rank += (other > mine || (other == mine && u < tid)) ? 1u : 0u;
        }
        atomicAdd(&s_occupied, 1u);
        atomicAdd(&s_width_count[bit_width_u32(rank)], mine);
    }
    ctl->lut[tid] = uint8_t(rank);
    __syncthreads();
    if (mine) ctl->unmap[rank] = uint8_t(tid);
    if (tid == 0) {
        const int n = s_occupied <= 1 ? 1 : bit_width_u32(s_occupied - 1);
        ctl->b = 0;
        ctl->n = n;
        int best_m = 1;
        double best_bits = expected_bits(s_width_count, n, 1);
        for (int m = 2; m <= n; ++m) {  // ties go to the smaller m
            const double bits = expected_bits(s_width_count, n, m);
            if (bits < best_bits) { best_m = m; best_bits = bits; }
        }
        ctl->m = best_m;
    }
}

// Sum of a row's 32 counters, by the thread that owns the bin (the rows of neighbouring threads are read
// in rotated order, so that they do not all go to the same banks); CLEAR leaves the row zeroed.
template <bool CLEAR>
__device__ __forceinline__ uint32_t fold_hist_row(uint32_t row, uint32_t tid) {
    uint32_t sum = 0;
#pragma unroll
    for (uint32_t q = 0; q < 8; ++q) {
        const uint32_t at = row + ((q + tid) & 7) * 16;
        const uint4 v = lds128(at);
        sum += v.x + v.y + v.z + v.w;
        if (CLEAR) sts128(at, make_uint4(0, 0, 0, 0));
    }
    return sum;
}

template <int DT, bool RANKED = false>
__global__ void __launch_bounds__(kHistThreads, 3)
enec_histogram_kernel(const uint16_t* __restrict__ in, uint64_t count, EncodeControl* ctl) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint32_t cta_hist[256];
    __shared__ int s_last;
    pdl_launch_dependents();
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t base = smem_u32(smem) + lane * 4;
    for (uint32_t i = tid; i < uint32_t(HistShape<DT>::kBytes / 16); i += kHistThreads)
        reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    cta_hist[tid] = 0;
    __syncthreads();
    pdl_wait();  // nothing above touches global memory

    constexpr int kPerLoad = HistShape<DT>::kPerLoad;
    const uint64_t nchunks = count / kPerLoad;  // 16-byte loads of eight 16-bit or four 32-bit values
    const uint4* in4 = reinterpret_cast<const uint4*>(in);
    // a warp takes 2 KB at a time (four 16-byte loads per lane) and asks for its next 2 KB before it counts
    // the ones it holds, so four to eight loads per lane are in flight all the time
    constexpr uint32_t kUnroll = 4;
    const uint64_t stride = uint64_t(gridDim.x) * (kHistThreads / 32) * (32 * kUnroll);
    uint64_t first = (uint64_t(blockIdx.x) * (kHistThreads / 32) + warp) * (32 * kUnroll);
    uint4 cur[kUnroll], nxt[kUnroll];
    // back to front, default caching: the encode pass reads the tensor again from the front, where the lines
    // touched last are the likeliest to be in L2 still
    auto load = [&](uint4 (&v)[kUnroll], uint64_t at) {
#pragma unroll
        for (uint32_t u = 0; u < kUnroll; ++u) {
            const uint64_t i = at + u * 32 + lane;
            v[u] = make_uint4(0, 0, 0, 0);
            if (i < nchunks) v[u] = in4[nchunks - 1 - i];
        }
    };
    auto count4 = [&](const uint4 (&v)[kUnroll], uint64_t at) {
#pragma unroll
        for (uint32_t u = 0; u < kUnroll; ++u) {
            if (at + u * 32 + lane < nchunks) {
                count_word_pair<DT>(base, v[u].x);
                count_word_pair<DT>(base, v[u].y);
                count_word_pair<DT>(base, v[u].z);
                count_word_pair<DT>(base, v[u].w);
            }
        }
    };
    if (first < nchunks) load(cur, first);
    while (first < nchunks) {
        load(nxt, first + stride);
        count4(cur, first);
        first += stride;
        if (first >= nchunks) break;
        load(cur, first + stride);
        count4(nxt, first);
        first += stride;
    }
    __syncthreads();
    if (tid < uint32_t(HistShape<DT>::kBins)) cta_hist[tid] = fold_hist_row<false>(smem_u32(smem) + tid * HistShape<DT>::kRowBytes, tid);
    __syncthreads();
    if (blockIdx.x == 0 && tid == 0) {  // the values behind the last whole 16-byte load
        constexpr int sh = DT == ENEC_BF16 ? 7 : 10;
        for (uint64_t e = nchunks * kPerLoad; e < count; ++e) {
            const uint32_t x = DT == ENEC_FP32 ? (reinterpret_cast<const uint32_t*>(in)[e] >> 23) & 0xFFu
                                               : (uint32_t(in[e]) >> sh) & (HistShape<DT>::kBins - 1);
            atomicAdd(&cta_hist[x], 1u);
        }
    }
    __syncthreads();
    if (cta_hist[tid]) atomicAdd(&ctl->hist[tid], (unsigned long long)cta_hist[tid]);
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = atomicAdd(&ctl->hist_done, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if constexpr (RANKED) parameter_search_ranked<DT>(ctl);
    else parameter_search<DT>(ctl);
}

// Histograms of a list of tensors in one launch. The tensors are cut into units of at most kHistUnitChunks
// 16-byte loads; a CTA takes unit after unit, adds the unit's counts to its tensor's histogram, and the CTA
// that finishes a tensor's last outstanding unit runs that tensor's parameter search.
constexpr uint32_t kHistUnitChunks = 16384;  // 256 KB
struct HistUnit {
    uint32_t job;            // tensor of the unit
    uint32_t index;          // unit number inside the tensor
    uint32_t units_of_job;
    uint32_t pad;
};

template <int DT>
__global__ void __launch_bounds__(kHistThreads, 3)
enec_histogram_batched_kernel(const EncodeJob* __restrict__ jobs, const HistUnit* __restrict__ units, uint32_t n_units,
                              uint32_t* ticket) {
    extern __shared__ __align__(128) uint8_t smem[];
    __shared__ uint32_t cta_hist[256];
    __shared__ int s_last;
    constexpr int kPerLoad = HistShape<DT>::kPerLoad;
    pdl_launch_dependents();
    const uint32_t tid = threadIdx.x, lane = tid & 31;
    const uint32_t base = smem_u32(smem) + lane * 4;
    for (uint32_t i = tid; i < uint32_t(HistShape<DT>::kBytes / 16); i += kHistThreads)
        reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    cta_hist[tid] = 0;
    __syncthreads();
    pdl_wait();  // nothing above touches global memory
    // CTA c starts on unit c; after that units are handed out by `ticket` (zero when the launch starts), asked for
    // a unit ahead: the CTAs of an SM do not progress equally
    __shared__ uint32_t s_next_unit;
    for (uint32_t u = blockIdx.x; u < n_units;) {
        uint32_t asked = 0;
        if (tid == 0) asked = atomicAdd(ticket, 1u);
        const HistUnit unit = units[u];
        const uint16_t* in = jobs[unit.job].in;
        const uint64_t count = jobs[unit.job].count;
        EncodeControl* ctl = jobs[unit.job].ctl;
        const uint64_t nchunks = count / kPerLoad;
        const uint64_t first = uint64_t(unit.index) * kHistUnitChunks;
        const uint64_t end = first + kHistUnitChunks < nchunks ? first + kHistUnitChunks : nchunks;
        const uint4* in4 = reinterpret_cast<const uint4*>(in);
        for (uint64_t at = first + tid; at < end; at += 4 * kHistThreads) {
            uint4 v[4];
#pragma unroll
            for (uint32_t q = 0; q < 4; ++q) {
                v[q] = make_uint4(0, 0, 0, 0);
                if (at + q * kHistThreads < end) v[q] = in4[at + q * kHistThreads];
            }
#pragma unroll
            for (uint32_t q = 0; q < 4; ++q) {
                if (at + q * kHistThreads < end) {
                    count_word_pair<DT>(base, v[q].x);
                    count_word_pair<DT>(base, v[q].y);
                    count_word_pair<DT>(base, v[q].z);
                    count_word_pair<DT>(base, v[q].w);
                }
            }
        }
        __syncthreads();
        // fold the row of bin `tid` and clear it for the next unit
        if (tid < uint32_t(HistShape<DT>::kBins)) cta_hist[tid] = fold_hist_row<true>(smem_u32(smem) + tid * HistShape<DT>::kRowBytes, tid);
        __syncthreads();
        if (tid == 0 && unit.index + 1 == unit.units_of_job) {  // the values behind the last whole 16-byte load
            constexpr int sh = DT == ENEC_BF16 ? 7 : 10;
            for (uint64_t e = nchunks * kPerLoad; e < count; ++e) {
                const uint32_t x = DT == ENEC_FP32 ? (reinterpret_cast<const uint32_t*>(in)[e] >> 23) & 0xFFu
                                                   : (uint32_t(in[e]) >> sh) & (HistShape<DT>::kBins - 1);
                cta_hist[x] += 1;
            }
        }
        __syncthreads();
        if (cta_hist[tid]) atomicAdd(&ctl->hist[tid], (unsigned long long)cta_hist[tid]);
        cta_hist[tid] = 0;
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            s_last = atomicAdd(&ctl->hist_done, 1u) == unit.units_of_job - 1;
            s_next_unit = gridDim.x + asked;
        }
        __syncthreads();
        u = s_next_unit;
        if (s_last) {
            __threadfence();
            parameter_search<DT>(ctl);
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------------
// Algorithm 2 on packed bytes (forward). A thread that owns the eight lanes j..j+7 of the deepest level
// owns, at every level, whole runs of eight consecutive lanes: the 64 elements {j + c N/8 + i : c, i < 8}.
// Their fields are merged into 16-bit lanes kept as a low and a high byte plane; the low bytes are the
// level's normalised bytes, the high bytes its residue, packed again by the next level.
// ---------------------------------------------------------------------------------------------------
// ORs the w-bit fields v (one per byte, no other bits set) into the 16-bit lanes (lo | hi << 8) at bit s.
__device__ __forceinline__ void insert_bits(uint32_t& lo, uint32_t& hi, uint32_t v, int s, int w) {
    if (s + w <= 8) {
        lo |= v << s;
    } else if (s >= 8) {
        hi |= v << (s - 8);
    } else {
        const uint32_t keep = 0xFFu >> s;  // bits of a field that stay in the low byte
        lo |= (v & rep4(keep)) << s;
        hi |= (v >> (8 - s)) & rep4(((1u << w) - 1) >> (8 - s));
    }
}

// in[e] (e < 2^LOG_UNITS) = W_IN-bit fields of the eight elements j + e * n8 + (0..7) of this level.
// Normalised bytes are written in their order before the final fold: byte i of the plane at S + i.
template <int W_IN, int LOG_UNITS>
__device__ __forceinline__ void pack_plane_level(uint32_t S, uint32_t nb_off, uint32_t j, uint32_t n8,
                                                 const uint2 (&in)[1 << LOG_UNITS]) {
    constexpr int F = folds_for(W_IN);
    static_assert(F <= LOG_UNITS, "lane runs must stay whole");
    constexpr int W = W_IN << F;
    constexpr int LOG_LANES = LOG_UNITS - F;
    constexpr int NL = 1 << LOG_LANES;
    constexpr int RES = W - 8;
    uint2 R[NL];
#pragma unroll
    for (int c = 0; c < NL; ++c) {
        uint2 V = make_uint2(0, 0);
        R[c] = make_uint2(0, 0);
#pragma unroll
        for (int q = 0; q < (1 << F); ++q) {
            const int e = c + q * NL;
            const int s = W_IN * bitrev(q, F);
            insert_bits(V.x, R[c].x, in[e].x, s, W_IN);
            insert_bits(V.y, R[c].y, in[e].y, s, W_IN);
        }
        sts64(S + nb_off + j + c * n8, V);
    }
    if constexpr (RES > 0) pack_plane_level<RES, LOG_LANES>(S, nb_off + NL * n8, j, n8, R);
}

template <int A>
__device__ __forceinline__ void pack_plane(uint32_t S, uint32_t j, uint32_t N, const uint2 (&v)[8]) {
    pack_plane_level<A, 3>(S, 0, j, N >> 3, v);
}

__device__ __forceinline__ void pack_plane_any(int a, uint32_t S, uint32_t j, uint32_t N, const uint2 (&v)[8]) {
    switch (a) {
        case 1: pack_plane<1>(S, j, N, v); break;
        case 2: pack_plane<2>(S, j, N, v); break;
        case 3: pack_plane<3>(S, j, N, v); break;
        case 4: pack_plane<4>(S, j, N, v); break;
        case 5: pack_plane<5>(S, j, N, v); break;
        case 6: pack_plane<6>(S, j, N, v); break;
        case 7: pack_plane<7>(S, j, N, v); break;
        default: pack_plane<8>(S, j, N, v); break;
    }
}

// Final fold of Algorithm 2: output byte 2i = normalised byte i, 2i + 1 = normalised byte i + T/2.
// Reads the plane (T bytes at shared address S) and writes it folded to `dst`, 16 bytes per step.
__device__ __forceinline__ void fold_plane_out(uint32_t S, uint32_t T, uint8_t* dst, uint32_t tid) {
    const uint32_t thalf = T >> 1;
    for (uint32_t u = tid; u < (thalf >> 3); u += kEncodeThreads) {
        const uint2 lo = lds64(S + 8 * u);
        const uint2 hi = lds64(S + thalf + 8 * u);
        uint4 w;
        w.x = prmt(lo.x, hi.x, 0x5140u);
        w.y = prmt(lo.x, hi.x, 0x7362u);
        w.z = prmt(lo.y, hi.y, 0x5140u);
        w.w = prmt(lo.y, hi.y, 0x7362u);
        *reinterpret_cast<uint4*>(dst + 16 * u) = w;
    }
}

// ---- wide-group records: Algorithm 2 with N = 16 and H bits per value -> H 16-bit words ---------------
// Same scheme with runs of two lanes. in[e] = fields of elements 2e, 2e + 1 in bytes 0 and 1.
template <int H, int W_IN, int LOG_UNITS, int NB_OFF>
__device__ __forceinline__ void pack_record_level(uint32_t (&q)[H], const uint32_t (&in)[1 << LOG_UNITS]) {
    constexpr int F = folds_for(W_IN);
    static_assert(F <= LOG_UNITS, "lane runs must stay whole");
    constexpr int W = W_IN << F;
    constexpr int LOG_LANES = LOG_UNITS - F;
    constexpr int NL = 1 << LOG_LANES;
    constexpr int RES = W - 8;
    uint32_t R[NL];
#pragma unroll
    for (int c = 0; c < NL; ++c) {
        uint32_t V = 0;
        R[c] = 0;
#pragma unroll
        for (int k = 0; k < (1 << F); ++k) {
            const int e = c + k * NL;
            insert_bits(V, R[c], in[e], W_IN * bitrev(k, F), W_IN);
        }
        // normalised bytes i0, i0 + 1 of the record; byte i sits at 2i (i < H) or 2(i - H) + 1
        const int i0 = NB_OFF + 2 * c;
        const int pa = i0 < H ? 2 * i0 : 2 * (i0 - H) + 1;
        const int pb = (i0 + 1) < H ? 2 * (i0 + 1) : 2 * (i0 + 1 - H) + 1;
        q[pa >> 1] |= (V & 0xFFu) << (8 * (pa & 1));
        q[pb >> 1] |= ((V >> 8) & 0xFFu) << (8 * (pb & 1));
    }
    if constexpr (RES > 0) pack_record_level<H, RES, LOG_LANES, NB_OFF + 2 * NL>(q, R);
}

// v = the sixteen H-bit values of a group, one per byte, element order; the record goes to shared
// address `dst` (2-byte aligned) as H 16-bit words.
template <int H>
__device__ __forceinline__ void pack_record(uint4 v, uint32_t dst) {
    uint32_t in[8] = {v.x & 0xFFFFu, v.x >> 16, v.y & 0xFFFFu, v.y >> 16,
                      v.z & 0xFFFFu, v.z >> 16, v.w & 0xFFFFu, v.w >> 16};
    uint32_t q[H];
#pragma unroll
    for (int i = 0; i < H; ++i) q[i] = 0;
    pack_record_level<H, H, 3, 0>(q, in);
#pragma unroll
    for (int i = 0; i < H; ++i) sts16(dst + 2 * i, q[i]);
}

__device__ __forceinline__ void pack_record_any(int hbits, uint4 v, uint32_t dst) {
    switch (hbits) {
        case 1: pack_record<1>(v, dst); break;
        case 2: pack_record<2>(v, dst); break;
        case 3: pack_record<3>(v, dst); break;
        case 4: pack_record<4>(v, dst); break;
        case 5: pack_record<5>(v, dst); break;
        case 6: pack_record<6>(v, dst); break;
        default: pack_record<7>(v, dst); break;
    }
}

// Where bit q of element e of a plane of N elements of `a` bits ends up: byte `pos` of the packed plane,
// bit `bit` (Algorithm 2 followed for one bit; used for blocks shorter than 128 elements).
__device__ inline void alg2_locate(uint32_t N, int a, uint32_t e, int q, uint32_t& pos, int& bit) {
    const uint32_t thalf = (N * uint32_t(a)) >> 4;
    int width = a, p = q;
    uint32_t length = N, idx = e, off = 0;
    while (true) {
        while (length > 1 && width < 8) {
            length >>= 1;
            if (idx >= length) { idx -= length; p += width; }
            width <<= 1;
        }
        if (p < 8) break;
        p -= 8;
        width -= 8;
        off += length;
    }
    const uint32_t i = off + idx;
    pos = i < thalf ? 2 * i : 2 * (i - thalf) + 1;
    bit = p;
}

// ---------------------------------------------------------------------------------------------------
// Split and transform on packed bytes.
// ---------------------------------------------------------------------------------------------------
struct Split4 {
    uint32_t x;   // exponent fields of four values, one per byte
    uint32_t sm;  // bf16: sign << 7 | mantissa ; fp16: mantissa bits 7..0
    uint32_t hs;  // fp16: sign << 2 | mantissa bits 9..8
};

template <int DT>
__device__ __forceinline__ Split4 split4(uint32_t w0, uint32_t w1) {
    const uint32_t lo = prmt(w0, w1, 0x6420u);  // low bytes of the four 16-bit words
    const uint32_t hi = prmt(w0, w1, 0x7531u);  // high bytes
    Split4 s;
    if (DT != ENEC_FP16) {
        s.x = ((hi << 1) & 0xFEFEFEFEu) | ((lo >> 7) & 0x01010101u);
        s.sm = (hi & 0x80808080u) | (lo & 0x7F7F7F7Fu);
        s.hs = 0;
    } else {
        s.x = (hi >> 2) & 0x1F1F1F1Fu;
        s.sm = lo;
        s.hs = ((hi >> 5) & 0x04040404u) | (hi & 0x03030303u);
    }
    return s;
}

struct TransformCtx {
    uint32_t b4_or_h;   // rep4(b) | 0x80808080
    uint32_t b4;        // rep4(b)
    uint32_t nmask4;    // rep4(2^n - 1)
    uint32_t s4;        // rep4(2^(n-1))
    uint32_t emask4;    // rep4(2^E - 1)
    int n, E;
    uint32_t lut;       // frequency-rank variant: shared address of the exponent -> rank table, else 0
};

// Four table look-ups: byte i of the result is the table entry of byte i of v.
__device__ __forceinline__ uint32_t lut4(uint32_t table, uint32_t v) {
    const uint32_t r0 = lds8(table + (v & 0xFFu)), r1 = lds8(table + ((v >> 8) & 0xFFu));
    const uint32_t r2 = lds8(table + ((v >> 16) & 0xFFu)), r3 = lds8(table + (v >> 24));
    return r0 | (r1 << 8) | (r2 << 16) | (r3 << 24);
}

// b - x modulo 256 in every byte
__device__ __forceinline__ uint32_t bytewise_b_minus(const TransformCtx& t, uint32_t x) {
    return (t.b4_or_h - (x & 0x7F7F7F7Fu)) ^ ((t.b4 ^ ~x) & 0x80808080u);
}

// Bytes whose exponent is not reproduced by (b, n): x != (b - sext_n(y)) mod 2^E. Non-zero = some byte fails.
__device__ __forceinline__ uint32_t lossy_bytes(const TransformCtx& t, uint32_t d, uint32_t y) {
    if (t.n == t.E) return 0;
    // sext_n(y) = (y ^ s) - s per byte; (y ^ s) < 128 because n < 8
    const uint32_t sext = (((y ^ t.s4) | 0x80808080u) - t.s4) ^ 0x80808080u;
    return (sext ^ d) & t.emask4;
}

// ---------------------------------------------------------------------------------------------------
struct EncodeShared {
    uint32_t mask[32];     // the block's group mask, bit g = group g is wide
    uint32_t group_or[8];  // short blocks: OR of y per group
    uint32_t next[2];      // tickets of the CTA's current and next block, by iteration parity
    uint32_t before;       // P_k
    uint32_t poisoned;
    uint32_t tainted;      // the block or a predecessor saw parameters that lose exponents
};

// fp32: the eight values at `p` (32 bytes, 16-byte aligned) as their high halves, which have bf16's layout; the
// low halves go to `lo_dst` (16 bytes) as they are.
__device__ __forceinline__ uint4 load_fp32_run(const uint8_t* __restrict__ p, uint8_t* __restrict__ lo_dst) {
    uint4 a0, a1;
    if ((reinterpret_cast<uintptr_t>(p) & 31) == 0) {
        // one 32-byte load: consecutive lanes read consecutive 32-byte pieces
        asm("ld.global.cs.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
            : "=r"(a0.x), "=r"(a0.y), "=r"(a0.z), "=r"(a0.w), "=r"(a1.x), "=r"(a1.y), "=r"(a1.z), "=r"(a1.w)
            : "l"(p));
    } else {
        a0 = __ldcs(reinterpret_cast<const uint4*>(p));
        a1 = __ldcs(reinterpret_cast<const uint4*>(p) + 1);
    }
    __stcs(reinterpret_cast<uint4*>(lo_dst), make_uint4(prmt(a0.x, a0.y, 0x5410u), prmt(a0.z, a0.w, 0x5410u),
                                                        prmt(a1.x, a1.y, 0x5410u), prmt(a1.z, a1.w, 0x5410u)));
    return make_uint4(prmt(a0.x, a0.y, 0x7632u), prmt(a0.z, a0.w, 0x7632u), prmt(a1.x, a1.y, 0x7632u),
                      prmt(a1.z, a1.w, 0x7632u));
}

// Phase 1 of a full block (16384 real elements), all 256 threads: loads, split, transform, sign/mantissa
// stores and group widths with immediate offsets and no bounds logic. Lanes l and l + 16 share a group, so
// the two halves of a ballot OR into the mask of the warp's sixteen groups of run c.
// SIMPLE (n < 8 and no loss check): only the low seven bits of b - x matter, so the exponent is taken
// without its top bit and a guard bit absorbs the borrow: y = ((b & 127 | 128) - (x & 127)) & (2^n - 1).
// Returns the wide flags of the thread's eight runs (bit c).
// With DT = ENEC_FP32 the values are 32-bit words: their high halves take bf16's path, their low halves are
// stored as they are to `lo_thread` (two bytes per value).
template <int DT, bool SIMPLE, bool RANKED = false>
__device__ __forceinline__ uint32_t encode_full_runs(const uint8_t* in_thread, uint8_t* sm_thread, uint8_t* lo_thread,
                                                     const TransformCtx& tc, int m, uint32_t warp, uint32_t lane,
                                                     uint32_t* mask_words, uint2 (&y)[8], uint2 (&hs)[8], int& bad) {
    constexpr uint32_t kRunStride = kBlockElems / 8;  // elements between a thread's runs
    uint4 raw[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        if constexpr (DT == ENEC_FP32) raw[c] = load_fp32_run(in_thread + c * kRunStride * 4, lo_thread + c * kRunStride * 2);
        else raw[c] = __ldcs(reinterpret_cast<const uint4*>(in_thread + c * kRunStride * 2));
    }
    const uint32_t c7 = (tc.b4 & 0x7F7F7F7Fu) | 0x80808080u;
    const uint32_t widemask4 = ~rep4((1u << m) - 1);
    uint32_t wide_bits = 0;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        uint32_t sm0, sm1;
        if constexpr (SIMPLE) {
            const uint32_t lo0 = prmt(raw[c].x, raw[c].y, 0x6420u), hi0 = prmt(raw[c].x, raw[c].y, 0x7531u);
            const uint32_t lo1 = prmt(raw[c].z, raw[c].w, 0x6420u), hi1 = prmt(raw[c].z, raw[c].w, 0x7531u);
            uint32_t x0, x1;  // exponent fields without bit 7
            if (DT != ENEC_FP16) {
                x0 = ((hi0 << 1) & 0x7E7E7E7Eu) | ((lo0 >> 7) & 0x01010101u);
                x1 = ((hi1 << 1) & 0x7E7E7E7Eu) | ((lo1 >> 7) & 0x01010101u);
                sm0 = (hi0 & 0x80808080u) | (lo0 & 0x7F7F7F7Fu);
                sm1 = (hi1 & 0x80808080u) | (lo1 & 0x7F7F7F7Fu);
                hs[c] = make_uint2(0, 0);
            } else {
                x0 = (hi0 >> 2) & 0x1F1F1F1Fu;
                x1 = (hi1 >> 2) & 0x1F1F1F1Fu;
                sm0 = lo0;
                sm1 = lo1;
                hs[c] = make_uint2(((hi0 >> 5) & 0x04040404u) | (hi0 & 0x03030303u),
                                   ((hi1 >> 5) & 0x04040404u) | (hi1 & 0x03030303u));
            }
            y[c] = make_uint2((c7 - x0) & tc.nmask4, (c7 - x1) & tc.nmask4);
        } else {
            const Split4 s0 = split4<DT>(raw[c].x, raw[c].y);
            const Split4 s1 = split4<DT>(raw[c].z, raw[c].w);
            if constexpr (RANKED) {  // frequency-rank variant: the stored value is the exponent's rank
                y[c] = make_uint2(lut4(tc.lut, s0.x), lut4(tc.lut, s1.x));
            } else {
                const uint32_t d0 = bytewise_b_minus(tc, s0.x), d1 = bytewise_b_minus(tc, s1.x);
                y[c] = make_uint2(d0 & tc.nmask4, d1 & tc.nmask4);
                bad |= (lossy_bytes(tc, d0, y[c].x) | lossy_bytes(tc, d1, y[c].y)) != 0;
            }
            hs[c] = make_uint2(s0.hs, s1.hs);
            sm0 = s0.sm;
            sm1 = s1.sm;
        }
        __stcs(reinterpret_cast<uint2*>(sm_thread + c * kRunStride), make_uint2(sm0, sm1));
        const bool wide_half = ((y[c].x | y[c].y) & widemask4) != 0;  // some value of this half needs more than m bits
        const uint32_t bal = __ballot_sync(0xFFFFFFFFu, wide_half);
        const uint32_t groups16 = (bal | (bal >> 16)) & 0xFFFFu;
        wide_bits |= ((groups16 >> (lane & 15)) & 1u) << c;
        if (lane == 0) reinterpret_cast<uint16_t*>(mask_words)[c * 8 + warp] = uint16_t(groups16);
    }
    return wide_bits;
}

// Blocks shorter than 128 elements (16, 32 or 64): one element per thread, bits placed one by one.
template <int DT>
__device__ __noinline__ int encode_short_block(const uint16_t* in, uint32_t N, uint32_t real, const TransformCtx& tc,
                                               int b, int n, int m, int check, uint8_t* out_sm, uint8_t* out_low,
                                               uint8_t* out_smhi, uint8_t* out_mask, uint8_t* out_smlo, EncodeShared* sh,
                                               uint32_t* s_low, uint32_t* s_hi3, uint32_t* s_rec) {
    const uint32_t tid = threadIdx.x;
    const int hbits = n - m;
    if (tid < 32) sh->mask[tid] = 0;
    if (tid < 8) sh->group_or[tid] = 0;
    if (tid < 16) { s_low[tid] = 0; s_rec[tid] = 0; }
    if (tid < 8) s_hi3[tid] = 0;
    __syncthreads();
    int bad = 0;
    uint32_t y = 0;
    if (tid < N) {
        uint32_t w = 0;
        if (DT == ENEC_FP32) {
            // the high half goes on as a bf16 word; the low half is stored as it is (zeros pad the plane to 16 bytes)
            const uint32_t full = tid < real ? reinterpret_cast<const uint32_t*>(in)[tid] : 0;
            w = full >> 16;
            if (2 * tid < uint32_t(align16(2 * real))) reinterpret_cast<uint16_t*>(out_smlo)[tid] = uint16_t(full);
        } else if (tid < real) {
            w = in[tid];
        }
        uint32_t x, sm, hs = 0;
        if (DT != ENEC_FP16) { x = (w >> 7) & 0xFF; sm = ((w >> 8) & 0x80) | (w & 0x7F); }
        else { x = (w >> 10) & 0x1F; sm = w & 0xFF; hs = ((w >> 13) & 4) | ((w >> 8) & 3); }
        if (tid < real) {
            y = tc.lut ? lds8(tc.lut + x) : uint32_t(b - int(x)) & ((1u << n) - 1);
            if (check && n < tc.E && !tc.lut) {
                const int v = (y >> (n - 1)) ? int(y) - (1 << n) : int(y);
                bad = (uint32_t(b - v) & ((1u << tc.E) - 1)) != x;
            }
            out_sm[tid] = uint8_t(sm);
        } else if (tid < uint32_t(align16(real))) {
            out_sm[tid] = 0;
        }
        atomicOr(&sh->group_or[tid >> 4], y);
        for (int q = 0; q < m; ++q)
            if ((y >> q) & 1) {
                uint32_t pos; int bit;
                alg2_locate(N, m, tid, q, pos, bit);
                atomicOr(&s_low[pos >> 2], 1u << (8 * (pos & 3) + bit));
            }
        if (DT == ENEC_FP16)
            for (int q = 0; q < 3; ++q)
                if ((hs >> q) & 1) {
                    uint32_t pos; int bit;
                    alg2_locate(N, 3, tid, q, pos, bit);
                    atomicOr(&s_hi3[pos >> 2], 1u << (8 * (pos & 3) + bit));
                }
    }
    __syncthreads();
    const bool wide = tid < N && (sh->group_or[tid >> 4] >> m) != 0;
    if (wide && (tid & 15) == 0) atomicOr(&sh->mask[0], 1u << (tid >> 4));
    __syncthreads();
    if (wide && hbits > 0) {
        const uint32_t rank = __popc(sh->mask[0] & ((1u << (tid >> 4)) - 1));
        const uint32_t hv = y >> m;
        for (int q = 0; q < hbits; ++q)
            if ((hv >> q) & 1) {
                uint32_t pos; int bit;
                alg2_locate(16, hbits, tid & 15, q, pos, bit);
                pos += rank * 2 * hbits;
                atomicOr(&s_rec[pos >> 2], 1u << (8 * (pos & 3) + bit));
            }
    }
    // planes out, padded to 16 bytes with zeros
    const uint32_t low_words = uint32_t(align16(N * uint32_t(m) / 8)) / 4;
    if (tid < low_words) reinterpret_cast<uint32_t*>(out_low)[tid] = s_low[tid];
    if (tid < 4) reinterpret_cast<uint32_t*>(out_mask)[tid] = tid == 0 ? sh->mask[0] : 0;
    if (DT == ENEC_FP16) {
        const uint32_t hi_words = uint32_t(align16(N * 3 / 8)) / 4;
        if (tid < hi_words) reinterpret_cast<uint32_t*>(out_smhi)[tid] = s_hi3[tid];
    }
    return bad;
}

// Dynamic shared memory of the encode kernel.
template <int DT>
struct EncodeSmem {
    static constexpr uint32_t kHi3Bytes = DT == ENEC_FP16 ? kBlockElems * 3 / 8 : 32;
    static constexpr uint32_t kRecBytes = kGroupsPerBlock * 16 + 16;  // one buffer: every group wide, plus a spare slot
    static constexpr uint32_t kBytes = kBlockElems + kHi3Bytes + 2 * kRecBytes;
};

// What every block of the tensor shares.
struct EncodeTensor {
    Geometry g;
    Sections sec;
    int b, n, m, hbits;
};

// Second half of a block's work, all threads: find P_k (wide groups before block k) by looking back over
// the predecessors' state words, publish the block's own prefix, copy its packed records (at shared
// address `rec`, `wide_count` of them) to their place in the stream and write its table entry; the last
// block also writes the header, the end of the table and the stream length. The look-back is done by
// warp 0, up to 256 words per round trip, down to the nearest block that already knows its prefix.
template <int DT, bool RANKED = false>
__device__ __forceinline__ void resolve_block(const EncodeJob& job, const EncodeTensor& t, uint32_t k, uint32_t wide_count,
                                              bool own_taint, const uint8_t* rec, EncodeShared& sh, int* status) {
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (warp == 0 && k > 0) {
        uint32_t before = 0;
        uint32_t tainted = own_taint ? 1u : 0u;
        int64_t pos = int64_t(k) - 1;
        int outcome = 0;  // 1 = done, 2 = poisoned, 3 = gave up
        uint32_t polls = 0;
        while (outcome == 0) {
            // eight coalesced loads of 32 consecutive words: word i * 32 + lane back from pos
            unsigned long long st[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int64_t idx = pos - (i * 32 + int64_t(lane));
                st[i] = idx >= 0 ? state_of_epoch(ld_relaxed_u64(&job.state[idx]), job.epoch) : kStatePrefix;
            }
            uint32_t mine = 0;      // this lane's share of the sum
            uint32_t advanced = 0;  // windows of 32 fully summed in this round
            bool blocked = false;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (outcome == 0 && !blocked) {
                    const uint32_t kind = uint32_t(st[i] >> 62);
                    const uint32_t prefix_lanes = __ballot_sync(0xFFFFFFFFu, kind == 2);
                    const uint32_t empty_lanes = __ballot_sync(0xFFFFFFFFu, kind == 0);
                    const uint32_t poison_lanes = __ballot_sync(0xFFFFFFFFu, kind == 3);
                    const uint32_t first = prefix_lanes ? uint32_t(__ffs(prefix_lanes)) - 1 : 32;
                    const uint32_t needed = first == 32 ? 0xFFFFFFFFu : (2u << first) - 1;  // lanes 0..first
                    if (poison_lanes & needed) {
                        outcome = 2;
                    } else if (empty_lanes & needed) {
                        blocked = true;  // a nearer block has not published yet
                    } else {
                        if ((needed >> lane) & 1) {
                            mine += uint32_t(st[i]);
                            tainted |= uint32_t(st[i] >> 61) & 1u;
                        }
                        if (first < 32) outcome = 1;
                        else ++advanced;
                    }
                }
            }
            if (outcome == 2) break;
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) mine += __shfl_xor_sync(0xFFFFFFFFu, mine, d);
            before += mine;
            pos -= 32 * int64_t(advanced);
            if (blocked) {
                if (++polls > (1u << 20)) { outcome = 3; break; }
                __nanosleep(polls > 2 ? 400 : 100);
            }
        }
        tainted = __any_sync(0xFFFFFFFFu, tainted != 0);
        if (lane == 0) {
            if (outcome == 1) {
                sh.before = before;
                sh.poisoned = 0;
                sh.tainted = tainted;
                st_relaxed_u64(&job.state[k], kStatePrefix | (tainted ? kStateTaint : 0ull) | epoch_bits(job.epoch) |
                                                  (unsigned long long)(before + wide_count));
            } else {
                if (outcome == 3) report(status, ENEC_ERR_TIMEOUT);
                st_relaxed_u64(&job.state[k], kStatePoison | epoch_bits(job.epoch));
                sh.poisoned = 1;
                sh.tainted = 1;
                sh.before = 0;
            }
        }
    } else if (tid == 0 && k == 0) {
        sh.before = 0;
        sh.poisoned = 0;
        sh.tainted = own_taint ? 1u : 0u;
    }
    __syncthreads();
    const uint32_t before = sh.before;
    const bool poisoned = sh.poisoned != 0;
    const uint32_t hbits = uint32_t(t.hbits);
    uint32_t* table = reinterpret_cast<uint32_t*>(job.out + t.sec.table);
    if (!poisoned) {
        // records to their place in the stream: record r of the tensor at r * 2 * hbits
        uint16_t* dst = reinterpret_cast<uint16_t*>(job.out + t.sec.high + uint64_t(before) * 2 * hbits);
        const uint16_t* src = reinterpret_cast<const uint16_t*>(rec);
        for (uint32_t i = tid; i < wide_count * hbits; i += kEncodeThreads) dst[i] = src[i];
        if (tid == 0) table[k] = before;
    }
    if constexpr (RANKED) {
        if (k + 1 == t.g.nblocks) job.out[t.sec.unmap + tid] = job.ctl->unmap[tid];  // 256 threads, 256 bytes
    }
    if (k + 1 == t.g.nblocks && tid == 0) {
        const uint32_t a_total = before + wide_count;
        const uint64_t high_bytes = uint64_t(a_total) * 2 * hbits;
        const uint64_t total = t.sec.high + align16(high_bytes);
        const bool failed = poisoned || sh.tainted != 0;
        Header hd;
        hd.magic = failed ? 0 : kMagic;
        hd.version = kVersion;
        hd.dtype = DT;
        hd.variant = RANKED ? 1 : 0;
        hd.count = job.count;
        hd.block = kBlockElems;
        hd.b = uint8_t(t.b); hd.n = uint8_t(t.n); hd.m = uint8_t(t.m); hd.L = kGroupElems;
        hd.nblocks = t.g.nblocks;
        hd.total_groups = t.g.total_groups;
        hd.a_total = a_total;
        hd.pad1 = 0;
        hd.total_bytes = total;
        hd.pad2[0] = hd.pad2[1] = 0;
        *reinterpret_cast<Header*>(job.out) = hd;
        if (!poisoned) {
            table[t.g.nblocks] = a_total;
            for (uint64_t i = uint64_t(t.g.nblocks) + 1; i < align16(4 * (uint64_t(t.g.nblocks) + 1)) / 4; ++i) table[i] = 0;
            for (uint64_t p = high_bytes; p < align16(high_bytes); p += 2)
                *reinterpret_cast<uint16_t*>(job.out + t.sec.high + p) = 0;
        }
        if (job.out_size) *job.out_size = failed ? 0ull : total;
    }
}

// A list of tensors compressed by one launch: the blocks of all tensors form one index space that the
// CTAs' tickets run over; every tensor keeps its own control words, state words and output.
struct EncodeBatch {
    const EncodeJob* jobs;   // device array [n_jobs]
    const uint32_t* prefix;  // device array [n_jobs + 1]: blocks before each tensor
    uint32_t n_jobs;
    uint32_t total_blocks;
    uint32_t* ticket;        // next block of the index space (zero when the launch starts)
};

// What a block needs to know about its tensor (batched launches keep it in shared memory per block).
struct BlockCtx {
    EncodeJob job;
    EncodeTensor tensor;
    TransformCtx tc;
    uint32_t k;  // block index inside the tensor
};

template <int DT, bool RANKED = false>
__device__ __forceinline__ void fill_tensor_ctx(const EncodeJob& job, EncodeTensor& tensor, TransformCtx& tc) {
    constexpr int E = DT == ENEC_FP16 ? 5 : 8;
    int b = job.b, n = job.n, m = job.m;
    if (job.from_search) { b = job.ctl->b; n = job.ctl->n; m = job.ctl->m; }
    tensor.g = make_geometry(job.count);
    tensor.sec = make_sections(DT, job.count, tensor.g, n, m, 0, RANKED);
    tensor.b = b; tensor.n = n; tensor.m = m; tensor.hbits = n - m;
    tc.b4 = rep4(uint32_t(b));
    tc.b4_or_h = tc.b4 | 0x80808080u;
    tc.nmask4 = rep4((1u << n) - 1);
    tc.s4 = rep4(1u << (n - 1));
    tc.emask4 = rep4((1u << E) - 1);
    tc.n = n;
    tc.E = E;
    tc.lut = 0;
}

// BATCH = false: one tensor, described by `single`. BATCH = true: the tensors of `batch`; `single` is unused.
// RANKED (one tensor only): the frequency-rank variant; a separate instance, so that the usual one carries
// nothing of the table look-ups.
template <int DT, bool BATCH, bool RANKED = false>
__global__ void __launch_bounds__(kEncodeThreads, 4)
enec_encode_kernel(const EncodeJob single, const EncodeBatch batch, int* status) {
    // dynamic shared memory: low plane | fp16 sign/mantissa-high plane | two record buffers
    extern __shared__ __align__(16) uint8_t enc_smem[];
    uint8_t* s_low = enc_smem;                                   // normalised bytes of the low plane
    uint8_t* s_hi3 = enc_smem + kBlockElems;                     // fp16 only
    uint8_t* s_rec_base = s_hi3 + EncodeSmem<DT>::kHi3Bytes;     // wide groups in rank order: 16 value bytes, then packed
    __shared__ EncodeShared sh;

    pdl_launch_dependents();
    pdl_wait();  // nothing above touches global memory
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    __shared__ uint8_t s_lut[RANKED ? 256 : 1];
    __shared__ BlockCtx s_ctx[BATCH ? 3 : 1];  // batched: this block's, the previous block's and the next block's tensor
    EncodeTensor single_tensor{};
    TransformCtx single_tc{};
    if constexpr (!BATCH) {
        if (blockIdx.x == 0) {  // the next call on this scratch area finds its control set zeroed
            single.ctl_next->hist[tid] = 0;
            if (tid == 0) { single.ctl_next->ticket = 0; single.ctl_next->hist_done = 0; single.ctl_next->reserved = 0; }
        }
        fill_tensor_ctx<DT, RANKED>(single, single_tensor, single_tc);
        if constexpr (RANKED) {  // the exponent -> rank table of the tensor, for every block of this CTA
            s_lut[tid] = single.ctl->lut[tid];
            single_tc.lut = smem_u32(s_lut);
        }
    }
    uint32_t* const ticket = BATCH ? batch.ticket : &single.ctl->ticket;
    const uint32_t total_blocks = BATCH ? batch.total_blocks : single_tensor.g.nblocks;
    // batched, thread 0 only: the tensor of a ticket (tickets of a CTA grow, so the search only moves forward)
    uint32_t ctx_j = 0;
    auto stage_ctx = [&](uint32_t ticket_value, uint32_t slot) {
        if (ticket_value >= total_blocks) return;
        while (batch.prefix[ctx_j + 1] <= ticket_value) ++ctx_j;
        BlockCtx& cx = s_ctx[slot];
        cx.job = batch.jobs[ctx_j];
        fill_tensor_ctx<DT>(cx.job, cx.tensor, cx.tc);
        cx.k = ticket_value - batch.prefix[ctx_j];
    };

    // Persistent loop over tickets. A block's look-back is put off until the CTA has done the first half of
    // its next block: by then the predecessors, which started at about the same time, have published their
    // counts, so the wait that would otherwise hold the whole CTA is gone. Every count is published
    // before its CTA waits for anything, and a wait only concerns blocks with smaller indices, so all
    // waits end.
    uint32_t pending_block = 0xFFFFFFFFu, pending_wide = 0, cur = 0;
    bool pending_bad = false;
    if (tid == 0) {
        sh.next[0] = atomicAdd(ticket, 1u);
        if constexpr (BATCH) stage_ctx(sh.next[0], 0);
    }
    uint32_t iter = 0;
    for (;; ++iter) {
    __syncthreads();
    if (sh.next[iter & 1] >= total_blocks) break;
    // the ticket after this one goes to the other slot, which nobody reads before the next barrier
    if (tid == 0) {
        sh.next[(iter + 1) & 1] = atomicAdd(ticket, 1u);
        if constexpr (BATCH) stage_ctx(sh.next[(iter + 1) & 1], (iter + 1) % 3);
    }
    const BlockCtx& cx = s_ctx[BATCH ? iter % 3 : 0];
    const EncodeJob& job = BATCH ? cx.job : single;
    const EncodeTensor& tensor = BATCH ? cx.tensor : single_tensor;
    const TransformCtx& tc = BATCH ? cx.tc : single_tc;
    const Geometry& g = tensor.g;
    const Sections& sec = tensor.sec;
    const int b = tensor.b, n = tensor.n, m = tensor.m, hbits = tensor.hbits;
    const uint32_t k = BATCH ? cx.k : sh.next[iter & 1];
    uint8_t* s_rec = s_rec_base + cur * EncodeSmem<DT>::kRecBytes;
    const bool last = k + 1 == g.nblocks;
    const uint32_t N = last ? g.tail_padded : kBlockElems;
    const uint32_t real = last ? g.tail_real : kBlockElems;
    constexpr uint32_t kElemBytes = DT == ENEC_FP32 ? 4 : 2;
    const uint8_t* in_bytes = reinterpret_cast<const uint8_t*>(job.in) + uint64_t(k) * kBlockElems * kElemBytes;
    const uint16_t* in = reinterpret_cast<const uint16_t*>(in_bytes);
    uint8_t* out_smlo = job.out + sec.smlo + uint64_t(k) * kBlockElems * 2;  // fp32 only
    uint8_t* out_sm = job.out + sec.sm + uint64_t(k) * kBlockElems;
    uint8_t* out_low = job.out + sec.low + uint64_t(k) * (kBlockElems / 8) * uint32_t(m);
    uint8_t* out_smhi = job.out + sec.smhi + uint64_t(k) * (kBlockElems / 8) * 3;
    uint8_t* out_mask = job.out + sec.mask + uint64_t(k) * (kGroupsPerBlock / 8);

    int bad = 0;
    uint2 y[8];
    uint32_t wide_bits = 0;  // bit c: the group of run c is wide
    const bool fast = N == kBlockElems && real == kBlockElems;
    // fast path: lanes l and l + 16 share a group, so a ballot's low half is the mask of sixteen groups
    const uint32_t perm = fast ? (warp * 32 + 2 * (lane & 15) + (lane >> 4)) : tid;
    const uint32_t pair_delta = fast ? 16 : 1;
    const bool first_of_pair = fast ? lane < 16 : (lane & 1) == 0;
    const uint32_t n8 = N >> 3;
    const uint32_t j = 8 * perm;
    const bool active = N >= 128 && perm < (N >> 6);

    uint2 hs[8];
    if (fast) {
        if (!RANKED && !job.check && n < 8)
            wide_bits = encode_full_runs<DT, true>(in_bytes + j * kElemBytes, out_sm + j, out_smlo + j * 2, tc, m, warp, lane, sh.mask, y, hs, bad);
        else
            wide_bits = encode_full_runs<DT, false, RANKED>(in_bytes + j * kElemBytes, out_sm + j, out_smlo + j * 2, tc, m, warp, lane, sh.mask, y, hs, bad);
        uint2 ylow[8];
        const uint32_t lowmask4 = rep4((1u << m) - 1);
#pragma unroll
        for (int c = 0; c < 8; ++c) ylow[c] = make_uint2(y[c].x & lowmask4, y[c].y & lowmask4);
        pack_plane_any(m, smem_u32(s_low), j, N, ylow);
        if (DT == ENEC_FP16) pack_plane<3>(smem_u32(s_hi3), j, N, hs);
    } else if (N >= 128) {
        if (tid < 32) sh.mask[tid] = 0;
        __syncthreads();
        uint4 raw[8];
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t e0 = c * n8 + j;
            raw[c] = make_uint4(0, 0, 0, 0);
            if (active) {
                if (e0 + 8 <= real) {
                    if constexpr (DT == ENEC_FP32) raw[c] = load_fp32_run(in_bytes + e0 * 4, out_smlo + e0 * 2);
                    else raw[c] = __ldcs(reinterpret_cast<const uint4*>(in + e0));
                } else if (e0 < real) {
                    uint32_t v[4] = {0, 0, 0, 0};
                    for (uint32_t i = 0; e0 + i < real; ++i) {
                        uint32_t half;  // the 16-bit word that takes the exponent path
                        if constexpr (DT == ENEC_FP32) {
                            const uint32_t full = reinterpret_cast<const uint32_t*>(in_bytes)[e0 + i];
                            reinterpret_cast<uint16_t*>(out_smlo)[e0 + i] = uint16_t(full);
                            half = full >> 16;
                        } else {
                            half = in[e0 + i];
                        }
                        v[i >> 1] |= half << (16 * (i & 1));
                    }
                    raw[c] = make_uint4(v[0], v[1], v[2], v[3]);
                }
                if constexpr (DT == ENEC_FP32) {  // zeros up to the plane's 16-byte boundary
                    for (uint32_t i = 0; i < 8; ++i)
                        if (e0 + i >= real && 2 * (e0 + i) < uint32_t(align16(2 * real)))
                            reinterpret_cast<uint16_t*>(out_smlo)[e0 + i] = 0;
                }
            }
        }
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t e0 = c * n8 + j;
            const Split4 s0 = split4<DT>(raw[c].x, raw[c].y);
            const Split4 s1 = split4<DT>(raw[c].z, raw[c].w);
            uint32_t d0 = 0, d1 = 0;
            if constexpr (RANKED) {  // frequency-rank variant (never with job.check)
                y[c] = make_uint2(lut4(tc.lut, s0.x), lut4(tc.lut, s1.x));
            } else {
                d0 = bytewise_b_minus(tc, s0.x);
                d1 = bytewise_b_minus(tc, s1.x);
                y[c] = make_uint2(d0 & tc.nmask4, d1 & tc.nmask4);
            }
            hs[c] = make_uint2(s0.hs, s1.hs);
            if (active && e0 + 8 > real) {  // padding elements carry y = 0
                const uint32_t valid = e0 < real ? real - e0 : 0;
                const uint32_t k0 = valid >= 4 ? 0xFFFFFFFFu : (1u << (8 * valid)) - 1;
                const uint32_t k1 = valid >= 8 ? 0xFFFFFFFFu : valid > 4 ? (1u << (8 * (valid - 4))) - 1 : 0;
                y[c].x &= k0;
                y[c].y &= k1;
            }
            if (!active) y[c] = make_uint2(0, 0);
            if (job.check && active && e0 + 8 <= real)
                bad |= (lossy_bytes(tc, d0, y[c].x) | lossy_bytes(tc, d1, y[c].y)) != 0;
            else if (job.check && active && e0 < real) {
                const uint32_t valid = real - e0;
                const uint32_t k0 = valid >= 4 ? 0xFFFFFFFFu : (1u << (8 * valid)) - 1;
                const uint32_t k1 = valid > 4 ? (1u << (8 * (valid - 4))) - 1 : 0;
                bad |= ((lossy_bytes(tc, d0, y[c].x) & k0) | (lossy_bytes(tc, d1, y[c].y) & k1)) != 0;
            }
            if (active && e0 < uint32_t(align16(real)))
                __stcs(reinterpret_cast<uint2*>(out_sm + e0), make_uint2(s0.sm, s1.sm));
            uint32_t o = y[c].x | y[c].y;
            o |= o >> 16;
            o |= o >> 8;
            o |= __shfl_xor_sync(0xFFFFFFFFu, o, pair_delta);
            const bool wide = ((o & 0xFFu) >> m) != 0;
            wide_bits |= uint32_t(wide) << c;
            if (fast) {
                const uint32_t bal = __ballot_sync(0xFFFFFFFFu, wide);
                if (lane == 0) reinterpret_cast<uint16_t*>(sh.mask)[c * 8 + warp] = uint16_t(bal);
            } else if (wide && first_of_pair && active) {
                const uint32_t grp = e0 >> 4;
                atomicOr(&sh.mask[grp >> 5], 1u << (grp & 31));
            }
        }
        if (active) {
            uint2 ylow[8];
            const uint32_t lowmask4 = rep4((1u << m) - 1);
#pragma unroll
            for (int c = 0; c < 8; ++c) ylow[c] = make_uint2(y[c].x & lowmask4, y[c].y & lowmask4);
            pack_plane_any(m, smem_u32(s_low), j, N, ylow);
            if (DT == ENEC_FP16) pack_plane<3>(smem_u32(s_hi3), j, N, hs);
        }
    } else {
        bad = encode_short_block<DT>(in, N, real, tc, b, n, m, job.check, out_sm, out_low, out_smhi, out_mask, out_smlo, &sh,
                                     reinterpret_cast<uint32_t*>(s_low), reinterpret_cast<uint32_t*>(s_hi3),
                                     reinterpret_cast<uint32_t*>(s_rec));
    }
    const int any_bad = __syncthreads_or(bad);
    {
        // the CTA's next block is known by now: pull its 32 KB towards L2 (one 128-byte line per thread, two for fp32)
        // so that the loads of the next iteration do not wait for DRAM
        const uint32_t next_block = BATCH ? 0xFFFFFFFFu : sh.next[(iter + 1) & 1];  // batched: tensors are small
        if (next_block < g.nblocks) {
            const uint8_t* base = reinterpret_cast<const uint8_t*>(job.in);
            const uint8_t* end = base + job.count * kElemBytes;
#pragma unroll
            for (uint32_t r = 0; r < kElemBytes / 2; ++r) {
                const uint8_t* line = base + uint64_t(next_block) * kBlockElems * kElemBytes + (r * kEncodeThreads + tid) * 128;
                if (line < end) asm volatile("prefetch.global.L2 [%0];" ::"l"(line));
            }
        }
    }

    // wide groups before each mask word and in the block: every warp scans the 32 mask words itself
    // (lane l holds word l), so no second barrier is needed
    const uint32_t mask_word = sh.mask[lane];
    uint32_t mask_incl = __popc(mask_word);
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, mask_incl, d);
        if (lane >= uint32_t(d)) mask_incl += t;
    }
    const uint32_t mask_excl = mask_incl - __popc(mask_word);
    const uint32_t wide_count = __shfl_sync(0xFFFFFFFFu, mask_incl, 31);
    if (tid == 31) {
        if (any_bad) report(status, ENEC_ERR_PARAMS_NOT_LOSSLESS);
        // publish this block's count at once; block 0 knows its prefix already
        st_relaxed_u64(&job.state[k], (k == 0 ? kStatePrefix : kStateAggregate) | (any_bad ? kStateTaint : 0ull) |
                                          epoch_bits(job.epoch) | wide_count);
    }
    if (N >= 128) {
        fold_plane_out(smem_u32(s_low), N * uint32_t(m) / 8, out_low, tid);
        if (DT == ENEC_FP16) fold_plane_out(smem_u32(s_hi3), N * 3 / 8, out_smhi, tid);
        const uint32_t mask_vecs = uint32_t(align16(((N >> 4) + 7) / 8)) / 16;
        if (tid < mask_vecs)
            reinterpret_cast<uint4*>(out_mask)[tid] = reinterpret_cast<const uint4*>(sh.mask)[tid];
        // high bits of wide groups into shared memory, rank order, sixteen value bytes per group: each
        // lane of a pair stores its own half; narrow groups store to a spare slot behind the buffer, so
        // there is no branch
        if (hbits > 0) {
            const uint32_t hmask4 = rep4(0xFFu >> m);
            const uint32_t half_off = first_of_pair ? 0 : 8;
            const uint32_t spare = kGroupsPerBlock * 16;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const uint32_t grp = (c * n8 + j) >> 4;
                const uint32_t word = (grp >> 5) & 31;
                const uint32_t rank = __shfl_sync(0xFFFFFFFFu, mask_excl, word) +
                                      __popc(__shfl_sync(0xFFFFFFFFu, mask_word, word) & ((1u << (grp & 31)) - 1));
                const bool wide = ((wide_bits >> c) & 1) && active;
                sts64(smem_u32(s_rec) + (wide ? rank * 16 : spare) + half_off,
                      make_uint2((y[c].x >> m) & hmask4, (y[c].y >> m) & hmask4));
            }
        }
    }
    // Algorithm 2 over each wide group, one group per thread, packed in place: record i (2 hbits bytes)
    // lands below the value bytes of every group that has not been read yet
    if (N >= 128 && hbits > 0) {
        __syncthreads();
        for (uint32_t base = 0; base < wide_count; base += kEncodeThreads) {
            const uint32_t i = base + tid;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (i < wide_count) v = lds128(smem_u32(s_rec) + i * 16);
            __syncthreads();
            if (i < wide_count) pack_record_any(hbits, v, smem_u32(s_rec) + i * 2 * hbits);
        }
    }

    // the previous block of this CTA, whose records wait in the other buffer
    if (pending_block != 0xFFFFFFFFu) {
        const BlockCtx& px = s_ctx[BATCH ? (iter + 2) % 3 : 0];
        resolve_block<DT, RANKED>(BATCH ? px.job : single, BATCH ? px.tensor : single_tensor, pending_block, pending_wide, pending_bad,
                          s_rec_base + (cur ^ 1) * EncodeSmem<DT>::kRecBytes, sh, status);
    }
    pending_block = k;
    pending_wide = wide_count;
    pending_bad = any_bad != 0;
    cur ^= 1;
    }
    if (pending_block != 0xFFFFFFFFu) {
        const BlockCtx& px = s_ctx[BATCH ? (iter + 2) % 3 : 0];
        resolve_block<DT, RANKED>(BATCH ? px.job : single, BATCH ? px.tensor : single_tensor, pending_block, pending_wide, pending_bad,
                          s_rec_base + (cur ^ 1) * EncodeSmem<DT>::kRecBytes, sh, status);
    }
}

// Stream of an empty tensor: header, (frequency-rank variant: an all-zero rank table) and a one-entry table
// (16 zero bytes in every variant).
__global__ void enec_encode_empty_kernel(uint8_t* out, int dt, int b, int n, int m, unsigned long long* out_size,
                                         int variant = 0) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const uint32_t table_at = kHeaderBytes + (variant == 1 ? kRankTableBytes : 0);
    Header hd;
    hd.magic = kMagic;
    hd.version = kVersion;
    hd.dtype = uint8_t(dt);
    hd.variant = uint8_t(variant);
    hd.count = 0;
    hd.block = kBlockElems;
    hd.b = uint8_t(b); hd.n = uint8_t(n); hd.m = uint8_t(m); hd.L = kGroupElems;
    hd.nblocks = 0;
    hd.total_groups = 0;
    hd.a_total = 0;
    hd.pad1 = 0;
    hd.total_bytes = table_at + 16;
    hd.pad2[0] = hd.pad2[1] = 0;
    *reinterpret_cast<Header*>(out) = hd;
    for (uint32_t at = kHeaderBytes; at <= table_at; at += 16) *reinterpret_cast<uint4*>(out + at) = make_uint4(0, 0, 0, 0);
    if (out_size) *out_size = table_at + 16;
}

}  // namespace enec
