// The block-wise variant of the compressor, kept for the ablation (Sec. 5.5 run on every block's own histogram
// instead of the tensor's; Sec. 6.4 / 6.6 discuss how far the parameters carry over).
//
// Stream: header byte 7 = 2, header bytes 20..22 zero; in place of the prefix table a block table of 16-byte
// entries {b, n, m, 0, u32 sum of m over the blocks before, u64 record bytes before}, one per block and one more
// with the totals; block k's low plane starts 2048 x (sum of m before) bytes into the low section, its records
// (record bytes before) into the record section. Everything else is laid out as by enec_compress.
//
//   enec_block_params_kernel  per block: histogram in shared memory, the search of Sec. 5.5 by the CTA, the
//                             block's wide groups counted from the values still in registers; the CTA that
//                             finishes the last outstanding block turns the entries into running sums (the
//                             block-offset scan of Sec. 5.1 / 5.4) and writes the header.
//   enec_pack_blocks_kernel   per block: split, transform, group widths, Algorithm 2, straight to the offsets
//                             the table gives. No CTA waits for another one.
// The input is read twice, as by enec_compress (histogram pass, encode pass).
#pragma once

#include "enec_pack.cuh"

namespace enec {

struct alignas(16) BlockEntry {
    uint8_t b, n, m, zero;
    uint32_t m_before;                // sum of m over the blocks before this one (low plane offset / 2048)
    unsigned long long rec_before;    // bytes of records before this block's first record
};
static_assert(sizeof(BlockEntry) == 16, "a block table entry is 16 bytes");

__host__ __device__ inline Sections make_sections_blockwise(int dt, uint64_t count, const Geometry& g, uint64_t low_bytes,
                                                           uint64_t high_bytes) {
    Sections s;
    s.unmap = kHeaderBytes;
    s.table = kHeaderBytes;
    s.mask = s.table + align16(16 * (uint64_t(g.nblocks) + 1));
    s.low = s.mask + align16((uint64_t(g.total_groups) + 7) / 8);
    s.smhi = s.low + align16(low_bytes);
    s.sm = s.smhi + (dt == ENEC_FP16 ? align16(g.padded_count * 3 / 8) : 0);
    s.smlo = s.sm + align16(count);
    s.high = s.smlo + (dt == ENEC_FP32 ? align16(count * 2) : 0);
    s.total = s.high + align16(high_bytes);
    return s;
}

struct BlockwiseJob {
    const uint16_t* in;
    uint8_t* out;
    uint64_t count;
    uint32_t* done;                // blocks whose entry is written (zero when the call starts); done[1] and done[2] are
                                   // the tickets that hand out the blocks in the two kernels (each zeroed by the other kernel)
    unsigned long long* out_size;  // device, may be null
};

constexpr int kBlockwiseThreads = kPackThreads;

// The block table's entries hold each block's own m and record bytes: turn them into sums over the blocks
// before, append the totals and write the header. All threads of one CTA, after every entry is visible.
template <int DT>
__device__ inline void finish_block_table(const BlockwiseJob& job, const Geometry& g) {
    __shared__ unsigned long long s_warp_total[8], s_warp_wide[8];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t nblocks = g.nblocks;
    unsigned long long* words = reinterpret_cast<unsigned long long*>(job.out + kHeaderBytes);  // two per entry
    unsigned long long carry = 0;   // bits 37..0 record bytes so far, bits 63..38 sum of m so far
    unsigned long long wide_total = 0;
    for (uint32_t base = 0; base < nblocks; base += kBlockwiseThreads * 8) {
        const uint32_t first = base + tid * 8;
        unsigned long long params[8], run[8];
        unsigned long long sum = 0, wide = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            params[q] = 0;
            if (first + q < nblocks) {
                const unsigned long long w0 = ld_relaxed_u64(&words[2 * (first + q)]);
                const unsigned long long rec = ld_relaxed_u64(&words[2 * (first + q) + 1]);
                params[q] = w0 & 0xFFFFFFFFull;
                const uint32_t n = uint32_t(w0 >> 8) & 0xFF, m = uint32_t(w0 >> 16) & 0xFF;
                run[q] = sum;
                sum += rec | ((unsigned long long)m << 38);
                wide += n > m ? rec / (2 * (n - m)) : 0;
            }
        }
        unsigned long long incl = sum;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
            if (lane >= uint32_t(d)) incl += t;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) wide += __shfl_xor_sync(0xFFFFFFFFu, wide, d);
        __syncthreads();  // the previous chunk's totals have been read
        if (lane == 31) s_warp_total[warp] = incl;
        if (lane == 0) s_warp_wide[warp] = wide;
        __syncthreads();
        unsigned long long offset = carry + incl - sum;
        unsigned long long chunk = 0;
#pragma unroll
        for (uint32_t wq = 0; wq < 8; ++wq) {
            if (wq < warp) offset += s_warp_total[wq];
            chunk += s_warp_total[wq];
            wide_total += s_warp_wide[wq];
        }
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            if (first + q < nblocks) {
                const unsigned long long p = offset + run[q];
                words[2 * (first + q)] = params[q] | ((p >> 38) << 32);
                words[2 * (first + q) + 1] = p & ((1ull << 38) - 1);
            }
        }
        carry += chunk;
    }
    __syncthreads();  // every entry is in its final form
    if (tid == 0) {
        const uint64_t m_sum = carry >> 38, high_bytes = carry & ((1ull << 38) - 1);
        words[2 * uint64_t(nblocks)] = m_sum << 32;
        words[2 * uint64_t(nblocks) + 1] = high_bytes;
        for (uint64_t i = 2 * (uint64_t(nblocks) + 1); i < align16(16 * (uint64_t(nblocks) + 1)) / 8; ++i) words[i] = 0;
        // low plane: 2048 m bytes per full block; the tail block's padded length times its m over 8
        const uint32_t m_tail = uint32_t(ld_relaxed_u64(&words[2 * uint64_t(nblocks - 1)]) >> 16) & 0xFF;
        const uint64_t low_bytes = (m_sum - m_tail) * (kBlockElems / 8) + uint64_t(g.tail_padded) * m_tail / 8;
        const Sections sec = make_sections_blockwise(DT, job.count, g, low_bytes, high_bytes);
        Header hd;
        hd.magic = kMagic;
        hd.version = kVersion;
        hd.dtype = DT;
        hd.variant = 2;
        hd.count = job.count;
        hd.block = kBlockElems;
        hd.b = 0; hd.n = 0; hd.m = 0; hd.L = kGroupElems;
        hd.nblocks = nblocks;
        hd.total_groups = g.total_groups;
        hd.a_total = uint32_t(wide_total);
        hd.pad1 = 0;
        hd.total_bytes = sec.total;
        hd.pad2[0] = hd.pad2[1] = 0;
        *reinterpret_cast<Header*>(job.out) = hd;
        // padding behind the variable sections that no block writes
        for (uint64_t p = low_bytes; p < align16(low_bytes); p += 2) *reinterpret_cast<uint16_t*>(job.out + sec.low + p) = 0;
        for (uint64_t p = high_bytes; p < align16(high_bytes); p += 2) *reinterpret_cast<uint16_t*>(job.out + sec.high + p) = 0;
        if (job.out_size) *job.out_size = sec.total;
        *job.done = 0;  // ready for the next call on this scratch
    }
}

// Wide groups of a full block from the values a thread holds (run c of thread t = elements c * 2048 + 8 t; lanes
// 2i and 2i + 1 hold the two halves of a group); the calling warp's share, the same in every lane.
template <int DT>
__device__ __forceinline__ uint32_t count_wide_full(const uint4 (&raw)[8], const TransformCtx& tc, int m) {
    const uint32_t widemask4 = ~rep4((1u << m) - 1);
    uint32_t count = 0;
#pragma unroll
    for (int c = 0; c < 8; ++c) {
        const Split4 s0 = split4<DT>(raw[c].x, raw[c].y);
        const Split4 s1 = split4<DT>(raw[c].z, raw[c].w);
        const uint32_t y0 = bytewise_b_minus(tc, s0.x) & tc.nmask4;
        const uint32_t y1 = bytewise_b_minus(tc, s1.x) & tc.nmask4;
        const uint32_t halves = __ballot_sync(0xFFFFFFFFu, ((y0 | y1) & widemask4) != 0);
        count += __popc((halves | (halves >> 1)) & 0x55555555u);
    }
    return count;
}

template <int DT>
__global__ void __launch_bounds__(kBlockwiseThreads, 3)
enec_block_params_kernel(const BlockwiseJob job, int* status) {
    extern __shared__ __align__(128) uint8_t smem[];  // the CTA's 32 copies of the histogram (see enec_histogram_kernel)
    __shared__ uint32_t s_part[kBlockwiseThreads / 32];
    __shared__ int s_last;
    constexpr uint32_t kElemBytes = DT == ENEC_FP32 ? 4 : 2;
    constexpr int E = HistShape<DT>::E;
    pdl_launch_dependents();
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t base = smem_u32(smem) + lane * 4;
    for (uint32_t i = tid; i < uint32_t(HistShape<DT>::kBytes / 16); i += kBlockwiseThreads)
        reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
    __syncthreads();
    pdl_wait();  // nothing above touches global memory
    const Geometry g = make_geometry(job.count);
    BlockEntry* table = reinterpret_cast<BlockEntry*>(job.out + kHeaderBytes);
    // CTA c starts on block c; after that blocks are handed out by a ticket, asked for a block ahead (the CTAs of an
    // SM do not progress equally). The pack kernel's ticket, last used by the call before, is cleared here.
    __shared__ uint32_t s_next_block;
    if (blockIdx.x == 0 && tid == 0) job.done[2] = 0;
    for (uint32_t k = blockIdx.x; k < g.nblocks;) {
        uint32_t asked = 0;
        if (tid == 0) asked = atomicAdd(&job.done[1], 1u);
        const bool last = k + 1 == g.nblocks;
        const uint32_t N = last ? g.tail_padded : kBlockElems;
        const uint32_t real = last ? g.tail_real : kBlockElems;
        const uint8_t* in_bytes = reinterpret_cast<const uint8_t*>(job.in) + uint64_t(k) * kBlockElems * kElemBytes;
        const bool full = real == kBlockElems;
        uint4 raw[8];  // full blocks: the thread's eight runs as 16-bit words (fp32: the high halves)
        if (full) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                if constexpr (DT == ENEC_FP32) {
                    const uint4* p = reinterpret_cast<const uint4*>(in_bytes + (c * (kBlockElems / 8) + 8 * tid) * 4);
                    const uint4 a0 = __ldg(p), a1 = __ldg(p + 1);
                    raw[c] = make_uint4(prmt(a0.x, a0.y, 0x7632u), prmt(a0.z, a0.w, 0x7632u), prmt(a1.x, a1.y, 0x7632u),
                                        prmt(a1.z, a1.w, 0x7632u));
                } else {
                    raw[c] = __ldg(reinterpret_cast<const uint4*>(in_bytes + (c * (kBlockElems / 8) + 8 * tid) * 2));
                }
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {  // the high halves of fp32 values have bf16's layout
                constexpr int HDT = DT == ENEC_FP32 ? ENEC_BF16 : DT;
                count_word_pair<HDT>(base, raw[c].x);
                count_word_pair<HDT>(base, raw[c].y);
                count_word_pair<HDT>(base, raw[c].z);
                count_word_pair<HDT>(base, raw[c].w);
            }
        } else {
            for (uint32_t i = tid; i < real; i += kBlockwiseThreads)
                red_add_one(base + exponent_of_word<DT>(exponent_word<DT>(in_bytes, i)) * HistShape<DT>::kRowBytes);
        }
        __syncthreads();
        const unsigned long long mine =
            tid < uint32_t(1 << E) ? fold_hist_row<true>(smem_u32(smem) + tid * HistShape<DT>::kRowBytes, tid) : 0u;
        int b, n, m;
        parameter_search_counts<DT>(mine, b, n, m);
        const TransformCtx tc = make_transform_ctx(E, b, n);
        uint32_t wide;
        if (full) {
            wide = count_wide_full<DT>(raw, tc, m);
        } else {
            wide = 0;
            for (uint32_t grp = tid; grp < (N >> 4); grp += kBlockwiseThreads) {
                uint32_t o = 0;
                for (uint32_t e = 0; e < 16 && grp * 16 + e < real; ++e)  // padding carries y = 0
                    o |= uint32_t(b - int(exponent_of_word<DT>(exponent_word<DT>(in_bytes, grp * 16 + e)))) & ((1u << n) - 1);
                wide += (o >> m) != 0;
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) wide += __shfl_xor_sync(0xFFFFFFFFu, wide, d);
        }
        if (lane == 0) s_part[warp] = wide;
        __syncthreads();
        if (tid == 0) {
            uint32_t total = 0;
            for (int w = 0; w < kBlockwiseThreads / 32; ++w) total += s_part[w];
            BlockEntry e;
            e.b = uint8_t(b); e.n = uint8_t(n); e.m = uint8_t(m); e.zero = 0;
            e.m_before = 0;
            e.rec_before = (unsigned long long)total * 2 * uint32_t(n - m);   // this block's own; summed up at the end
            table[k] = e;
            __threadfence();
            s_last = atomicAdd(job.done, 1u) + 1 == g.nblocks;
            s_next_block = gridDim.x + asked;
        }
        __syncthreads();
        k = s_next_block;
        if (s_last) {
            __threadfence();
            finish_block_table<DT>(job, g);
        }
    }
    (void)status;
}

// CTA c packs the blocks c, c + grid, ...; everything it needs about a block is in the block's table entry.
template <int DT>
__global__ void __launch_bounds__(kBlockwiseThreads, 4)
enec_pack_blocks_kernel(const BlockwiseJob job, int* status) {
    extern __shared__ __align__(16) uint8_t pack_smem[];
    __shared__ __align__(16) uint32_t s_mask[32];
    constexpr uint32_t kElemBytes = DT == ENEC_FP32 ? 4 : 2;
    pdl_launch_dependents();
    pdl_wait();  // nothing above touches global memory
    const Geometry g = make_geometry(job.count);
    const BlockEntry* table = reinterpret_cast<const BlockEntry*>(job.out + kHeaderBytes);
    const BlockEntry totals = table[g.nblocks];
    const uint32_t m_tail = table[g.nblocks - 1].m;
    const uint64_t low_bytes = uint64_t(totals.m_before - m_tail) * (kBlockElems / 8) + uint64_t(g.tail_padded) * m_tail / 8;
    const Sections sec = make_sections_blockwise(DT, job.count, g, low_bytes, totals.rec_before);
    // blocks c and c + grid, then blocks handed out by the call's second ticket, asked for two blocks ahead; the first
    // kernel's ticket is cleared here for the next call
    __shared__ uint32_t s_next;
    const uint32_t tid = threadIdx.x;
    if (blockIdx.x == 0 && tid == 0) job.done[1] = 0;
    uint32_t k = blockIdx.x, k_next = blockIdx.x + gridDim.x;
    while (k < g.nblocks) {
        uint32_t asked = 0;
        if (tid == 0) asked = atomicAdd(&job.done[2], 1u);
        const BlockEntry entry = table[k];
        const int b = entry.b, n = entry.n, m = entry.m;
        const bool last = k + 1 == g.nblocks;
        const uint32_t N = last ? g.tail_padded : kBlockElems;
        const uint32_t real = last ? g.tail_real : kBlockElems;
        const uint8_t* in_bytes = reinterpret_cast<const uint8_t*>(job.in) + uint64_t(k) * kBlockElems * kElemBytes;
        uint8_t* out_smlo = job.out + sec.smlo + uint64_t(k) * kBlockElems * 2;  // fp32 only
        uint8_t* out_sm = job.out + sec.sm + uint64_t(k) * kBlockElems;
        uint8_t* out_low = job.out + sec.low + uint64_t(entry.m_before) * (kBlockElems / 8);
        uint8_t* out_smhi = job.out + sec.smhi + uint64_t(k) * (kBlockElems / 8) * 3;
        uint8_t* out_mask = job.out + sec.mask + uint64_t(k) * (kGroupsPerBlock / 8);
        uint8_t* out_rec = job.out + sec.high + entry.rec_before;
        if (real != kBlockElems)
            pack_tail_block<DT>(in_bytes, N, real, b, n, m, out_sm, out_low, out_smhi, out_mask, out_smlo, out_rec, pack_smem);
        else
            pack_full_block<DT>(in_bytes, b, n, m, out_sm, out_smlo, out_low, out_smhi, out_mask, out_rec, pack_smem, s_mask);
        if (tid == 0) s_next = 2 * gridDim.x + asked;
        __syncthreads();
        k = k_next;
        k_next = s_next;
        __syncthreads();  // s_next is read before the next round's write
    }
    (void)status;
}

}  // namespace enec
