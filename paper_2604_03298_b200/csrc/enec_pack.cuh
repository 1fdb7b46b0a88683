// Packing of one block without any knowledge of other blocks, shared by the block-wise variant and by the
// split form of enec_compress:
//
//   pack_full_block   a block of 16384 elements: split, transform (Sec. 5.3), group widths (Sec. 5.2), Algorithm 2
//                     for the low plane and for every wide group's record, everything written to the addresses
//                     the caller gives.
//   pack_tail_block   a tensor's last block when it is shorter.
//   enec_pack_tensor_kernel / enec_place_records_kernel
//                     enec_compress for large tensors in two kernels instead of one with a look-back: the first
//                     packs every block and leaves its records at the place they would have if every group before
//                     were wide (inside the output buffer, whose capacity covers that case), the second moves the
//                     records down to their final places (the block-offset prefix sum of Sec. 5.1 / 5.4), writes
//                     the prefix table and the header. No CTA of the first kernel waits for another one.
#pragma once

#include "enec_encode.cuh"

namespace enec {

constexpr int kPackThreads = 256;

__device__ __forceinline__ TransformCtx make_transform_ctx(int dt_exp_bits, int b, int n) {
    TransformCtx tc;
    tc.b4 = rep4(uint32_t(b));
    tc.b4_or_h = tc.b4 | 0x80808080u;
    tc.nmask4 = rep4((1u << n) - 1);
    tc.s4 = rep4(1u << (n - 1));
    tc.emask4 = rep4((1u << dt_exp_bits) - 1);
    tc.n = n;
    tc.E = dt_exp_bits;
    tc.lut = 0;
    return tc;
}

// Exponent field of element i of a block at `in_bytes`, and the 16-bit word that carries it (for fp32 the high half).
template <int DT>
__device__ __forceinline__ uint32_t exponent_word(const uint8_t* in_bytes, uint32_t i) {
    return DT == ENEC_FP32 ? reinterpret_cast<const uint32_t*>(in_bytes)[i] >> 16
                           : uint32_t(reinterpret_cast<const uint16_t*>(in_bytes)[i]);
}
template <int DT>
__device__ __forceinline__ uint32_t exponent_of_word(uint32_t w) {
    return DT != ENEC_FP16 ? (w >> 7) & 0xFFu : (w >> 10) & 0x1Fu;
}

// A tensor's last block when it is not full (N padded elements, N a power of two up to 16384, `real` present), all
// 256 threads, element by element and bit by bit (Algorithm 2 followed for every set bit). `work` is shared memory:
// mask [32 words] | low plane [16384 bytes; the fp16 plane 10240 bytes in, behind a low plane of m <= 5] | records.
template <int DT>
__device__ __forceinline__ uint32_t tail_word(const uint8_t* in_bytes, uint32_t i) {
    return DT == ENEC_FP32 ? reinterpret_cast<const uint32_t*>(in_bytes)[i] >> 16
                           : uint32_t(reinterpret_cast<const uint16_t*>(in_bytes)[i]);
}

constexpr uint32_t kTailWorkWords = 32 + kBlockElems / 4 + kGroupsPerBlock * 14 / 4;

template <int DT>
__device__ __noinline__ uint32_t pack_tail_block(const uint8_t* in_bytes, uint32_t N, uint32_t real, int b, int n, int m,
                                             uint8_t* out_sm, uint8_t* out_low, uint8_t* out_smhi, uint8_t* out_mask,
                                             uint8_t* out_smlo, uint8_t* out_rec, uint8_t* work) {
    const uint32_t tid = threadIdx.x;
    const uint32_t hbits = uint32_t(n - m);
    const uint32_t groups = N >> 4;
    const uint32_t nmask = (1u << n) - 1;
    uint32_t* s_mask = reinterpret_cast<uint32_t*>(work);
    uint32_t* s_low = s_mask + 32;
    uint32_t* s_hi3 = s_low + 10240 / 4;
    uint32_t* s_rec = s_low + kBlockElems / 4;
    for (uint32_t i = tid; i < kTailWorkWords; i += kPackThreads) s_mask[i] = 0;
    __syncthreads();
    for (uint32_t i = tid; i < N; i += kPackThreads) {
        uint32_t y = 0, hs = 0;
        if (i < real) {
            if (DT == ENEC_FP32)
                reinterpret_cast<uint16_t*>(out_smlo)[i] = uint16_t(reinterpret_cast<const uint32_t*>(in_bytes)[i]);
            const uint32_t w = tail_word<DT>(in_bytes, i);
            y = uint32_t(b - int(exponent_of_word<DT>(w))) & nmask;
            if (DT != ENEC_FP16) {
                out_sm[i] = uint8_t(((w >> 8) & 0x80) | (w & 0x7F));
            } else {
                out_sm[i] = uint8_t(w);
                hs = ((w >> 13) & 4) | ((w >> 8) & 3);
            }
        } else {
            if (i < uint32_t(align16(real))) out_sm[i] = 0;
            if (DT == ENEC_FP32 && 2 * i < uint32_t(align16(2 * uint64_t(real)))) reinterpret_cast<uint16_t*>(out_smlo)[i] = 0;
        }
        if (y >> m) atomicOr(&s_mask[i >> 9], 1u << ((i >> 4) & 31));
        for (int q = 0; q < m; ++q)
            if ((y >> q) & 1) {
                uint32_t pos; int bit;
                alg2_locate(N, m, i, q, pos, bit);
                atomicOr(&s_low[pos >> 2], 1u << (8 * (pos & 3) + bit));
            }
        if (DT == ENEC_FP16)
            for (int q = 0; q < 3; ++q)
                if ((hs >> q) & 1) {
                    uint32_t pos; int bit;
                    alg2_locate(N, 3, i, q, pos, bit);
                    atomicOr(&s_hi3[pos >> 2], 1u << (8 * (pos & 3) + bit));
                }
    }
    __syncthreads();
    if (hbits > 0) {
        for (uint32_t i = tid; i < real; i += kPackThreads) {
            const uint32_t grp = i >> 4;
            if (!((s_mask[grp >> 5] >> (grp & 31)) & 1)) continue;
            const uint32_t hv = (uint32_t(b - int(exponent_of_word<DT>(tail_word<DT>(in_bytes, i)))) & nmask) >> m;
            if (!hv) continue;
            uint32_t rank = __popc(s_mask[grp >> 5] & ((1u << (grp & 31)) - 1));
            for (uint32_t wq = 0; wq < (grp >> 5); ++wq) rank += __popc(s_mask[wq]);
            for (uint32_t q = 0; q < hbits; ++q)
                if ((hv >> q) & 1) {
                    uint32_t pos; int bit;
                    alg2_locate(16, int(hbits), i & 15, int(q), pos, bit);
                    pos += rank * 2 * hbits;
                    atomicOr(&s_rec[pos >> 2], 1u << (8 * (pos & 3) + bit));
                }
        }
    }
    __syncthreads();
    // planes out, padded to 16 bytes with zeros (the shared words behind them are zero)
    for (uint32_t i = tid; i < uint32_t(align16(uint64_t(N) * m / 8)) / 4; i += kPackThreads)
        reinterpret_cast<uint32_t*>(out_low)[i] = s_low[i];
    for (uint32_t i = tid; i < uint32_t(align16((groups + 7) / 8)) / 4; i += kPackThreads)
        reinterpret_cast<uint32_t*>(out_mask)[i] = s_mask[i];
    if (DT == ENEC_FP16)
        for (uint32_t i = tid; i < uint32_t(align16(uint64_t(N) * 3 / 8)) / 4; i += kPackThreads)
            reinterpret_cast<uint32_t*>(out_smhi)[i] = s_hi3[i];
    uint32_t wide_count = 0;
    for (uint32_t wq = 0; wq < 32; ++wq) wide_count += __popc(s_mask[wq]);
    for (uint32_t i = tid; i < wide_count * hbits; i += kPackThreads)
        reinterpret_cast<uint16_t*>(out_rec)[i] = reinterpret_cast<const uint16_t*>(s_rec)[i];
    __syncthreads();
    return wide_count;
}

constexpr uint32_t kPackSmemBytes = 2 * kBlockElems + 16;  // low plane (fp16 plane behind it) | wide groups' values + a spare slot
static_assert(kTailWorkWords * 4 <= kPackSmemBytes, "the tail packer works inside the pack kernels' shared memory");


// One full block, all 256 threads of the CTA; returns the number of wide groups (the same in every thread).
// pack_smem: kPackSmemBytes of shared memory; s_mask: 32 words of shared memory, 16-byte aligned. Ends with a
// barrier, after which both are free again.
template <int DT>
__device__ __forceinline__ uint32_t pack_full_block(const uint8_t* in_bytes, int b, int n, int m, uint8_t* out_sm,
                                                    uint8_t* out_smlo, uint8_t* out_low, uint8_t* out_smhi,
                                                    uint8_t* out_mask, uint8_t* out_rec, uint8_t* pack_smem,
                                                    uint32_t* s_mask) {
    constexpr uint32_t N = kBlockElems;
    constexpr uint32_t kSpare = kGroupsPerBlock * 16;
    constexpr uint32_t kElemBytes = DT == ENEC_FP32 ? 4 : 2;
    constexpr int E = HistShape<DT>::E;
    uint8_t* s_low = pack_smem;
    uint8_t* s_hi3 = pack_smem + 10240;  // fp16 only (m <= 5, so the low plane ends below)
    const uint32_t s_exp = smem_u32(pack_smem) + kBlockElems;
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int hbits = n - m;
    // lanes l and l + 16 share a group, so a ballot's two halves OR into the mask of sixteen groups
    const uint32_t perm = warp * 32 + 2 * (lane & 15) + (lane >> 4);
    const uint32_t j = 8 * perm;
    const uint32_t lower = (1u << ((j >> 4) & 31)) - 1;  // groups below this thread's in its mask word
    const TransformCtx tc = make_transform_ctx(E, b, n);
    uint2 y[8], hs[8];
    int bad = 0;
    uint32_t wide_bits;
    if (n < 8)
        wide_bits = encode_full_runs<DT, true>(in_bytes + j * kElemBytes, out_sm + j, out_smlo + j * 2, tc, m, warp, lane, s_mask, y, hs, bad);
    else
        wide_bits = encode_full_runs<DT, false>(in_bytes + j * kElemBytes, out_sm + j, out_smlo + j * 2, tc, m, warp, lane, s_mask, y, hs, bad);
    {
        uint2 ylow[8];
        const uint32_t lowmask4 = rep4((1u << m) - 1);
#pragma unroll
        for (int c = 0; c < 8; ++c) ylow[c] = make_uint2(y[c].x & lowmask4, y[c].y & lowmask4);
        pack_plane_any(m, smem_u32(s_low), j, N, ylow);
        if (DT == ENEC_FP16) pack_plane<3>(smem_u32(s_hi3), j, N, hs);
    }
    __syncthreads();
    // wide groups before each mask word and in the block: every warp scans the 32 mask words itself
    const uint32_t mask_word = s_mask[lane];
    uint32_t mask_incl = __popc(mask_word);
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, mask_incl, d);
        if (lane >= uint32_t(d)) mask_incl += t;
    }
    const uint32_t mask_excl = mask_incl - __popc(mask_word);
    const uint32_t wide_count = __shfl_sync(0xFFFFFFFFu, mask_incl, 31);
    fold_plane_out(smem_u32(s_low), N * uint32_t(m) / 8, out_low, tid);
    if (DT == ENEC_FP16) fold_plane_out(smem_u32(s_hi3), N * 3 / 8, out_smhi, tid);
    if (tid < kGroupsPerBlock / 8 / 16) reinterpret_cast<uint4*>(out_mask)[tid] = reinterpret_cast<const uint4*>(s_mask)[tid];
    if (hbits > 0) {
        // high bits of wide groups into shared memory, rank order, sixteen value bytes per group; narrow groups
        // store to a spare slot behind the buffer, so there is no branch
        const uint32_t hmask4 = rep4(0xFFu >> m);
        const uint32_t half_off = lane < 16 ? 0 : 8;
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            const uint32_t word = ((c * (kBlockElems / 8) + j) >> 9) & 31;
            const uint32_t rank = __shfl_sync(0xFFFFFFFFu, mask_excl, word) +
                                  __popc(__shfl_sync(0xFFFFFFFFu, mask_word, word) & lower);
            sts64(s_exp + (((wide_bits >> c) & 1) ? rank * 16 : kSpare) + half_off,
                  make_uint2((y[c].x >> m) & hmask4, (y[c].y >> m) & hmask4));
        }
        __syncthreads();
        // Algorithm 2 over each wide group, one group per thread, packed in place: record i lands below the
        // value bytes of every group that has not been read yet
        for (uint32_t base = 0; base < wide_count; base += kPackThreads) {
            const uint32_t i = base + tid;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (i < wide_count) v = lds128(s_exp + i * 16);
            __syncthreads();
            if (i < wide_count) pack_record_any(hbits, v, s_exp + i * 2 * hbits);
        }
        __syncthreads();
        for (uint32_t i = tid; i < wide_count * uint32_t(hbits); i += kPackThreads)
            reinterpret_cast<uint16_t*>(out_rec)[i] = uint16_t(lds16(s_exp + 2 * i));
    }
    __syncthreads();  // the shared planes and the mask are free for the next block
    return wide_count;
}

// ---------------------------------------------------------------------------------------------------
// enec_compress of a large tensor without a look-back.
//
// enec_pack_tensor_kernel: CTA c packs the blocks c, c + grid, ... with the tensor's (b, n, m) from the search.
// Block k's records go to byte k * 1024 * 2 (n - m) of the record section: the place they would have if all
// groups before were wide, which is never below their final place and always inside the capacity that
// enec_max_compressed_size asks for. The block's number of wide groups goes to its state word.
//
// enec_place_records_kernel: CTA v (numbered by a ticket, so that every CTA with a smaller number has started)
// owns a run of consecutive blocks. It sums the counts of the blocks before its run (their prefix, Sec. 5.1 /
// 5.4), then, a round of blocks at a time: reads their records into shared memory, says so in its progress word,
// waits until every block whose slot lies under the bytes it is about to write has been read by its owner (a
// block with a smaller number, hence a CTA with a smaller or the same number: waits only look down, and a
// CTA reads without waiting for anyone, so all waits end; they are bounded all the same), and writes the
// records and the table entries to their final places. The owner of the last block writes the header.
// ---------------------------------------------------------------------------------------------------
constexpr uint32_t kPlaceThreads = 256;
constexpr uint32_t kPlaceSmemBytes = 64 * 1024;  // records of the blocks in flight (a block has at most 14336 bytes)
constexpr uint32_t kPlaceMaxCtas = 1024;         // progress words behind the state words

__device__ __forceinline__ uint32_t record_slot_bytes(int hbits) { return kGroupsPerBlock * 2 * uint32_t(hbits); }

template <int DT>
__global__ void __launch_bounds__(kPackThreads, 4)
enec_pack_tensor_kernel(const EncodeJob job, int* status) {
    extern __shared__ __align__(16) uint8_t pack_smem[];
    __shared__ __align__(16) uint32_t s_mask[32];
    constexpr uint32_t kElemBytes = DT == ENEC_FP32 ? 4 : 2;
    pdl_launch_dependents();
    pdl_wait();  // nothing above touches global memory
    const uint32_t tid = threadIdx.x;
    if (blockIdx.x == 0) {  // the next call on this scratch area finds its control set zeroed
        job.ctl_next->hist[tid] = 0;
        if (tid == 0) { job.ctl_next->ticket = 0; job.ctl_next->hist_done = 0; job.ctl_next->reserved = 0; }
    }
    const int b = job.ctl->b, n = job.ctl->n, m = job.ctl->m;
    const Geometry g = make_geometry(job.count);
    const Sections sec = make_sections(DT, job.count, g, n, m, 0);
    const uint32_t slot = record_slot_bytes(n - m);
    const uint8_t* in_base = reinterpret_cast<const uint8_t*>(job.in);
    const uint8_t* in_end = in_base + job.count * kElemBytes;
    // CTA c takes blocks c and c + grid; after that blocks are handed out by the call's ticket, asked for two blocks
    // ahead (the CTAs of an SM do not progress equally), so that the answer and the block's L2 prefetch are never waited for
    __shared__ uint32_t s_next;
    uint32_t k = blockIdx.x, k_next = blockIdx.x + gridDim.x;
    for (; k < g.nblocks; ) {
        uint32_t asked = 0;
        if (tid == 0) asked = atomicAdd(&job.ctl->ticket, 1u);
        const bool last = k + 1 == g.nblocks;
        const uint32_t N = last ? g.tail_padded : kBlockElems;
        const uint32_t real = last ? g.tail_real : kBlockElems;
        const uint8_t* in_bytes = in_base + uint64_t(k) * kBlockElems * kElemBytes;
        uint8_t* out_smlo = job.out + sec.smlo + uint64_t(k) * kBlockElems * 2;  // fp32 only
        uint8_t* out_sm = job.out + sec.sm + uint64_t(k) * kBlockElems;
        uint8_t* out_low = job.out + sec.low + uint64_t(k) * (kBlockElems / 8) * uint32_t(m);
        uint8_t* out_smhi = job.out + sec.smhi + uint64_t(k) * (kBlockElems / 8) * 3;
        uint8_t* out_mask = job.out + sec.mask + uint64_t(k) * (kGroupsPerBlock / 8);
        uint8_t* out_rec = job.out + sec.high + uint64_t(k) * slot;
        if (k_next < g.nblocks) {   // the CTA's next block towards L2 (one 128-byte line per thread, two for fp32)
            const uint8_t* next = in_base + uint64_t(k_next) * kBlockElems * kElemBytes;
#pragma unroll
            for (uint32_t r = 0; r < kElemBytes / 2; ++r) {
                const uint8_t* line = next + (r * kPackThreads + tid) * 128;
                if (line < in_end) asm volatile("prefetch.global.L2 [%0];" ::"l"(line));
            }
        }
        uint32_t wide;
        if (real != kBlockElems)
            wide = pack_tail_block<DT>(in_bytes, N, real, b, n, m, out_sm, out_low, out_smhi, out_mask, out_smlo, out_rec, pack_smem);
        else
            wide = pack_full_block<DT>(in_bytes, b, n, m, out_sm, out_smlo, out_low, out_smhi, out_mask, out_rec, pack_smem, s_mask);
        if (tid == 0) {
            job.state[k] = wide;  // read by the next kernel
            s_next = 2 * gridDim.x + asked;
        }
        __syncthreads();
        k = k_next;
        k_next = s_next;
        __syncthreads();  // s_next is read before the next round's write
    }
    (void)status;
}

template <int DT>
__global__ void __launch_bounds__(kPlaceThreads, 2)
enec_place_records_kernel(const EncodeJob job, int* status) {
    extern __shared__ __align__(16) uint8_t place_smem[];
    __shared__ unsigned long long s_sum[kPlaceThreads / 32];
    __shared__ uint32_t s_virtual, s_failed, s_round_wide;
    __shared__ uint32_t s_warp_cnt[kPlaceThreads / 32], s_warp_len[kPlaceThreads / 32];
    __shared__ uint32_t s_cnt[kPlaceThreads], s_rec_before[kPlaceThreads], s_at[kPlaceThreads];
    pdl_launch_dependents();
    pdl_wait();  // nothing above touches global memory
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) { s_virtual = atomicAdd(&job.ctl->reserved, 1u); s_failed = 0; }
    const int n = job.ctl->n, m = job.ctl->m, hbits = n - m;  // in flight together with the ticket
    __syncthreads();
    const uint32_t v = s_virtual;
    const Geometry g = make_geometry(job.count);
    const Sections sec = make_sections(DT, job.count, g, n, m, 0);
    const uint32_t slot = record_slot_bytes(hbits);
    const uint32_t rec_bytes = 2 * uint32_t(hbits);
    const uint32_t per_cta = (g.nblocks + gridDim.x - 1) / gridDim.x;
    const uint32_t k0 = v * per_cta;
    const uint32_t k1 = k0 + per_cta < g.nblocks ? k0 + per_cta : g.nblocks;
    if (k0 >= g.nblocks) return;
    unsigned long long* progress = job.state + g.nblocks;  // one word per CTA of this kernel
    uint32_t* table = reinterpret_cast<uint32_t*>(job.out + sec.table);
    uint8_t* high = job.out + sec.high;
    // wide groups before the run: the counts are final (the pack kernel has ended), so every CTA adds them up
    // itself, eight loads per thread in flight
    uint32_t first_cnt = k0 + tid < k1 ? uint32_t(job.state[k0 + tid]) : 0u;  // the first round's counts, in flight with the sums
    unsigned long long before = 0;
    for (uint32_t base = 0; base < k0; base += kPlaceThreads * 8) {
        unsigned long long part[8];
#pragma unroll
        for (uint32_t u = 0; u < 8; ++u) {
            const uint32_t i = base + u * kPlaceThreads + tid;
            part[u] = i < k0 ? job.state[i] : 0ull;
        }
#pragma unroll
        for (uint32_t u = 0; u < 8; ++u) before += part[u];
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) before += __shfl_xor_sync(0xFFFFFFFFu, before, d);
    if (lane == 0) s_sum[warp] = before;
    __syncthreads();
    before = 0;
    for (uint32_t w = 0; w < kPlaceThreads / 32; ++w) before += s_sum[w];

    for (uint32_t a = k0; a < k1;) {
        // the blocks of this round: thread t looks at block a + t; the round takes the longest run of blocks from a
        // whose records fit the shared memory together (at least four always do)
        const uint32_t cand = k1 - a < kPlaceThreads ? k1 - a : kPlaceThreads;
        const uint32_t cnt = a == k0 ? first_cnt : tid < cand ? uint32_t(job.state[a + tid]) : 0u;
        const uint32_t len16 = uint32_t(align16(cnt * rec_bytes));
        uint32_t cnt_incl = cnt, len_incl = len16;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t c = __shfl_up_sync(0xFFFFFFFFu, cnt_incl, d), l = __shfl_up_sync(0xFFFFFFFFu, len_incl, d);
            if (lane >= uint32_t(d)) { cnt_incl += c; len_incl += l; }
        }
        if (lane == 31) { s_warp_cnt[warp] = cnt_incl; s_warp_len[warp] = len_incl; }
        __syncthreads();
        for (uint32_t w = 0; w < warp; ++w) { cnt_incl += s_warp_cnt[w]; len_incl += s_warp_len[w]; }
        const bool fits = tid < cand && len_incl <= kPlaceSmemBytes;
        s_cnt[tid] = cnt;
        s_rec_before[tid] = cnt_incl - cnt;
        s_at[tid] = len_incl - len16;
        const uint32_t take = uint32_t(__syncthreads_count(fits));   // blocks a .. a + take - 1
        if (tid == take - 1) s_round_wide = cnt_incl;
        // read: a warp per block
        for (uint32_t t = warp; t < take; t += kPlaceThreads / 32) {
            const uint32_t vecs = uint32_t(align16(s_cnt[t] * rec_bytes)) / 16;
            const uint4* src = reinterpret_cast<const uint4*>(high + uint64_t(a + t) * slot);
            uint4* dst = reinterpret_cast<uint4*>(place_smem + s_at[t]);
            for (uint32_t i = lane; i < vecs; i += 32) dst[i] = src[i];
        }
        __syncthreads();
        if (tid == 0) {
            __threadfence();
            st_relaxed_u64(&progress[v], kStatePrefix | epoch_bits(job.epoch) | (unsigned long long)(a + take - k0));
        }
        // every block whose slot starts under the end of what this round writes must have been read
        const unsigned long long write_end = (before + s_round_wide) * rec_bytes;
        uint32_t need_below = slot ? uint32_t((write_end + slot - 1) / slot) : 0;  // blocks 0 .. need_below - 1
        if (need_below > k0) need_below = k0;                                      // the CTA's own blocks are read
        if (warp == 0 && need_below > 0) {
            const uint32_t owners = (need_below + per_cta - 1) / per_cta;           // CTAs 0 .. owners - 1
            bool ok = true;
            for (uint32_t u = lane; u < owners; u += 32) {
                const uint32_t want = (need_below - u * per_cta) < per_cta ? need_below - u * per_cta : per_cta;
                uint32_t polls = 0;
                for (;;) {
                    const unsigned long long w = state_of_epoch(ld_relaxed_u64(&progress[u]), job.epoch);
                    if ((w >> 62) == 2 && uint32_t(w) >= want) break;
                    if (++polls > (1u << 20)) { ok = false; break; }
                    __nanosleep(200);
                }
            }
            if (!__all_sync(0xFFFFFFFFu, ok) && lane == 0) { s_failed = 1; report(status, ENEC_ERR_TIMEOUT); }
            __threadfence();
        }
        __syncthreads();
        if (s_failed) return;
        // write: a warp per block, two 16-bit halves per 32-bit store where the destination allows it
        for (uint32_t t = warp; t < take; t += kPlaceThreads / 32) {
            const unsigned long long p = before + s_rec_before[t];
            if (lane == 0) table[a + t] = uint32_t(p);
            if (p * rec_bytes == uint64_t(a + t) * slot) continue;  // the records are in place already
            const uint32_t halves = s_cnt[t] * uint32_t(hbits);
            uint16_t* dst = reinterpret_cast<uint16_t*>(high + p * rec_bytes);
            const uint16_t* src = reinterpret_cast<const uint16_t*>(place_smem + s_at[t]);
            const uint32_t odd = (reinterpret_cast<uintptr_t>(dst) >> 1) & 1;  // a leading half before the first aligned word
            if (odd && lane == 0 && halves > 0) dst[0] = src[0];
            const uint32_t words = halves > odd ? (halves - odd) / 2 : 0;
            uint32_t* dst32 = reinterpret_cast<uint32_t*>(dst + odd);
            for (uint32_t i = lane; i < words; i += 32)
                dst32[i] = uint32_t(src[odd + 2 * i]) | (uint32_t(src[odd + 2 * i + 1]) << 16);
            if (lane == 0 && halves > odd && ((halves - odd) & 1)) dst[halves - 1] = src[halves - 1];
        }
        before += s_round_wide;
        a += take;
        __syncthreads();  // the shared memory is free for the next round
    }
    if (k1 == g.nblocks && tid == 0) {
        const uint32_t a_total = uint32_t(before);
        const uint64_t high_bytes = uint64_t(a_total) * rec_bytes;
        const uint64_t total = sec.high + align16(high_bytes);
        Header hd;
        hd.magic = kMagic;
        hd.version = kVersion;
        hd.dtype = DT;
        hd.variant = 0;
        hd.count = job.count;
        hd.block = kBlockElems;
        hd.b = uint8_t(job.ctl->b); hd.n = uint8_t(n); hd.m = uint8_t(m); hd.L = kGroupElems;
        hd.nblocks = g.nblocks;
        hd.total_groups = g.total_groups;
        hd.a_total = a_total;
        hd.pad1 = 0;
        hd.total_bytes = total;
        hd.pad2[0] = hd.pad2[1] = 0;
        *reinterpret_cast<Header*>(job.out) = hd;
        table[g.nblocks] = a_total;
        for (uint64_t i = uint64_t(g.nblocks) + 1; i < align16(4 * (uint64_t(g.nblocks) + 1)) / 4; ++i) table[i] = 0;
        for (uint64_t q = high_bytes; q < align16(high_bytes); q += 2) *reinterpret_cast<uint16_t*>(high + q) = 0;
        if (job.out_size) *job.out_size = total;
    }
}

}  // namespace enec
