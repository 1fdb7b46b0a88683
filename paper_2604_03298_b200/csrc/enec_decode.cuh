// Decompression kernel: unpack + reconstruct (Sec. 5.1 decompression flow).
//
// One persistent CTA per resident slot. A loader warp stages each 16384-element block's compressed
// segments (group mask, low plane, fp16 sign/mantissa-high plane, sign/mantissa bytes, wide-group
// records) into shared memory with bulk asynchronous copies completing on an mbarrier. Eight consumer
// warps first turn the block's mask into per-group record ranks (popcount prefix) and expand the staged
// records to one byte per value, meet at a named barrier, then undo Algorithm 2 on packed bytes (four
// elements per 32-bit operation), merge the high bits of wide groups, apply the inverse transform of
// Sec. 5.3 and write 16-byte coalesced stores. Full blocks whose records all fit in the stage take a
// branch-free body; tail blocks and overfull blocks take a general one. Every wait is bounded and ends
// in an error status, never a hang.
#pragma once

#include "enec_common.cuh"

namespace enec {

constexpr int kConsumerWarps = 8;
constexpr int kDecodeThreads = (kConsumerWarps + 1) * 32;
constexpr int kStages = 2;
constexpr uint32_t kDecodeSmemBytes = 75 * 1024;  // three CTAs per SM
constexpr uint32_t kStageMetaBytes = 128;
constexpr uint32_t kStageBytes = ((kDecodeSmemBytes - 128) / kStages) & ~15u;
constexpr uint32_t kNotWide = 0xFFFFu;            // rank-array entry of a group stored with m bits

// ---------------------------------------------------------------------------------------------------
// Inverse of Algorithm 2 on packed bytes.
//
// Algorithm 2 folds the upper half of the lanes onto the lower half (shifted by the current width) until
// a lane holds at least 8 bits, peels the low byte of every lane ("normalised bytes"), and repeats on
// the residues; the final fold interleaves the first and second half of the normalised bytes. For an
// input of N elements of A bits, element e ends in lane (e mod N_l) of level l at a bit offset that
// depends only on (e div N_l), so a thread that owns eight consecutive lanes j..j+7 of the N/8 lanes of
// the deepest level owns, at every level, whole runs of eight consecutive lanes: it can rebuild the 64
// elements {j + c N/8 + i : c, i < 8} from a few 16-byte shared-memory loads with shifts and masks whose
// amounts are compile-time constants.
// ---------------------------------------------------------------------------------------------------
// bits [s, s + w) of the 16-bit lanes (v | r << 8), four lanes per register, one lane per byte
__device__ __forceinline__ uint32_t extract_bits(uint32_t v, uint32_t r, int s, int w) {
    const uint32_t m = (1u << w) - 1;
    if (s + w <= 8) return (v >> s) & rep4(m);
    if (s >= 8) return (r >> (s - 8)) & rep4(m);
    const uint32_t lo = 0xFFu >> s;
    return ((v >> s) & rep4(lo)) | ((r << (8 - s)) & rep4(m & ~lo));
}

// Normalised bytes nb[i0 .. i0+7] (i0 a multiple of 8) of a plane in shared memory whose final fold has
// half-length thalf (a multiple of 8): nb[i] sits at byte 2i (i < thalf) or 2(i - thalf) + 1.
__device__ __forceinline__ uint2 load_octet(uint32_t S, uint32_t i0, uint32_t thalf) {
    const bool odd = i0 >= thalf;
    const uint32_t pos = 2 * (odd ? i0 - thalf : i0);
    const uint4 v = lds128(S + pos);
    const uint32_t sel = odd ? 0x7531u : 0x6420u;
    return make_uint2(prmt(v.x, v.y, sel), prmt(v.z, v.w, sel));
}

// out[e] (e < 2^LOG_UNITS) = packed W_IN-bit values of the eight elements j + e * n8 + (0..7) of this level.
template <int W_IN, int LOG_UNITS>
__device__ __forceinline__ void unpack_plane_level(uint32_t S, uint32_t nb_off, uint32_t j, uint32_t n8,
                                                   uint32_t thalf, uint2 (&out)[1 << LOG_UNITS]) {
    constexpr int F = folds_for(W_IN);
    static_assert(F <= LOG_UNITS, "lane runs must stay whole");
    constexpr int W = W_IN << F;
    constexpr int LOG_LANES = LOG_UNITS - F;
    constexpr int NL = 1 << LOG_LANES;
    constexpr int RES = W - 8;
    uint2 V[NL];
    uint2 R[NL];
#pragma unroll
    for (int c = 0; c < NL; ++c) {
        V[c] = load_octet(S, nb_off + j + c * n8, thalf);
        R[c] = make_uint2(0, 0);
    }
    if constexpr (RES > 0) unpack_plane_level<RES, LOG_LANES>(S, nb_off + NL * n8, j, n8, thalf, R);
#pragma unroll
    for (int e = 0; e < (1 << LOG_UNITS); ++e) {
        const int c = e & (NL - 1);
        const int s = W_IN * bitrev(e >> LOG_LANES, F);
        out[e].x = extract_bits(V[c].x, R[c].x, s, W_IN);
        out[e].y = extract_bits(V[c].y, R[c].y, s, W_IN);
    }
}

// Eight runs of eight A-bit values: y[c] = elements j + c * N/8 + (0..7) of a plane of N elements.
template <int A>
__device__ __forceinline__ void unpack_plane(uint32_t S, uint32_t j, uint32_t N, uint2 (&y)[8]) {
    unpack_plane_level<A, 3>(S, 0, j, N >> 3, (N * A) >> 4, y);
}

// One element of a plane of N >= 16 elements of `a` bits, bit by bit (used only for blocks shorter than
// 128 elements, where lane runs of eight do not exist).
template <class LoadByte>
__device__ inline uint32_t unpack_scalar(LoadByte load_byte, uint32_t N, int a, uint32_t e) {
    const uint32_t thalf = (N * uint32_t(a)) >> 4;
    uint32_t value = 0;
    for (int q = 0; q < a; ++q) {
        int width = a;
        uint32_t length = N, idx = e, off = 0;
        int p = q;
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
        const uint32_t pos = i < thalf ? 2 * i : 2 * (i - thalf) + 1;
        value |= ((load_byte(pos) >> p) & 1u) << q;
    }
    return value;
}

// ---- wide-group records: Algorithm 2 with N = 16, H bits per value, 2H bytes --------------------------
// Same scheme with runs of two lanes (N/8 = 2). q[i] = 16-bit word i of the record.
template <int H>
__device__ __forceinline__ uint32_t record_pair(const uint32_t (&q)[H], int i0) {
    // normalised bytes nb[i0], nb[i0 + 1] of a record: nb[i] at byte 2i (i < H) or 2(i - H) + 1
    const int pa = i0 < H ? 2 * i0 : 2 * (i0 - H) + 1;
    const int pb = (i0 + 1) < H ? 2 * (i0 + 1) : 2 * (i0 + 1 - H) + 1;
    const uint32_t sel = uint32_t(pa & 1) | (uint32_t(4 + (pb & 1)) << 4) | 0x2200u;  // bytes 2, 3 of q are zero
    return prmt(q[pa >> 1], q[pb >> 1], sel);
}

template <int H, int W_IN, int LOG_UNITS>
__device__ __forceinline__ void unpack_record_level(const uint32_t (&q)[H], int nb_off, uint32_t (&out)[1 << LOG_UNITS]) {
    constexpr int F = folds_for(W_IN);
    static_assert(F <= LOG_UNITS, "lane runs must stay whole");
    constexpr int W = W_IN << F;
    constexpr int LOG_LANES = LOG_UNITS - F;
    constexpr int NL = 1 << LOG_LANES;
    constexpr int RES = W - 8;
    uint32_t V[NL];
    uint32_t R[NL];
#pragma unroll
    for (int c = 0; c < NL; ++c) {
        V[c] = record_pair<H>(q, nb_off + 2 * c);
        R[c] = 0;
    }
    if constexpr (RES > 0) unpack_record_level<H, RES, LOG_LANES>(q, nb_off + 2 * NL, R);
#pragma unroll
    for (int e = 0; e < (1 << LOG_UNITS); ++e) {
        const int c = e & (NL - 1);
        const int s = W_IN * bitrev(e >> LOG_LANES, F);
        out[e] = extract_bits(V[c], R[c], s, W_IN);
    }
}

// The sixteen H-bit values of a record, one per byte, element order.
template <int H, class LoadWord>
__device__ __forceinline__ uint4 unpack_record(LoadWord load_word) {
    uint32_t q[H];
#pragma unroll
    for (int i = 0; i < H; ++i) q[i] = load_word(i);  // 16-bit word i of the record
    uint32_t pr[8];  // pr[e] = elements 2e, 2e + 1
    unpack_record_level<H, H, 3>(q, 0, pr);
    return make_uint4(prmt(pr[0], pr[1], 0x5410u), prmt(pr[2], pr[3], 0x5410u), prmt(pr[4], pr[5], 0x5410u),
                      prmt(pr[6], pr[7], 0x5410u));
}

// ---------------------------------------------------------------------------------------------------
// Per-tensor context derived from the stream header.
struct DecodeJob {
    const uint8_t* in;
    uint16_t* out;
    uint64_t count;
    uint64_t in_size;
};

struct JobCtx {
    const uint8_t* in;
    uint16_t* out;
    uint32_t nblocks, tail_real, tail_padded;
    uint32_t a_total;
    int b, n, m;
    uint64_t off_table, off_mask, off_low, off_smhi, off_sm, off_smlo, off_high, total;
    bool blockwise;  // parameters and offsets per block, from the block table (header byte 7 = 2)
};

// Reads and validates the header. Returns 0 or an enec_status.
template <int DT, bool MAPPED = false>
__device__ inline int load_job(const DecodeJob& job, JobCtx& c, bool blockwise = false) {
    if (job.in_size < kHeaderBytes + 16) return ENEC_ERR_BAD_STREAM;
    const Header h = *reinterpret_cast<const Header*>(job.in);
    if (h.magic != kMagic || h.version != kVersion || h.dtype != DT || h.count != job.count ||
        h.block != kBlockElems || h.L != kGroupElems)
        return ENEC_ERR_BAD_STREAM;
    constexpr int E = exp_bits(DT);
    if (h.variant != (blockwise ? 2 : MAPPED ? 1 : 0)) return ENEC_ERR_BAD_STREAM;
    if (blockwise ? (h.b | h.n | h.m) != 0 : (h.n < 1 || h.n > E || h.m < 1 || h.m > h.n || h.b >= (1 << E)))
        return ENEC_ERR_BAD_STREAM;
    const Geometry g = make_geometry(job.count);
    if (h.nblocks != g.nblocks || h.total_groups != g.total_groups || h.a_total > g.total_groups)
        return ENEC_ERR_BAD_STREAM;
    Sections s;
    if (blockwise) {
        // the block table's last entry holds the sums that fix the sizes of the two variable sections
        const uint64_t table_bytes = 16 * (uint64_t(g.nblocks) + 1);
        if (job.in_size < kHeaderBytes + table_bytes) return ENEC_ERR_BAD_STREAM;
        const uint4 totals = *reinterpret_cast<const uint4*>(job.in + kHeaderBytes + 16 * uint64_t(g.nblocks));
        uint64_t low_bytes = 0;
        if (g.nblocks) {
            const uint32_t m_tail = (*reinterpret_cast<const uint32_t*>(job.in + kHeaderBytes + 16 * uint64_t(g.nblocks - 1)) >> 16) & 0xFFu;
            if (totals.y < m_tail || totals.y > 8ull * g.nblocks) return ENEC_ERR_BAD_STREAM;
            low_bytes = uint64_t(totals.y - m_tail) * (kBlockElems / 8) + uint64_t(g.tail_padded) * m_tail / 8;
        }
        const uint64_t high_bytes = uint64_t(totals.z) | (uint64_t(totals.w) << 32);
        if (totals.x != 0 || high_bytes > uint64_t(g.total_groups) * 14) return ENEC_ERR_BAD_STREAM;
        s.unmap = kHeaderBytes;
        s.table = kHeaderBytes;
        s.mask = s.table + align16(table_bytes);
        s.low = s.mask + align16((uint64_t(g.total_groups) + 7) / 8);
        s.smhi = s.low + align16(low_bytes);
        s.sm = s.smhi + (DT == ENEC_FP16 ? align16(g.padded_count * 3 / 8) : 0);
        s.smlo = s.sm + align16(job.count);
        s.high = s.smlo + (DT == ENEC_FP32 ? align16(job.count * 2) : 0);
        s.total = s.high + align16(high_bytes);
    } else {
        s = make_sections(DT, job.count, g, h.n, h.m, h.a_total, MAPPED);
    }
    if (h.total_bytes != s.total || job.in_size < s.total) return ENEC_ERR_BAD_STREAM;
    c.in = job.in;
    c.out = job.out;
    c.nblocks = g.nblocks;
    c.tail_real = g.tail_real;
    c.tail_padded = g.tail_padded;
    c.a_total = h.a_total;
    c.b = h.b; c.n = h.n; c.m = h.m;
    c.off_table = s.table; c.off_mask = s.mask; c.off_low = s.low; c.off_smhi = s.smhi; c.off_sm = s.sm;
    c.off_smlo = s.smlo; c.off_high = s.high; c.total = s.total;
    c.blockwise = blockwise;
    return 0;
}

// Shared-memory layout of one pipeline stage (offsets from the stage base; all multiples of 16).
//   descriptor | mask | rank array | low plane | fp16 sm-hi plane | sm bytes | raw records | expanded records
// rank array: one u16 per group = rank of the group's record inside the block, or kNotWide.
// expanded records: sixteen bytes per wide group (its high bits, one element per byte), rank order, and
// one more slot at index cap that the rank entries of narrow groups point to in blocks that fit.
// cap = records per block that fit; records beyond it are read from global memory by the consumers.
// nibble: the expanded records take eight bytes each (n - m <= 4: byte j of a record's two words holds element j in
// its low and element j + 4 in its high half), which lets full blocks with many wide groups still fit.
struct StageLayout {
    uint32_t mask, rank, low, smhi, sm, raw, expanded, cap, bytes;
};
constexpr uint32_t kStageRankTable = kStageBytes - kRankTableBytes;  // where a stage keeps a stream's rank table
// mapped: the stage also holds the stream's rank -> exponent table (its last 256 bytes).
__host__ __device__ inline StageLayout make_stage_layout(int dt, int m, int hbits, bool mapped = false, bool nibble = false) {
    StageLayout L;
    const uint32_t usable = mapped ? kStageRankTable : kStageBytes;
    L.mask = kStageMetaBytes;
    L.rank = L.mask + kGroupsPerBlock / 8;
    L.low = L.rank + kGroupsPerBlock * 2;
    L.smhi = L.low + kBlockElems * uint32_t(m) / 8;
    L.sm = L.smhi + (dt == ENEC_FP16 ? kBlockElems * 3 / 8 : 0);
    L.raw = L.sm + kBlockElems;  // at most 35072 (m = 8, or fp16 with m = 5), so a stage always has room
    const uint32_t expanded_size = nibble ? 8 : 16;
    uint32_t cap = hbits > 0 ? (usable - L.raw - 64) / (uint32_t(2 * hbits) + expanded_size) : 0;
    if (cap > kGroupsPerBlock) cap = kGroupsPerBlock;
    L.cap = cap;
    L.expanded = L.raw + uint32_t(align16(uint64_t(cap) * 2 * hbits + 32));
    L.bytes = L.expanded + (cap + 1) * expanded_size;
    return L;
}
static_assert(kStageMetaBytes + kGroupsPerBlock / 8 + kGroupsPerBlock * 2 + 2 * kBlockElems + 64 + kRankTableBytes <= kStageBytes,
              "the fixed part of the widest block fits a stage");

struct RunCtx {
    uint32_t sm;          // shared address: sign/mantissa bytes of the block
    uint32_t rank;        // shared address: rank array
    uint32_t expanded;    // shared address: expanded records
    uint32_t cap;         // records expanded in shared memory
    const uint8_t* high;  // global: first record of the block
    uint16_t* out;        // global: first element of the block (fp32: four bytes per element)
    const uint16_t* lo;   // global, fp32 only: mantissa bits 15..0 of the block's elements
    uint32_t real;        // real elements in the block
    uint32_t c4_or_h, fix, s4, b4;  // packed transform constants
    uint32_t c4;                    // rep4(b + 2^(n-1)) when that sum fits a byte
    int n;
};

// The eight-byte form of the expanded records exists in the fp16 kernel only: fp16 weights have five exponent
// bits and (n, m) = (5, 3), so half of their groups can be wide, more than a stage holds in the sixteen-byte form;
// the bf16 and fp32 kernels, whose blocks fit, carry none of its code (measured: with it their one-stream rate
// fell by 1.5 to 4 %, from code layout alone).
template <int DT, bool MAPPED>
constexpr bool kNibbleForm = DT == ENEC_FP16 && !MAPPED;

// Whether x = (b + 2^(n-1)) - (y ^ 2^(n-1)) can be taken as one subtraction per word (what the branch-free bodies do).
template <int DT>
__host__ __device__ inline bool plain_subtraction(uint32_t b, uint32_t n) {
    return DT == ENEC_FP16 || n == 8 || b + (1u << (n - 1)) <= 255;
}

// Inverse transform on four packed bytes: x = (b - sext_n(y)) mod 2^E  (Sec. 5.3).
// sext_n(y) = (y ^ s) - s with s = 2^(n-1), so x = (b + s) - (y ^ s) per byte.
template <int DT>
__device__ __forceinline__ uint32_t inverse_transform4(const RunCtx& r, uint32_t y) {
    constexpr uint32_t Hm = 0x80808080u;
    uint32_t x;
    if (r.n < 8) {
        // u = y ^ s < 128: ((c | 0x80) - u) never borrows across bytes; bit 7 is repaired by `fix`
        const uint32_t u = y ^ r.s4;
        x = (r.c4_or_h - u) ^ r.fix;
    } else {
        // n = 8: plain bytewise b - y (mod 256)
        x = ((r.b4 | Hm) - (y & ~Hm)) ^ ((r.b4 ^ ~y) & Hm);
    }
    if (DT == ENEC_FP16) x &= 0x1F1F1F1Fu;
    return x;
}

// Four table look-ups (frequency-rank variant): byte i of the result is the exponent of the rank in byte i of y.
__device__ __forceinline__ uint32_t table4(uint32_t table, uint32_t y) {
    const uint32_t r0 = lds8(table + (y & 0xFFu)), r1 = lds8(table + ((y >> 8) & 0xFFu));
    const uint32_t r2 = lds8(table + ((y >> 16) & 0xFFu)), r3 = lds8(table + (y >> 24));
    return r0 | (r1 << 8) | (r2 << 16) | (r3 << 24);
}

// High bits of eight elements of a wide group whose record was not expanded in shared memory.
template <int HB>
__device__ __noinline__ uint2 record_half_from_global(const uint8_t* rp, uint32_t second_half) {
    const uint4 v = unpack_record<HB>([&](int i) { return uint32_t(*reinterpret_cast<const uint16_t*>(rp + 2 * i)); });
    return second_half ? make_uint2(v.z, v.w) : make_uint2(v.x, v.y);
}

// fp32: joins the high halves of eight values (w, element order) with their low halves and stores 32 bytes:
// as one 32-byte store where the address allows it, so that consecutive lanes fill whole sectors.
__device__ __forceinline__ void store_fp32_run(uint32_t* out, uint4 w, uint4 lo) {
    const uint4 a = make_uint4(prmt(lo.x, w.x, 0x5410u), prmt(lo.x, w.x, 0x7632u), prmt(lo.y, w.y, 0x5410u),
                      prmt(lo.y, w.y, 0x7632u));
    const uint4 b = make_uint4(prmt(lo.z, w.z, 0x5410u), prmt(lo.z, w.z, 0x7632u), prmt(lo.w, w.w, 0x5410u),
                      prmt(lo.w, w.w, 0x7632u));
    if ((reinterpret_cast<uintptr_t>(out) & 31) == 0) {
        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(out), "r"(a.x), "r"(a.y), "r"(a.z),
                     "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w)
                     : "memory");
    } else {
        uint4* o = reinterpret_cast<uint4*>(out);
        o[0] = a;
        o[1] = b;
    }
}

// Finishes eight consecutive elements e0 .. e0+7 of a block: high bits of wide groups, inverse transform,
// rejoin with sign/mantissa, store.
template <int DT, int M, int HB, bool MAPPED = false>
__device__ __forceinline__ void finish_run(const RunCtx& r, uint2 y, uint2 hs, uint32_t e0, bool active) {
    if constexpr (HB > 0) {
        const uint32_t rk = lds16(r.rank + ((e0 >> 4) << 1));
        if (rk != kNotWide) {
            uint2 hi;
            if (rk < r.cap) hi = lds64(r.expanded + rk * 16 + (e0 & 8));
            else hi = record_half_from_global<HB>(r.high + rk * (2 * HB), e0 & 8);
            y.x |= hi.x << M;
            y.y |= hi.y << M;
        }
    }
    // frequency-rank variant: r.c4 is the shared address of the stage's rank -> exponent table
    const uint32_t x0 = MAPPED ? table4(r.c4, y.x) : inverse_transform4<DT>(r, y.x);
    const uint32_t x1 = MAPPED ? table4(r.c4, y.y) : inverse_transform4<DT>(r, y.y);
    const uint2 smv = lds64(r.sm + e0);
    uint32_t lo0, lo1, hi0, hi1;
    if (DT != ENEC_FP16) {
        // word = sign << 15 | x << 7 | mant7 ; sm byte = sign << 7 | mant7 (fp32: the high half of the value)
        hi0 = (smv.x & 0x80808080u) | ((x0 >> 1) & 0x7F7F7F7Fu);
        hi1 = (smv.y & 0x80808080u) | ((x1 >> 1) & 0x7F7F7F7Fu);
        lo0 = ((x0 << 7) & 0x80808080u) | (smv.x & 0x7F7F7F7Fu);
        lo1 = ((x1 << 7) & 0x80808080u) | (smv.y & 0x7F7F7F7Fu);
    } else {
        // word = sign << 15 | x << 10 | mant10 ; sm byte = mant[7:0] ; hs = sign << 2 | mant[9:8]
        hi0 = ((hs.x << 5) & 0x80808080u) | (x0 << 2) | (hs.x & 0x03030303u);
        hi1 = ((hs.y << 5) & 0x80808080u) | (x1 << 2) | (hs.y & 0x03030303u);
        lo0 = smv.x;
        lo1 = smv.y;
    }
    uint4 w;
    w.x = prmt(lo0, hi0, 0x5140u);
    w.y = prmt(lo0, hi0, 0x7362u);
    w.z = prmt(lo1, hi1, 0x5140u);
    w.w = prmt(lo1, hi1, 0x7362u);
    if (!active) return;
    if constexpr (DT == ENEC_FP32) {
        uint32_t* out32 = reinterpret_cast<uint32_t*>(r.out) + e0;
        if (e0 + 8 <= r.real) {
            store_fp32_run(out32, w, __ldg(reinterpret_cast<const uint4*>(r.lo + e0)));
        } else if (e0 < r.real) {
            for (uint32_t i = 0; e0 + i < r.real; ++i) {
                const uint32_t pair = (i >> 1) == 0 ? w.x : (i >> 1) == 1 ? w.y : (i >> 1) == 2 ? w.z : w.w;
                out32[i] = ((pair >> (16 * (i & 1))) << 16) | r.lo[e0 + i];
            }
        }
        return;
    }
    if (e0 + 8 <= r.real) {
        *reinterpret_cast<uint4*>(r.out + e0) = w;
    } else if (e0 < r.real) {
        for (uint32_t i = 0; e0 + i < r.real; ++i) {
            const uint32_t pair = (i >> 1) == 0 ? w.x : (i >> 1) == 1 ? w.y : (i >> 1) == 2 ? w.z : w.w;
            r.out[e0 + i] = uint16_t(pair >> (16 * (i & 1)));
        }
    }
}

// One block, all consumer threads. tid = 0..255. N = padded block length.
template <int DT, int M, int HB, bool MAPPED = false>
__device__ __forceinline__ void decode_block(const RunCtx& r, uint32_t s_low, uint32_t s_smhi, uint32_t N,
                                             uint32_t tid) {
    if (N >= 128) {
        const uint32_t items = N >> 6;
        const uint32_t n8 = N >> 3;
        for (uint32_t base = 0; base < items; base += kConsumerWarps * 32) {
            if (base + (tid & ~31u) >= items) break;  // whole warp idle
            const bool active = base + tid < items;
            const uint32_t j = active ? 8 * (base + tid) : 0;
            uint2 y[8];
            uint2 hs[8];
            unpack_plane<M>(s_low, j, N, y);
            if (DT == ENEC_FP16) unpack_plane<3>(s_smhi, j, N, hs);
#pragma unroll
            for (int c = 0; c < 8; ++c)
                finish_run<DT, M, HB, MAPPED>(r, y[c], DT == ENEC_FP16 ? hs[c] : make_uint2(0, 0), c * n8 + j, active);
        }
    } else {
        // short tail block (16, 32 or 64 elements): one run of eight per thread, values rebuilt bit by bit
        if (tid * 8 >= N) return;
        const uint32_t e0 = tid * 8;
        uint32_t yb[2] = {0, 0}, hb[2] = {0, 0};
        for (uint32_t i = 0; i < 8; ++i) {
            yb[i >> 2] |= unpack_scalar([&](uint32_t p) { return lds8(s_low + p); }, N, M, e0 + i) << (8 * (i & 3));
            if (DT == ENEC_FP16)
                hb[i >> 2] |= unpack_scalar([&](uint32_t p) { return lds8(s_smhi + p); }, N, 3, e0 + i) << (8 * (i & 3));
        }
        finish_run<DT, M, HB, MAPPED>(r, make_uint2(yb[0], yb[1]), make_uint2(hb[0], hb[1]), e0, true);
    }
}

// Branch-free body for a full block (16384 real elements) whose records are all expanded in shared memory.
// The expanded high bits are stored with the sign position 2^(n-1) already flipped, and the rank entry of
// a narrow group points to a slot that holds just that flip, so low + (slot << M) is y ^ 2^(n-1) for every
// run. bf16 with n < 8 uses it only when b + 2^(n-1) <= 255: then x = (b + 2^(n-1)) - (y ^ 2^(n-1)) never
// borrows across bytes for a stream that came from real data (x is a field value), and a plain
// subtraction serves; other bf16 tensors with n < 8 take the general body.
// The frequency-rank variant (MAPPED) has no sign position: nothing is flipped, the slot of narrow groups holds
// zeros, and the exponent comes from the stage's rank table (shared address in r.c4) instead of the subtraction.
// tid = 0..255; thread tid owns the runs c * 2048 + 8 tid (c < 8).
// NIBBLE: the expanded records are in the eight-byte form (see StageLayout).
template <int DT, int M, int HB, bool MAPPED = false, bool NIBBLE = false>
__device__ __forceinline__ void decode_full_block(const RunCtx& r, uint32_t s_low, uint32_t s_smhi, uint32_t tid) {
    constexpr int n = M + HB;
    constexpr uint32_t Hm = 0x80808080u;
    const uint32_t rank_addr = r.rank + (tid >> 1) * 2;
    const uint32_t exp_addr = r.expanded + (tid & 1) * (NIBBLE ? 4 : 8);
    const uint32_t sm_addr = r.sm + 8 * tid;
    uint4* out = reinterpret_cast<uint4*>(r.out + 8 * tid);
    [[maybe_unused]] uint32_t* out32 = reinterpret_cast<uint32_t*>(r.out) + 8 * tid;
    [[maybe_unused]] const uint4* lo_plane = reinterpret_cast<const uint4*>(r.lo + 8 * tid);
    // Shared-memory loads are issued in batches ahead of the arithmetic that uses them (the load helpers
    // keep program order): all rank entries first, then the planes, then per half of the runs the
    // expanded high bits and the sign/mantissa bytes.
    uint32_t rk[8];
    if constexpr (HB > 0) {
#pragma unroll
        for (int c = 0; c < 8; ++c) rk[c] = lds16(rank_addr + c * (kBlockElems / 8 / 16) * 2);
    }
    uint2 y[8];
    uint2 hs[8];
    unpack_plane<M>(s_low, 8 * tid, kBlockElems, y);
    if (DT == ENEC_FP16) unpack_plane<3>(s_smhi, 8 * tid, kBlockElems, hs);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        uint2 hi[4];
        uint2 smv[4];
        [[maybe_unused]] uint4 lov[4];
        if constexpr (DT == ENEC_FP32) {
#pragma unroll
            for (int q = 0; q < 4; ++q) lov[q] = __ldg(lo_plane + (4 * h + q) * (kBlockElems / 8 / 8));
        }
        if constexpr (HB > 0) {
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if constexpr (NIBBLE) {
                    const uint32_t w = lds32(exp_addr + rk[4 * h + q] * 8);
                    hi[q] = make_uint2(w & 0x0F0F0F0Fu, (w >> 4) & 0x0F0F0F0Fu);
                } else {
                    hi[q] = lds64(exp_addr + rk[4 * h + q] * 16);
                }
            }
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) smv[q] = lds64(sm_addr + (4 * h + q) * (kBlockElems / 8));
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int c = 4 * h + q;
            uint2 v = y[c];
            if constexpr (HB > 0) {
                v.x += hi[q].x << M;  // disjoint bits
                v.y += hi[q].y << M;
            } else if constexpr (!MAPPED) {
                v.x ^= r.s4;
                v.y ^= r.s4;
            }
            uint32_t x0, x1;
            if constexpr (MAPPED) {
                x0 = table4(r.c4, v.x);
                x1 = table4(r.c4, v.y);
            } else if constexpr (DT == ENEC_FP16) {
                // b + 2^(n-1) < 128: the guard bit absorbs any borrow and is masked away with the field
                x0 = r.c4_or_h - v.x;
                x1 = r.c4_or_h - v.y;
            } else if constexpr (n < 8) {
                x0 = r.c4 - v.x;
                x1 = r.c4 - v.y;
            } else {  // n = 8: bytewise (b + 128) - (y ^ 128) modulo 256
                x0 = (r.c4_or_h - (v.x & ~Hm)) ^ ((r.c4 ^ ~v.x) & Hm);
                x1 = (r.c4_or_h - (v.y & ~Hm)) ^ ((r.c4 ^ ~v.y) & Hm);
            }
            uint32_t lo0, lo1, hi0, hi1;
            if (DT != ENEC_FP16) {
                hi0 = (smv[q].x & Hm) | ((x0 >> 1) & ~Hm);
                hi1 = (smv[q].y & Hm) | ((x1 >> 1) & ~Hm);
                lo0 = ((x0 << 7) & Hm) | (smv[q].x & ~Hm);
                lo1 = ((x1 << 7) & Hm) | (smv[q].y & ~Hm);
            } else {
                x0 &= 0x1F1F1F1Fu;
                x1 &= 0x1F1F1F1Fu;
                hi0 = ((hs[c].x << 5) & Hm) | (x0 << 2) | (hs[c].x & 0x03030303u);
                hi1 = ((hs[c].y << 5) & Hm) | (x1 << 2) | (hs[c].y & 0x03030303u);
                lo0 = smv[q].x;
                lo1 = smv[q].y;
            }
            uint4 w;
            w.x = prmt(lo0, hi0, 0x5140u);
            w.y = prmt(lo0, hi0, 0x7362u);
            w.z = prmt(lo1, hi1, 0x5140u);
            w.w = prmt(lo1, hi1, 0x7362u);
            if constexpr (DT == ENEC_FP32) store_fp32_run(out32 + c * (kBlockElems / 8), w, lov[q]);
            else out[c * (kBlockElems / 8 / 8)] = w;
        }
    }
}

// Consumer preparation of a block, all 256 consumer threads: per-group record ranks from the mask
// (popcount prefix; a narrow group gets `narrow_entry`). Returns the number of wide groups the mask holds.
__device__ __forceinline__ uint32_t build_rank_array(uint32_t s_mask, uint32_t s_rank, uint32_t N, uint32_t tid,
                                                     uint32_t narrow_entry) {
    const uint32_t lane = tid & 31;
    const uint32_t groups = N >> 4;
    uint32_t mw = 0;  // every warp holds all 32 mask words, one per lane
    if (lane * 32 < groups) {
        mw = lds32(s_mask + 4 * lane);
        if (groups - lane * 32 < 32) mw &= (1u << (groups - lane * 32)) - 1;
    }
    uint32_t incl = __popc(mw);
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= uint32_t(d)) incl += t;
    }
    // thread tid writes the entries of groups 4 tid .. 4 tid + 3 (word tid / 8, bits 4 (tid % 8) ..)
    const uint32_t word = tid >> 3, bit0 = (tid & 7) * 4;
    const uint32_t w = __shfl_sync(0xFFFFFFFFu, mw, word);
    uint32_t run = __shfl_sync(0xFFFFFFFFu, incl - __popc(mw), word) + __popc(w & ((1u << bit0) - 1));
    const uint32_t bits = (w >> bit0) & 15;
    const uint32_t e0 = bits & 1 ? run : narrow_entry;
    run += bits & 1;
    const uint32_t e1 = bits & 2 ? run : narrow_entry;
    run += (bits >> 1) & 1;
    const uint32_t e2 = bits & 4 ? run : narrow_entry;
    run += (bits >> 2) & 1;
    const uint32_t e3 = bits & 8 ? run : narrow_entry;
    if (4 * tid < groups) sts64(s_rank + 8 * tid, make_uint2(e0 | (e1 << 16), e2 | (e3 << 16)));
    return __shfl_sync(0xFFFFFFFFu, incl, 31);
}

// The staged records expanded to sixteen bytes each (one value per byte), all consumer threads.
// `flip` is XORed into every expanded word (the branch-free body wants the sign position flipped).
// nibble: eight bytes per record instead (values below 16: elements 0..3 and 8..11 in the low halves of the two words'
// bytes, elements 4..7 and 12..15 in the high halves).
template <int HB>
__device__ __forceinline__ void expand_records(uint32_t s_raw, uint32_t s_expanded, uint32_t count, uint32_t tid,
                                               uint32_t flip, bool nibble = false) {
    for (uint32_t i = tid; i < count; i += kConsumerWarps * 32) {
        const uint32_t rp = s_raw + i * (2 * HB);
        uint4 v = unpack_record<HB>([&](int w) { return lds16(rp + 2 * w); });
        v.x ^= flip; v.y ^= flip; v.z ^= flip; v.w ^= flip;
        if (HB <= 4 && nibble) sts64(s_expanded + i * 8, make_uint2(v.x | (v.y << 4), v.z | (v.w << 4)));
        else sts128(s_expanded + i * 16, v);
    }
}

__device__ __forceinline__ void expand_records_any(int hbits, uint32_t s_raw, uint32_t s_expanded, uint32_t count,
                                                   uint32_t tid, uint32_t flip, bool nibble = false) {
    switch (hbits) {
        case 0: break;
        case 1: expand_records<1>(s_raw, s_expanded, count, tid, flip, nibble); break;
        case 2: expand_records<2>(s_raw, s_expanded, count, tid, flip, nibble); break;
        case 3: expand_records<3>(s_raw, s_expanded, count, tid, flip, nibble); break;
        case 4: expand_records<4>(s_raw, s_expanded, count, tid, flip, nibble); break;
        case 5: expand_records<5>(s_raw, s_expanded, count, tid, flip); break;
        case 6: expand_records<6>(s_raw, s_expanded, count, tid, flip); break;
        default: expand_records<7>(s_raw, s_expanded, count, tid, flip); break;
    }
}

// Barrier of the consumer threads only (the loader warp does not take part) that also ORs a flag over
// them, so that all consumers take the same decision whatever the moment another warp raised the flag.
__device__ __forceinline__ bool consumer_barrier_or(bool flag) {
    uint32_t any;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.or.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(any)
        : "r"(uint32_t(flag)), "n"(kConsumerWarps * 32)
        : "memory");
    return any != 0;
}

struct DecodeShared {
    uint64_t full[4];   // bulk copies of a stage have landed (kStages used)
    uint64_t empty[4];  // all consumer warps are done with a stage
    int abort;
    int pad[15];
};
static_assert(sizeof(DecodeShared) == 128, "control area is 128 bytes");

#define ENEC_FOR_EACH_MH(X, DT)                                                                         \
    X(DT, 1, 0) X(DT, 1, 1) X(DT, 1, 2) X(DT, 1, 3) X(DT, 1, 4)                                       \
    X(DT, 2, 0) X(DT, 2, 1) X(DT, 2, 2) X(DT, 2, 3)                                                   \
    X(DT, 3, 0) X(DT, 3, 1) X(DT, 3, 2)                                                               \
    X(DT, 4, 0) X(DT, 4, 1)                                                                           \
    X(DT, 5, 0)
#define ENEC_FOR_EACH_MH_BF16_ONLY(X, DT)                                                               \
    X(DT, 1, 5) X(DT, 1, 6) X(DT, 1, 7)                                                               \
    X(DT, 2, 4) X(DT, 2, 5) X(DT, 2, 6)                                                               \
    X(DT, 3, 3) X(DT, 3, 4) X(DT, 3, 5)                                                               \
    X(DT, 4, 2) X(DT, 4, 3) X(DT, 4, 4)                                                               \
    X(DT, 5, 1) X(DT, 5, 2) X(DT, 5, 3)                                                               \
    X(DT, 6, 0) X(DT, 6, 1) X(DT, 6, 2)                                                               \
    X(DT, 7, 0) X(DT, 7, 1)                                                                           \
    X(DT, 8, 0)

// What the loader tells the consumers about the block in a stage (first bytes of the stage).
struct BlockDesc {
    uint32_t first;     // offset of the block's first record inside the staged window
    uint32_t staged;    // records staged in shared memory
    uint32_t expect;    // wide groups of the block according to the prefix table
    uint32_t N;         // padded block length
    uint32_t real;      // real elements
    uint32_t code;      // m * 8 + (n - m); bit 7: the expanded records take the eight-byte form
    uint32_t b, n;
    StageLayout L;
    uint16_t* out;        // global: first element of the block
    const uint8_t* high;  // global: first record of the block
    const uint16_t* lo;   // global, fp32 only: low halves of the block's elements
};
static_assert(sizeof(BlockDesc) <= kStageMetaBytes, "descriptor fits the stage's meta area");

constexpr uint32_t kInlineJobs = 16;  // tensors of a short batch that fit the kernel's parameter space

// A launch decodes the blocks of one tensor or of a list of tensors. Blocks of all tensors form one
// index space; a CTA takes a contiguous range of it, so it changes tensor rarely. Long lists (the kernel instance
// with TICKET) hand the index space out in chunks of kTicketChunk consecutive blocks instead: the CTAs of an SM
// progress unequally, and with a fixed share each the launch ends when the slowest has finished. Such a list's
// device arrays are laid out as [jobs | prefix, padded to 16 bytes | ticket word, 16 bytes, zero at launch | the
// tensor of every chunk's first block], so the kernel finds the last two behind the prefix.
constexpr uint32_t kTicketChunk = 8;
constexpr uint32_t kSingleTicketChunk = 2;  // one large tensor: its blocks all cost the same, and a launch has few per CTA
__host__ __device__ inline uint64_t ticket_offset_behind_prefix(uint32_t n_jobs) {
    return align16((uint64_t(n_jobs) + 1) * sizeof(uint32_t));
}
struct DecodeBatch {
    const DecodeJob* jobs;    // device array, or null when the tensors travel inside the launch parameters
    const uint32_t* prefix;   // device array [n_jobs + 1]: blocks before each tensor (null with jobs)
    uint32_t n_jobs;
    uint32_t total_blocks;
    uint32_t blockwise;       // the streams are of the block-wise variant (one tensor only)
    DecodeJob inline_jobs[kInlineJobs];          // used when jobs is null (one tensor, or a short list)
    uint32_t inline_prefix[kInlineJobs + 1];
};

// 16 bytes from global memory through L2 only (no copy is left in L1, which is not coherent).
__device__ __forceinline__ uint4 ldg_l2_only(const void* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// Runs before the wait on the previous kernel of the stream, one thread per CTA: asks L2 for the
// compressed bytes of the CTA's first blocks, so that the copies issued after the wait find them there.
// What it reads may still be about to be written by that previous kernel, so nothing read here is
// used for anything but prefetch addresses, every address stays inside the caller's buffer
// [in, in + in_size), and the loads bypass L1; L2 is coherent, so a line prefetched too early is simply
// updated by the writer. Only for tensor lists that travel in the kernel parameters.
template <int DT, bool MAPPED = false>
__device__ __forceinline__ void prefetch_before_wait(const DecodeBatch& batch, uint32_t first_block, uint32_t n_mine) {
    if (batch.jobs != nullptr || n_mine == 0) return;
    uint32_t j = 0;
    while (j + 1 < batch.n_jobs && batch.inline_prefix[j + 1] <= first_block) ++j;
    const DecodeJob& job = batch.inline_jobs[j];
    const uint32_t k = first_block - batch.inline_prefix[j];
    if (job.in_size < kHeaderBytes + 4 * (uint64_t(k) + 3) + 16) return;
    const uint4 h0 = ldg_l2_only(job.in);        // magic, version/dtype, count
    const uint4 h1 = ldg_l2_only(job.in + 16);   // block, b/n/m/L, nblocks, total_groups
    const uint4 h2 = ldg_l2_only(job.in + 32);   // a_total
    const int n = int((h1.y >> 8) & 0xFF), m = int((h1.y >> 16) & 0xFF);
    if (h0.x != kMagic || n < 1 || n > exp_bits(DT) || m < 1 || m > n) return;
    const Geometry g = make_geometry(job.count);
    if (k >= g.nblocks) return;
    const Sections sec = make_sections(DT, job.count, g, n, m, h2.x, MAPPED);
    if (sec.total > job.in_size) return;
    const uint32_t* table = reinterpret_cast<const uint32_t*>(job.in + sec.table);
    const uint32_t ahead = n_mine < kStages ? n_mine : kStages;
    for (uint32_t i = 0; i < ahead && k + i < g.nblocks; ++i) {
        const uint32_t kk = k + i;
        const bool tail = kk + 1 == g.nblocks;
        const uint32_t N = tail ? g.tail_padded : kBlockElems;
        const uint32_t real = tail ? g.tail_real : kBlockElems;
        uint32_t t0, t1;
        asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(t0) : "l"(table + kk));
        asm volatile("ld.global.cg.u32 %0, [%1];" : "=r"(t1) : "l"(table + kk + 1));
        bulk_prefetch_l2(job.in + sec.mask + uint64_t(kk) * (kGroupsPerBlock / 8), uint32_t(align16(((N >> 4) + 7) / 8)));
        bulk_prefetch_l2(job.in + sec.low + uint64_t(kk) * (kBlockElems / 8) * m, uint32_t(align16(uint64_t(N) * m / 8)));
        if (DT == ENEC_FP16)
            bulk_prefetch_l2(job.in + sec.smhi + uint64_t(kk) * (kBlockElems / 8) * 3, uint32_t(align16(uint64_t(N) * 3 / 8)));
        bulk_prefetch_l2(job.in + sec.sm + uint64_t(kk) * kBlockElems, uint32_t(align16(real)));
        if (DT == ENEC_FP32)
            bulk_prefetch_l2(job.in + sec.smlo + uint64_t(kk) * kBlockElems * 2, uint32_t(align16(uint64_t(real) * 2)));
        const uint32_t hbits = uint32_t(n - m);
        if (hbits > 0 && t1 > t0 && t1 - t0 <= (N >> 4)) {
            const uint64_t r0 = (sec.high + uint64_t(t0) * 2 * hbits) & ~uint64_t(15);
            const uint64_t r1 = align16(sec.high + uint64_t(t1) * 2 * hbits);
            if (r1 <= sec.total && r1 > r0) bulk_prefetch_l2(job.in + r0, uint32_t(r1 - r0));
        }
    }
}

// MAPPED: the instance for streams of the frequency-rank variant (general block body with table look-ups only);
// each instance refuses the other kind of stream. TICKET: blocks are handed out by batch.ticket; the loader ends the
// consumers' loop with a descriptor of zero length.
// TICKET = 2: one large tensor. The ticket is a 64-bit word of the library's scratch that is never cleared: its high
// half is the number of the launch that uses it (inline_jobs[1].count; the word's address is inline_jobs[1].in), and
// the first CTA to find another number there starts it at zero for this launch (all earlier launches of the stream
// have ended by then). In both forms CTA c starts on chunk c without asking, and tickets count on from the grid size.
template <int DT, bool MAPPED = false, int TICKET = 0>
__global__ void __launch_bounds__(kDecodeThreads, 3)
enec_decode_kernel(const __grid_constant__ DecodeBatch batch, int* status) {
    extern __shared__ __align__(128) uint8_t smem[];
    DecodeShared* ctl = reinterpret_cast<DecodeShared*>(smem);
    const uint32_t stages = smem_u32(smem) + uint32_t(sizeof(DecodeShared));
    constexpr uint32_t S = kStages;

    pdl_launch_dependents();
    // everything up to pdl_wait() may run while the previous kernel of the stream still does
    const uint32_t first_block = uint32_t(uint64_t(blockIdx.x) * batch.total_blocks / gridDim.x);
    const uint32_t end_block = uint32_t(uint64_t(blockIdx.x + 1) * batch.total_blocks / gridDim.x);
    const uint32_t n_mine = end_block - first_block;
    if (threadIdx.x == kConsumerWarps * 32) {
        if constexpr (TICKET == 2)  // the CTA's first chunk
            prefetch_before_wait<DT, MAPPED>(batch, blockIdx.x * kSingleTicketChunk,
                                             blockIdx.x * kSingleTicketChunk < batch.total_blocks ? kSingleTicketChunk : 0);
        else
            prefetch_before_wait<DT, MAPPED>(batch, first_block, n_mine);
    }
    if (threadIdx.x == 0) {
        for (uint32_t s = 0; s < S; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], kConsumerWarps);
        }
        ctl->abort = 0;
        mbar_fence_init();
    }
    __syncthreads();
    pdl_wait();  // nothing above uses what it read from global memory, except as prefetch addresses
    if (blockIdx.x == 0) {
        // tensors without elements have no block that would bring their header before the loader: check them here
        const DecodeJob* all_jobs = batch.jobs ? batch.jobs : batch.inline_jobs;
        for (uint32_t q = threadIdx.x; q < batch.n_jobs; q += blockDim.x) {
            if (all_jobs[q].count == 0) {
                JobCtx jc;
                const int err = load_job<DT, MAPPED>(all_jobs[q], jc, batch.blockwise != 0);
                if (err) report(status, err);
            }
        }
    }
    if (batch.total_blocks == 0) return;

    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31;
    volatile int* abort_flag = &ctl->abort;

    if (warp == kConsumerWarps) {
        // ---------------- loader warp: lane 0 issues the copies of block after block ----------------
        if (lane != 0) return;
        // the tensor that holds first_block
        uint32_t j = 0;
        const DecodeJob* jobs = batch.jobs ? batch.jobs : batch.inline_jobs;
        const uint32_t* prefix = batch.jobs ? batch.prefix : batch.inline_prefix;
        // TICKET: the chunk in hand, the one after it (asked for a chunk ahead, so that the answer is there in time),
        // and the blocks of the chunk in hand that are issued
        [[maybe_unused]] uint32_t chunk = 0, next_chunk = 0, in_chunk = 0;
        [[maybe_unused]] uint32_t next_j = 0, next_first = 0, next_end = 0;  // the next chunk's tensor and its range of blocks
        constexpr uint32_t kChunk = TICKET == 2 ? kSingleTicketChunk : kTicketChunk;
        [[maybe_unused]] const uint32_t n_chunks = TICKET ? (batch.total_blocks + kChunk - 1) / kChunk : 0;
        [[maybe_unused]] uint32_t* const ticket =
            TICKET == 1 ? reinterpret_cast<uint32_t*>(reinterpret_cast<uintptr_t>(batch.prefix) + ticket_offset_behind_prefix(batch.n_jobs))
                        : nullptr;
        [[maybe_unused]] const uint32_t* const chunk_job = TICKET == 1 ? ticket + 4 : nullptr;
        [[maybe_unused]] unsigned long long* const ticket64 =
            TICKET == 2 ? reinterpret_cast<unsigned long long*>(const_cast<uint8_t*>(batch.inline_jobs[1].in)) : nullptr;
        [[maybe_unused]] auto take_ticket = [&]() -> uint32_t {
            if constexpr (TICKET == 2) return gridDim.x + uint32_t(atomicAdd(ticket64, 1ull));
            else return gridDim.x + atomicAdd(ticket, 1u);
        };
        [[maybe_unused]] auto look_up_next = [&]() {
            if constexpr (TICKET == 1) {
                if (next_chunk < n_chunks) {
                    next_j = chunk_job[next_chunk];
                    next_first = prefix[next_j];
                    next_end = prefix[next_j + 1];
                }
            } else {  // one tensor
                next_j = 0;
                next_first = 0;
                next_end = batch.total_blocks;
            }
        };
        if constexpr (TICKET) {
            if constexpr (TICKET == 2) {
                const unsigned long long mine = (unsigned long long)uint32_t(batch.inline_jobs[1].count) << 32;
                unsigned long long seen;
                asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(seen) : "l"(ticket64) : "memory");
                if ((seen >> 32) != (mine >> 32)) atomicCAS(ticket64, seen, mine);  // one CTA wins; the others find it done
            }
            chunk = blockIdx.x;
            next_chunk = take_ticket();
            if constexpr (TICKET == 1) { if (chunk < n_chunks) j = chunk_job[chunk]; }
            look_up_next();
        } else {
            uint32_t lo = 0, hi = batch.n_jobs;  // largest j with prefix[j] <= first_block
            while (hi - lo > 1) {
                const uint32_t mid = (lo + hi) >> 1;
                if (prefix[mid] <= first_block) lo = mid; else hi = mid;
            }
            j = lo;
        }
        uint32_t job_first = prefix[j];
        uint32_t job_end = prefix[j + 1];
        bool parsed = false;
        JobCtx jc;
        StageLayout L;
        int hbits = 0;
        const uint32_t* table = nullptr;
        uint32_t t1 = 0, t2 = 0;  // table[k + 1], table[k + 2] of the block about to be issued (one ahead)
        uint32_t issued = 0;
        bool failed = false;
        for (; TICKET || issued < n_mine; ++issued) {
            uint32_t gb = first_block + issued;
            [[maybe_unused]] bool jumped = false;  // TICKET: this block does not follow the one issued before it
            if constexpr (TICKET) {
                if (in_chunk == kChunk) {
                    chunk = next_chunk;
                    if (chunk >= n_chunks) break;
                    if (next_j != j) parsed = false;
                    j = next_j;
                    job_first = next_first;
                    job_end = next_end;
                    next_chunk = take_ticket();
                    look_up_next();
                    in_chunk = 0;
                    jumped = true;
                }
                gb = chunk * kChunk + in_chunk;
                ++in_chunk;
                if (chunk >= n_chunks || gb >= batch.total_blocks) break;
            }
            while (gb >= job_end) {  // next tensor (tensors without blocks are skipped)
                ++j;
                job_first = job_end;
                job_end = prefix[j + 1];
                parsed = false;
            }
            const uint32_t k = gb - job_first;
            uint32_t t0;
            if (!parsed) {
                const DecodeJob job = jobs[j];
                // the table sits right behind the header: fetch the block's two entries along with the
                // header instead of after it (they are only used once the header has been checked)
                uint32_t e0 = 0, e1 = 0;
                const bool early = job.in_size >= kHeaderBytes + 4 * (uint64_t(k) + 2);
                if (early) {
                    const uint32_t* tb = reinterpret_cast<const uint32_t*>(job.in + kHeaderBytes);
                    e0 = tb[k];
                    e1 = tb[k + 1];
                }
                const int err = early ? load_job<DT, MAPPED>(job, jc, batch.blockwise != 0) : ENEC_ERR_BAD_STREAM;
                if (err) {
                    *abort_flag = 1;
                    report(status, err);
                    failed = true;
                    break;
                }
                hbits = jc.n - jc.m;
                L = make_stage_layout(DT, jc.m, hbits, MAPPED);
                table = reinterpret_cast<const uint32_t*>(jc.in + jc.off_table);
                t0 = e0;
                t1 = e1;
                if constexpr (MAPPED) {  // the table of a frequency-rank stream sits behind its rank table
                    t0 = table[k];
                    t1 = table[k + 1];
                }
                parsed = true;
            } else {
                t0 = t1;
                t1 = t2;
                if constexpr (TICKET) {
                    if (jumped) {
                        t0 = table[k];
                        t1 = table[k + 1];
                    }
                }
            }
            const uint32_t s = issued % S, use = issued / S;
            if (use > 0 && !suspended_wait(&ctl->empty[s], (use - 1) & 1, abort_flag)) { failed = true; break; }
            const bool tail = (k + 1 == jc.nblocks);
            const uint32_t N = tail ? jc.tail_padded : kBlockElems;
            const uint32_t real = tail ? jc.tail_real : kBlockElems;
            int blk_b = jc.b, blk_n = jc.n, blk_m = jc.m;
            uint64_t low_src = jc.off_low + uint64_t(k) * (kBlockElems / 8) * uint32_t(jc.m);
            uint64_t h0;
            uint32_t expect;
            bool sound;
            if (jc.blockwise) {
                // this block's parameters and offsets, and the next entry for the end of its records
                const uint4 own = *reinterpret_cast<const uint4*>(jc.in + kHeaderBytes + 16 * uint64_t(k));
                const uint4 nxt = *reinterpret_cast<const uint4*>(jc.in + kHeaderBytes + 16 * uint64_t(k + 1));
                blk_b = int(own.x & 0xFFu); blk_n = int((own.x >> 8) & 0xFFu); blk_m = int((own.x >> 16) & 0xFFu);
                sound = blk_n >= 1 && blk_n <= exp_bits(DT) && blk_m >= 1 && blk_m <= blk_n && blk_b < (1 << exp_bits(DT)) &&
                        (own.x >> 24) == 0;
                hbits = sound ? blk_n - blk_m : 0;
                if (sound) L = make_stage_layout(DT, blk_m, hbits, false);
                const uint64_t rec0 = uint64_t(own.z) | (uint64_t(own.w) << 32), rec1 = uint64_t(nxt.z) | (uint64_t(nxt.w) << 32);
                const uint64_t rec_size = 2 * uint64_t(hbits);
                sound = sound && (k != 0 || (own.y == 0 && rec0 == 0));  // the sums start at zero
                sound = sound && rec1 >= rec0 && rec1 <= jc.total - jc.off_high && nxt.y == own.y + uint32_t(blk_m) &&
                        (rec_size ? (rec1 - rec0) % rec_size == 0 : rec1 == rec0);
                expect = sound && rec_size ? uint32_t((rec1 - rec0) / rec_size) : 0;
                low_src = jc.off_low + uint64_t(own.y) * (kBlockElems / 8);
                sound = sound && expect <= (N >> 4) && low_src + uint64_t(N) * uint32_t(blk_m) / 8 <= jc.off_smhi;
                h0 = jc.off_high + rec0;
            } else {
                sound = t1 >= t0 && t1 - t0 <= (N >> 4) && t1 <= jc.a_total;
                expect = t1 - t0;
                h0 = jc.off_high + uint64_t(t0) * (2 * hbits);
            }
            if (!sound) {
                *abort_flag = 1;
                report(status, ENEC_ERR_BAD_STREAM);
                failed = true;
                break;
            }
            // a full block with more wide groups than the stage holds in the sixteen-byte form takes the eight-byte
            // form when that holds them all (and its consumers will take the branch-free body)
            StageLayout Lb = L;
            bool nibble = false;
            if (kNibbleForm<DT, MAPPED> && hbits >= 1 && hbits <= 4 && expect > L.cap && real == kBlockElems &&
                plain_subtraction<DT>(uint32_t(blk_b), uint32_t(blk_n))) {
                const StageLayout L8 = make_stage_layout(DT, blk_m, hbits, false, true);
                if (expect <= L8.cap) { Lb = L8; nibble = true; }
            }
            const uint64_t w0 = h0 & ~uint64_t(15);
            uint32_t staged = expect < Lb.cap ? expect : Lb.cap;  // records staged in shared memory
            if (hbits == 0) staged = 0;
            const uint64_t w1 = align16(h0 + uint64_t(staged) * (2 * hbits));
            const uint32_t mask_bytes = uint32_t(align16(((N >> 4) + 7) / 8));
            const uint32_t low_bytes = uint32_t(align16(uint64_t(N) * uint32_t(blk_m) / 8));
            const uint32_t smhi_bytes = DT == ENEC_FP16 ? uint32_t(align16(uint64_t(N) * 3 / 8)) : 0;
            const uint32_t sm_bytes = uint32_t(align16(real));
            const uint32_t raw_bytes = staged ? uint32_t(w1 - w0) : 0;
            uint8_t* st = smem + sizeof(DecodeShared) + size_t(s) * kStageBytes;
            BlockDesc* d = reinterpret_cast<BlockDesc*>(st);
            d->first = uint32_t(h0 - w0);
            d->staged = staged;
            d->expect = expect;
            d->N = N;
            d->real = real;
            d->code = uint32_t(blk_m * 8 + hbits) | (nibble ? 128u : 0u);
            d->b = uint32_t(blk_b);
            d->n = uint32_t(blk_n);
            d->L = Lb;
            d->out = jc.out + uint64_t(k) * kBlockElems * (DT == ENEC_FP32 ? 2 : 1);
            if (DT == ENEC_FP32) {
                // the low halves go from global memory straight to the consumers' registers: start them
                // towards L2 along with the block's copies
                const uint8_t* lo = jc.in + jc.off_smlo + uint64_t(k) * kBlockElems * 2;
                d->lo = reinterpret_cast<const uint16_t*>(lo);
                bulk_prefetch_l2(lo, uint32_t(align16(uint64_t(real) * 2)));
            } else {
                d->lo = nullptr;
            }
            d->high = jc.in + h0;
            mbar_expect_tx(&ctl->full[s], mask_bytes + low_bytes + smhi_bytes + sm_bytes + raw_bytes +
                                              (MAPPED ? kRankTableBytes : 0u));
            if constexpr (MAPPED) bulk_g2s(st + kStageRankTable, jc.in + kHeaderBytes, kRankTableBytes, &ctl->full[s]);
            bulk_g2s(st + Lb.mask, jc.in + jc.off_mask + uint64_t(k) * (kGroupsPerBlock / 8), mask_bytes, &ctl->full[s]);
            bulk_g2s(st + Lb.low, jc.in + low_src, low_bytes, &ctl->full[s]);
            if (DT == ENEC_FP16)
                bulk_g2s(st + Lb.smhi, jc.in + jc.off_smhi + uint64_t(k) * (kBlockElems / 8) * 3, smhi_bytes, &ctl->full[s]);
            bulk_g2s(st + Lb.sm, jc.in + jc.off_sm + uint64_t(k) * kBlockElems, sm_bytes, &ctl->full[s]);
            if (raw_bytes) bulk_g2s(st + Lb.raw, jc.in + w0, raw_bytes, &ctl->full[s]);
            if (!jc.blockwise && k + 2 <= jc.nblocks) t2 = table[k + 2];  // for the tensor's next block
        }
        if constexpr (TICKET) {
            if (!failed) {  // tell the consumers that this was the last block
                const uint32_t s = issued % S, use = issued / S;
                if (use > 0 && !suspended_wait(&ctl->empty[s], (use - 1) & 1, abort_flag)) {
                    failed = true;
                } else {
                    BlockDesc* d = reinterpret_cast<BlockDesc*>(smem + sizeof(DecodeShared) + size_t(s) * kStageBytes);
                    d->N = 0;
                    mbar_expect_tx(&ctl->full[s], 0u);
                }
            }
        }
        if (failed) {
            if (!*abort_flag) { *abort_flag = 1; report(status, ENEC_ERR_TIMEOUT); }
            // let copies still in flight land before the CTA's shared memory is released
            const uint32_t from = issued > S ? issued - S : 0;
            for (uint32_t i = from; i < issued; ++i) mbar_wait_bounded(&ctl->full[i % S], (i / S) & 1);
        }
        return;
    }

    // ---------------- consumers ----------------
    const uint32_t tid = threadIdx.x;
    for (uint32_t i = 0; TICKET || i < n_mine; ++i) {
        const uint32_t s = i % S, use = i / S;
        const uint32_t st = stages + s * kStageBytes;
        // every consumer thread waits on the stage's mbarrier itself; the wait suspends the thread in hardware,
        // so waiting threads take no issue slots and wake the moment the copies have landed
        const bool arrived = suspended_wait(&ctl->full[s], use & 1, abort_flag);
        if (__any_sync(0xFFFFFFFFu, !arrived)) {
            if (lane == 0 && !*abort_flag) { *abort_flag = 1; report(status, ENEC_ERR_TIMEOUT); }
            consumer_barrier_or(true);  // the block's one barrier: the other warps leave with this one
            break;
        }
        const BlockDesc* d = reinterpret_cast<const BlockDesc*>(smem + sizeof(DecodeShared) + size_t(s) * kStageBytes);
        if (TICKET && d->N == 0) break;  // the loader's end mark
        const uint32_t N = d->N, expect = d->expect, code = kNibbleForm<DT, MAPPED> ? d->code & 127u : d->code;
        const bool nibble = kNibbleForm<DT, MAPPED> && (d->code & 128u) != 0;  // only set for blocks that take the branch-free body
        const uint32_t b = d->b, n = d->n;
        const uint32_t hbits = code & 7;
        const uint32_t cap = d->L.cap;
        const uint32_t o_rank = d->L.rank, o_low = d->L.low, o_smhi = d->L.smhi, o_sm = d->L.sm, o_raw = d->L.raw,
                       o_exp = d->L.expanded;
        const uint32_t sbit = 1u << (n - 1);
        const bool simple_sub = plain_subtraction<DT>(b, n);
        const bool full_block = N == kBlockElems && d->real == kBlockElems && expect <= cap && (MAPPED || simple_sub);
        // preparation: ranks of the wide groups and expanded records
        if (hbits > 0) {
            // the branch-free body wants narrow groups to point at the flip slot and flipped records
            const uint32_t flip4 = MAPPED ? 0u : rep4(1u << (hbits - 1));
            if (tid == 0) {
                if (nibble) sts64(st + o_exp + cap * 8, make_uint2(flip4 | (flip4 << 4), flip4 | (flip4 << 4)));
                else sts128(st + o_exp + cap * 16, make_uint4(flip4, flip4, flip4, flip4));
            }
            const uint32_t wide = build_rank_array(st + d->L.mask, st + o_rank, N, tid, full_block ? cap : kNotWide);
            if (wide != expect && lane == 0) {  // the prefix table must agree with the mask
                *abort_flag = 1;
                report(status, ENEC_ERR_BAD_STREAM);
            }
            expand_records_any(int(hbits), st + o_raw + d->first, st + o_exp, d->staged, tid, full_block ? flip4 : 0, nibble);
        }
        RunCtx r;
        {
            const uint32_t c = (b + sbit) & 0xFF;
            r.s4 = rep4(sbit);
            r.c4_or_h = rep4(c) | 0x80808080u;
            r.fix = ~rep4(c) & 0x80808080u;
            r.b4 = rep4(b);
            r.c4 = rep4(c);
            r.n = int(n);
            r.cap = cap;
            r.sm = st + o_sm;
            r.rank = st + o_rank;
            r.expanded = st + o_exp;
            r.out = d->out;
            r.high = d->high;
            r.lo = d->lo;
            if constexpr (MAPPED) r.c4 = st + kStageRankTable;  // the ranked bodies' table
            r.real = d->real;
        }
        if (consumer_barrier_or(*abort_flag != 0)) break;
        if (nibble) {  // a full block with more wide groups than the sixteen-byte form holds
            if constexpr (kNibbleForm<DT, MAPPED>) {
                switch (code) {
#define ENEC_CASE(DTV, MV, HV)                                                               \
    case MV * 8 + HV:                                                                        \
        if constexpr (HV >= 1 && HV <= 4 && (DTV != ENEC_FP16 || MV + HV <= 5))               \
            decode_full_block<DTV, MV, HV, false, true>(r, st + o_low, st + o_smhi, tid);    \
        break;
                    ENEC_FOR_EACH_MH(ENEC_CASE, DT)
                    ENEC_FOR_EACH_MH_BF16_ONLY(ENEC_CASE, DT)
#undef ENEC_CASE
                    default: break;
                }
            }
        } else
        switch (code) {
#define ENEC_CASE(DTV, MV, HV)                                                               \
    case MV * 8 + HV:                                                                        \
        if (full_block) decode_full_block<DTV, MV, HV, MAPPED>(r, st + o_low, st + o_smhi, tid); \
        else decode_block<DTV, MV, HV, MAPPED>(r, st + o_low, st + o_smhi, N, tid);          \
        break;
            ENEC_FOR_EACH_MH(ENEC_CASE, DT)
#undef ENEC_CASE
#define ENEC_CASE(DTV, MV, HV)                                                               \
    case MV * 8 + HV:                                                                        \
        if constexpr (DTV != ENEC_FP16) {                                                    \
            if (full_block) decode_full_block<DTV, MV, HV, MAPPED>(r, st + o_low, st + o_smhi, tid); \
            else decode_block<DTV, MV, HV, MAPPED>(r, st + o_low, st + o_smhi, N, tid);      \
        }                                                                                    \
        break;
            ENEC_FOR_EACH_MH_BF16_ONLY(ENEC_CASE, DT)
#undef ENEC_CASE
            default: break;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&ctl->empty[s]);
    }
}

}  // namespace enec
