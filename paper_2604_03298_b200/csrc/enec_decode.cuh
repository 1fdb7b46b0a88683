// Decompression kernel: unpack + reconstruct (Sec. 5.1 decompression flow).
//
// One persistent CTA per resident slot. A producer warp stages each 16384-element block's compressed
// segments (group mask, low plane, fp16 sign/mantissa-high plane, sign/mantissa bytes, wide-group
// records) into shared memory with bulk asynchronous copies completing on an mbarrier; eight consumer
// warps undo Algorithm 2 on packed bytes (four elements per 32-bit operation), locate each wide group's
// record with a popcount prefix over the block's mask, apply the inverse transform of Sec. 5.3 and
// write 16-byte coalesced stores. Every wait is bounded and ends in an error status, never a hang.
#pragma once

#include "enec_common.cuh"

namespace enec {

constexpr int kConsumerWarps = 8;
constexpr int kDecodeThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 4;
constexpr uint32_t kDecodeSmemBytes = 74 * 1024;  // three CTAs per SM
constexpr uint32_t kStageMetaBytes = 16;

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
__host__ __device__ constexpr int folds_for(int w) {
    int f = 0;
    while ((w << f) < 8) ++f;
    return f;
}
__host__ __device__ constexpr int bitrev(int t, int f) {
    int r = 0;
    for (int i = 0; i < f; ++i) r |= ((t >> i) & 1) << (f - 1 - i);
    return r;
}

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
__device__ __forceinline__ uint2 load_octet(const uint8_t* S, uint32_t i0, uint32_t thalf) {
    const bool odd = i0 >= thalf;
    const uint32_t pos = 2 * (odd ? i0 - thalf : i0);
    const uint4 v = *reinterpret_cast<const uint4*>(S + pos);
    const uint32_t sel = odd ? 0x7531u : 0x6420u;
    return make_uint2(prmt(v.x, v.y, sel), prmt(v.z, v.w, sel));
}

// out[e] (e < 2^LOG_UNITS) = packed W_IN-bit values of the eight elements j + e * n8 + (0..7) of this level.
template <int W_IN, int LOG_UNITS>
__device__ __forceinline__ void unpack_plane_level(const uint8_t* S, uint32_t nb_off, uint32_t j, uint32_t n8,
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
__device__ __forceinline__ void unpack_plane(const uint8_t* S, uint32_t j, uint32_t N, uint2 (&y)[8]) {
    unpack_plane_level<A, 3>(S, 0, j, N >> 3, (N * A) >> 4, y);
}

// One element of a plane of N >= 16 elements of `a` bits, bit by bit (used only for blocks shorter than
// 128 elements, where lane runs of eight do not exist).
__device__ inline uint32_t unpack_plane_scalar(const uint8_t* S, uint32_t N, int a, uint32_t e) {
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
        value |= ((uint32_t(S[pos]) >> p) & 1u) << q;
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

// The eight H-bit values of half `half` (elements 8 half .. 8 half + 7) of the record at rp (2-byte aligned).
template <int H>
__device__ __forceinline__ uint2 unpack_record_half(const uint8_t* rp, uint32_t half) {
    uint32_t q[H];
#pragma unroll
    for (int i = 0; i < H; ++i) q[i] = *reinterpret_cast<const uint16_t*>(rp + 2 * i);
    uint32_t pr[8];  // pr[e] = elements 2e, 2e + 1
    unpack_record_level<H, H, 3>(q, 0, pr);
    const uint2 h0 = make_uint2(prmt(pr[0], pr[1], 0x5410u), prmt(pr[2], pr[3], 0x5410u));
    const uint2 h1 = make_uint2(prmt(pr[4], pr[5], 0x5410u), prmt(pr[6], pr[7], 0x5410u));
    return half ? h1 : h0;
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
    uint64_t off_table, off_mask, off_low, off_smhi, off_sm, off_high, total;
};

// Reads and validates the header. Returns 0 or an enec_status.
template <int DT>
__device__ inline int load_job(const DecodeJob& job, JobCtx& c) {
    const Header h = *reinterpret_cast<const Header*>(job.in);
    if (job.in_size < kHeaderBytes + 16) return ENEC_ERR_BAD_STREAM;
    if (h.magic != kMagic || h.version != kVersion || h.dtype != DT || h.count != job.count ||
        h.block != kBlockElems || h.L != kGroupElems)
        return ENEC_ERR_BAD_STREAM;
    constexpr int E = DT == ENEC_BF16 ? 8 : 5;
    if (h.n < 1 || h.n > E || h.m < 1 || h.m > h.n || h.b >= (1 << E)) return ENEC_ERR_BAD_STREAM;
    const Geometry g = make_geometry(job.count);
    if (h.nblocks != g.nblocks || h.total_groups != g.total_groups || h.a_total > g.total_groups)
        return ENEC_ERR_BAD_STREAM;
    const Sections s = make_sections(DT, job.count, g, h.n, h.m, h.a_total);
    if (h.total_bytes != s.total || job.in_size < s.total) return ENEC_ERR_BAD_STREAM;
    c.in = job.in;
    c.out = job.out;
    c.nblocks = g.nblocks;
    c.tail_real = g.tail_real;
    c.tail_padded = g.tail_padded;
    c.a_total = h.a_total;
    c.b = h.b; c.n = h.n; c.m = h.m;
    c.off_table = s.table; c.off_mask = s.mask; c.off_low = s.low; c.off_smhi = s.smhi; c.off_sm = s.sm;
    c.off_high = s.high; c.total = s.total;
    return 0;
}

// Shared-memory layout of one pipeline stage (offsets from the stage base; all multiples of 16).
struct StageLayout {
    uint32_t meta, mask, low, smhi, sm, high, bytes;
};
__device__ __forceinline__ StageLayout make_stage_layout(int dt, int m, int hbits) {
    StageLayout L;
    L.meta = 0;
    L.mask = kStageMetaBytes;
    L.low = L.mask + kGroupsPerBlock / 8;
    L.smhi = L.low + kBlockElems * uint32_t(m) / 8;
    L.sm = L.smhi + (dt == ENEC_FP16 ? kBlockElems * 3 / 8 : 0);
    L.high = L.sm + kBlockElems;
    L.bytes = L.high + uint32_t(align16(uint64_t(kGroupsPerBlock) * 2 * hbits + 32));  // window may start/end off-boundary
    return L;
}

struct RunCtx {
    const uint8_t* sm;    // shared: sign/mantissa bytes of the block
    const uint8_t* high;  // shared: first record of the block
    uint16_t* out;        // global: first element of the block
    uint32_t real;        // real elements in the block
    uint32_t c4_or_h, fix, s4, b4;  // packed transform constants
    int n;
};

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

// Finishes eight consecutive elements e0 .. e0+7 of a block: wide-group high bits, inverse transform,
// rejoin with sign/mantissa, store.
template <int DT, int M, int HB>
__device__ __forceinline__ void finish_run(const RunCtx& r, uint2 y, uint2 hs, uint32_t e0, uint32_t mword,
                                           uint32_t mprefix, bool active) {
    if constexpr (HB > 0) {
        const uint32_t bit = (e0 >> 4) & 31;
        if ((mword >> bit) & 1) {
            const uint32_t rank = mprefix + __popc(mword & ((1u << bit) - 1));
            const uint2 hi = unpack_record_half<HB>(r.high + rank * (2 * HB), (e0 >> 3) & 1);
            y.x |= hi.x << M;
            y.y |= hi.y << M;
        }
    }
    const uint32_t x0 = inverse_transform4<DT>(r, y.x);
    const uint32_t x1 = inverse_transform4<DT>(r, y.y);
    const uint2 smv = *reinterpret_cast<const uint2*>(r.sm + e0);
    uint32_t lo0, lo1, hi0, hi1;
    if (DT == ENEC_BF16) {
        // word = sign << 15 | x << 7 | mant7 ; sm byte = sign << 7 | mant7
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
    if (e0 + 8 <= r.real) {
        *reinterpret_cast<uint4*>(r.out + e0) = w;
    } else if (e0 < r.real) {
        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
        for (uint32_t i = 0; e0 + i < r.real; ++i) r.out[e0 + i] = uint16_t(ww[i >> 1] >> (16 * (i & 1)));
    }
}

// One block, all consumer threads. tid = 0..255. N = padded block length.
template <int DT, int M, int HB>
__device__ __forceinline__ void decode_block(const RunCtx& r, const uint8_t* s_low, const uint8_t* s_smhi,
                                             const uint32_t* s_mask, uint32_t N, uint32_t tid) {
    const uint32_t lane = tid & 31;
    const uint32_t groups = N >> 4;
    // per-warp exclusive popcount prefix over the block's mask words
    uint32_t mw = 0;
    if (lane * 32 < groups) {
        mw = s_mask[lane];
        if (groups - lane * 32 < 32) mw &= (1u << (groups - lane * 32)) - 1;
    }
    if (HB == 0) mw = 0;
    uint32_t incl = __popc(mw);
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= uint32_t(d)) incl += t;
    }
    const uint32_t excl = incl - __popc(mw);

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
            for (int c = 0; c < 8; ++c) {
                const uint32_t e0 = c * n8 + j;
                const uint32_t wi = e0 >> 9;
                const uint32_t mword = __shfl_sync(0xFFFFFFFFu, mw, wi);
                const uint32_t mpre = __shfl_sync(0xFFFFFFFFu, excl, wi);
                finish_run<DT, M, HB>(r, y[c], DT == ENEC_FP16 ? hs[c] : make_uint2(0, 0), e0, mword, mpre, active);
            }
        }
    } else if (tid < 32) {
        // short tail block (16, 32 or 64 elements): one run of eight per lane, values rebuilt bit by bit
        const bool active = lane * 8 < N;
        const uint32_t e0 = active ? lane * 8 : 0;
        uint32_t yb[2] = {0, 0}, hb[2] = {0, 0};
        for (uint32_t i = 0; i < 8; ++i) {
            yb[i >> 2] |= unpack_plane_scalar(s_low, N, M, e0 + i) << (8 * (i & 3));
            if (DT == ENEC_FP16) hb[i >> 2] |= unpack_plane_scalar(s_smhi, N, 3, e0 + i) << (8 * (i & 3));
        }
        const uint32_t mword = __shfl_sync(0xFFFFFFFFu, mw, 0);
        const uint32_t mpre = __shfl_sync(0xFFFFFFFFu, excl, 0);
        finish_run<DT, M, HB>(r, make_uint2(yb[0], yb[1]), make_uint2(hb[0], hb[1]), e0, mword, mpre, active);
    }
}

struct DecodeShared {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
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

template <int DT>
__global__ void __launch_bounds__(kDecodeThreads, 3)
enec_decode_kernel(DecodeJob job, int* status) {
    extern __shared__ __align__(128) uint8_t smem[];
    DecodeShared* ctl = reinterpret_cast<DecodeShared*>(smem);
    uint8_t* stages = smem + sizeof(DecodeShared);

    JobCtx jc;
    const int err = load_job<DT>(job, jc);
    if (err) {
        if (threadIdx.x == 0 && blockIdx.x == 0) report(status, err);
        return;
    }
    const int hbits = jc.n - jc.m;
    const StageLayout L = make_stage_layout(DT, jc.m, hbits);
    int nstages = int((kDecodeSmemBytes - sizeof(DecodeShared)) / L.bytes);
    if (nstages > kMaxStages) nstages = kMaxStages;
    if (nstages < 1) {  // cannot happen for valid (m, n): the largest stage is below 54 KB
        if (threadIdx.x == 0 && blockIdx.x == 0) report(status, ENEC_ERR_BAD_STREAM);
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < nstages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], kConsumerWarps);
        }
        ctl->abort = 0;
        mbar_fence_init();
    }
    __syncthreads();

    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31;
    volatile int* abort_flag = &ctl->abort;

    if (warp == kConsumerWarps) {
        // ---------------- producer ----------------
        if (lane != 0) return;
        const uint32_t* table = reinterpret_cast<const uint32_t*>(jc.in + jc.off_table);
        uint32_t issued = 0;
        for (uint32_t k = blockIdx.x; k < jc.nblocks; k += gridDim.x, ++issued) {
            const int s = int(issued % uint32_t(nstages));
            const uint32_t use = issued / uint32_t(nstages);
            if (use > 0 && !mbar_wait_bounded(&ctl->empty[s], (use - 1) & 1)) {
                *abort_flag = 1;
                report(status, ENEC_ERR_TIMEOUT);
                break;
            }
            if (*abort_flag) break;
            const bool tail = (k + 1 == jc.nblocks);
            const uint32_t N = tail ? jc.tail_padded : kBlockElems;
            const uint32_t real = tail ? jc.tail_real : kBlockElems;
            const uint32_t t0 = table[k], t1 = table[k + 1];
            uint8_t* st = stages + size_t(s) * L.bytes;
            uint32_t* meta = reinterpret_cast<uint32_t*>(st + L.meta);
            const uint64_t h0 = jc.off_high + uint64_t(t0) * (2 * hbits);
            const uint64_t h1 = jc.off_high + uint64_t(t1) * (2 * hbits);
            const uint64_t w0 = h0 & ~uint64_t(15), w1 = align16(h1);
            bool bad = t1 < t0 || t1 - t0 > (N >> 4) || t1 > jc.a_total || w1 > jc.total;
            if (bad) {
                *abort_flag = 1;
                report(status, ENEC_ERR_BAD_STREAM);
                break;
            }
            const uint32_t mask_bytes = uint32_t(align16(((N >> 4) + 7) / 8));
            const uint32_t low_bytes = uint32_t(align16(uint64_t(N) * jc.m / 8));
            const uint32_t smhi_bytes = DT == ENEC_FP16 ? uint32_t(align16(uint64_t(N) * 3 / 8)) : 0;
            const uint32_t sm_bytes = uint32_t(align16(real));
            const uint32_t high_bytes = (hbits > 0 && t1 > t0) ? uint32_t(w1 - w0) : 0;
            meta[0] = uint32_t(h0 - w0);  // offset of the block's first record inside the staged window
            meta[1] = t1 - t0;
            mbar_expect_tx(&ctl->full[s], mask_bytes + low_bytes + smhi_bytes + sm_bytes + high_bytes);
            bulk_g2s(st + L.mask, jc.in + jc.off_mask + uint64_t(k) * (kGroupsPerBlock / 8), mask_bytes, &ctl->full[s]);
            bulk_g2s(st + L.low, jc.in + jc.off_low + uint64_t(k) * (kBlockElems / 8) * jc.m, low_bytes, &ctl->full[s]);
            if (DT == ENEC_FP16)
                bulk_g2s(st + L.smhi, jc.in + jc.off_smhi + uint64_t(k) * (kBlockElems / 8) * 3, smhi_bytes, &ctl->full[s]);
            bulk_g2s(st + L.sm, jc.in + jc.off_sm + uint64_t(k) * kBlockElems, sm_bytes, &ctl->full[s]);
            if (high_bytes) bulk_g2s(st + L.high, jc.in + w0, high_bytes, &ctl->full[s]);
        }
        if (*abort_flag) {
            // let copies still in flight land before the CTA's shared memory is released
            const uint32_t first = issued > uint32_t(nstages) ? issued - uint32_t(nstages) : 0;
            for (uint32_t i = first; i < issued; ++i)
                mbar_wait_bounded(&ctl->full[i % uint32_t(nstages)], (i / uint32_t(nstages)) & 1);
        }
        return;
    }

    // ---------------- consumers ----------------
    RunCtx r;
    {
        const uint32_t sbit = 1u << (jc.n - 1);
        const uint32_t c = (uint32_t(jc.b) + sbit) & 0xFF;
        r.s4 = rep4(sbit);
        r.c4_or_h = rep4(c) | 0x80808080u;
        r.fix = ~rep4(c) & 0x80808080u;
        r.b4 = rep4(uint32_t(jc.b));
        r.n = jc.n;
    }
    const int code = jc.m * 8 + hbits;
    uint32_t done = 0;
    for (uint32_t k = blockIdx.x; k < jc.nblocks; k += gridDim.x, ++done) {
        const int s = int(done % uint32_t(nstages));
        const uint32_t use = done / uint32_t(nstages);
        bool ok = true;
        if (lane == 0) {
            ok = false;
            for (uint32_t it = 0; it < (1u << 22); ++it) {
                if (mbar_try_wait(&ctl->full[s], use & 1)) { ok = true; break; }
                if (*abort_flag) break;
                if (it > 32) __nanosleep(128);
            }
            if (!ok && !*abort_flag) {
                *abort_flag = 1;
                report(status, ENEC_ERR_TIMEOUT);
            }
        }
        ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        if (lane != 0) mbar_try_wait(&ctl->full[s], use & 1);  // acquire the staged bytes in every lane
        const bool tail = (k + 1 == jc.nblocks);
        const uint32_t N = tail ? jc.tail_padded : kBlockElems;
        const uint8_t* st = stages + size_t(s) * L.bytes;
        const uint32_t* meta = reinterpret_cast<const uint32_t*>(st + L.meta);
        r.sm = st + L.sm;
        r.high = st + L.high + meta[0];
        r.out = jc.out + uint64_t(k) * kBlockElems;
        r.real = tail ? jc.tail_real : kBlockElems;
        const uint8_t* s_low = st + L.low;
        const uint8_t* s_smhi = st + L.smhi;
        const uint32_t* s_mask = reinterpret_cast<const uint32_t*>(st + L.mask);
        switch (code) {
#define ENEC_CASE(DTV, MV, HV)                                                        \
    case MV * 8 + HV:                                                                 \
        decode_block<DTV, MV, HV>(r, s_low, s_smhi, s_mask, N, threadIdx.x);          \
        break;
            ENEC_FOR_EACH_MH(ENEC_CASE, DT)
#undef ENEC_CASE
#define ENEC_CASE(DTV, MV, HV)                                                        \
    case MV * 8 + HV:                                                                 \
        if constexpr (DTV == ENEC_BF16) decode_block<DTV, MV, HV>(r, s_low, s_smhi, s_mask, N, threadIdx.x); \
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
