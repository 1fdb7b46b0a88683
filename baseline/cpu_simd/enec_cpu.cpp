// A multi-threaded, vectorised CPU implementation of the ENEC stream format (Sec. 7.1 "Hardware-Specific
// Optimizations" mentions a CPU version built on AVX2 and BMI2: the method's
// stages map onto CPU SIMD; this is such a variant, kept as a stronger host baseline than the plain oracle).
// It writes and reads exactly the stream layout of the CUDA library and of the oracle, but shares no code with
// either: it is a third, independent implementation whose streams the tests compare byte for byte.
//
// Vectorisation: the front end of a full bf16 block uses AVX2 directly (one 256-bit vector is one group of
// sixteen values, so the group's width test is a single vptest); Algorithm 2 is written as whole-array steps
// over 16-bit lanes that gcc turns into AVX2 code at -O3; blocks are spread over std::thread workers.
// Not part of the product: nothing in the CUDA library or its Python binding uses this file.
#include <immintrin.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <thread>
#include <vector>

namespace {

constexpr uint32_t kBlock = 16384;
constexpr uint32_t kGroup = 16;
constexpr uint32_t kGroupsPerBlock = kBlock / kGroup;
constexpr size_t kHeader = 64;

inline size_t a16(size_t v) { return (v + 15) & ~size_t(15); }
inline int exp_bits(int dt) { return dt == 1 ? 5 : 8; }
inline int bits_of(uint64_t v) { int w = 0; while (v) { ++w; v >>= 1; } return w; }

struct Shape {
    uint32_t nblocks = 0, tail_real = 0, tail_padded = 0, groups = 0;
    uint64_t padded = 0;
};
Shape shape_of(size_t count) {
    Shape s;
    if (!count) return s;
    s.nblocks = uint32_t((count + kBlock - 1) / kBlock);
    s.tail_real = uint32_t(count - size_t(s.nblocks - 1) * kBlock);
    uint32_t p = kGroup;
    while (p < s.tail_real) p <<= 1;
    s.tail_padded = p;
    s.padded = uint64_t(s.nblocks - 1) * kBlock + p;
    s.groups = uint32_t(s.padded / kGroup);
    return s;
}
struct Layout { size_t table, mask, low, smhi, sm, smlo, high, total; };
Layout layout_of(int dt, size_t count, const Shape& s, int n, int m, uint64_t wide_total) {
    Layout L;
    L.table = kHeader;
    L.mask = L.table + a16(4 * (size_t(s.nblocks) + 1));
    L.low = L.mask + a16((size_t(s.groups) + 7) / 8);
    L.smhi = L.low + a16(size_t(s.padded) * m / 8);
    L.sm = L.smhi + (dt == 1 ? a16(size_t(s.padded) * 3 / 8) : 0);
    L.smlo = L.sm + a16(count);
    L.high = L.smlo + (dt == 2 ? a16(count * 2) : 0);
    L.total = L.high + a16(size_t(wide_total) * 2 * (n - m));
    return L;
}

// ---- Algorithm 2 as whole-array steps ------------------------------------------------------------
// lanes[0..N) are overwritten; nb is scratch of at least N * a / 8 + 2 bytes. Returns the bytes written.
size_t pack_lanes(uint16_t* __restrict__ lanes, size_t N, int a, uint8_t* __restrict__ nb, uint8_t* __restrict__ out) {
    int width = a;
    size_t length = N, total = 0;
    while (width > 0) {
        while (length > 1 && width < 8) {
            length >>= 1;
            const uint16_t* upper = lanes + length;
            for (size_t i = 0; i < length; ++i) lanes[i] = uint16_t(lanes[i] | (upper[i] << width));
            width <<= 1;
        }
        uint8_t* dst = nb + total;
        for (size_t j = 0; j < length; ++j) {
            dst[j] = uint8_t(lanes[j]);
            lanes[j] = uint16_t(lanes[j] >> 8);
        }
        width -= 8;
        total += length;
    }
    if (total & 1) nb[total++] = 0;
    const size_t half = total >> 1;
    for (size_t i = 0; i < half; ++i) {
        out[2 * i] = nb[i];
        out[2 * i + 1] = nb[i + half];
    }
    return total;
}

// Inverse: the forward schedule is replayed to find the byte ranges, then undone last step first.
void unpack_lanes(const uint8_t* __restrict__ in, size_t N, int a, uint16_t* __restrict__ lanes, uint8_t* __restrict__ nb) {
    struct Step { uint32_t fold, length, width, offset; };
    Step steps[40];
    int ns = 0;
    size_t total = 0;
    {
        int width = a;
        size_t length = N;
        while (width > 0) {
            while (length > 1 && width < 8) {
                length >>= 1;
                steps[ns++] = {1u, uint32_t(length), uint32_t(width), 0u};
                width <<= 1;
            }
            steps[ns++] = {0u, uint32_t(length), 0u, uint32_t(total)};
            width -= 8;
            total += length;
        }
        if (total & 1) ++total;
    }
    const size_t half = total >> 1;
    for (size_t i = 0; i < half; ++i) {
        nb[i] = in[2 * i];
        nb[i + half] = in[2 * i + 1];
    }
    memset(lanes, 0, N * sizeof(uint16_t));
    for (int s = ns - 1; s >= 0; --s) {
        const Step& st = steps[s];
        if (st.fold) {
            const uint16_t keep = uint16_t((1u << st.width) - 1);
            uint16_t* upper = lanes + st.length;
            for (uint32_t i = 0; i < st.length; ++i) {
                upper[i] = uint16_t(lanes[i] >> st.width);
                lanes[i] = uint16_t(lanes[i] & keep);
            }
        } else {
            const uint8_t* src = nb + st.offset;
            for (uint32_t j = 0; j < st.length; ++j) lanes[j] = uint16_t((lanes[j] << 8) | src[j]);
        }
    }
}

// ---- parameter choice (Sec. 5.5: Eq. 1, Eq. 3, Eq. 4 at L = 16) -------------------------------------
inline uint32_t forward(uint32_t x, int b, int n) { return (uint32_t(b) - x) & ((1u << n) - 1); }

void choose_params(const uint64_t* hist, int E, int* b_out, int* n_out, int* m_out) {
    const int bins = 1 << E;
    int lo = -1, hi = -1;
    uint64_t total = 0;
    for (int x = 0; x < bins; ++x)
        if (hist[x]) { if (lo < 0) lo = x; hi = x; total += hist[x]; }
    if (!total) { *b_out = 0; *n_out = 1; *m_out = 1; return; }
    int best_b = lo, best_n = 0;
    uint64_t best_cost = ~0ull;
    for (int b = lo; b <= hi; ++b) {
        const int up = hi - b;
        int n = std::max(bits_of(uint64_t(b - lo)), up <= 1 ? 0 : bits_of(uint64_t(up - 1))) + 1;
        n = std::min(std::max(n, 1), E);
        uint64_t cost = 0;
        for (int x = lo; x <= hi; ++x) cost += hist[x] * forward(uint32_t(x), b, n);
        if (cost < best_cost || (cost == best_cost && n < best_n)) { best_cost = cost; best_b = b; best_n = n; }
    }
    uint64_t by_width[9] = {0};
    for (int x = lo; x <= hi; ++x) by_width[bits_of(forward(uint32_t(x), best_b, best_n))] += hist[x];
    int best_m = 1;
    double best_bits = 0.0;
    uint64_t fit = by_width[0];
    for (int m = 1; m <= best_n; ++m) {
        fit += by_width[m];
        const double p = double(fit) / double(total);
        const double p2 = p * p, p4 = p2 * p2, p8 = p4 * p4, p16 = p8 * p8;
        const double bits = (double(best_n) + 0.0625) + double(m - best_n) * p16;
        if (m == 1 || bits < best_bits) { best_m = m; best_bits = bits; }
    }
    *b_out = best_b; *n_out = best_n; *m_out = best_m;
}

// ---- workers ---------------------------------------------------------------------------------------
template <class Fn>
void parallel_blocks(uint32_t nblocks, int threads, Fn fn) {
    threads = std::max(1, std::min<int>(threads, int(nblocks)));
    if (threads == 1) { fn(0, 0u, nblocks); return; }
    std::vector<std::thread> pool;
    for (int t = 0; t < threads; ++t) {
        const uint32_t first = uint32_t(uint64_t(nblocks) * t / threads), last = uint32_t(uint64_t(nblocks) * (t + 1) / threads);
        pool.emplace_back([=] { fn(t, first, last); });
    }
    for (auto& th : pool) th.join();
}

struct Scratch {
    std::vector<uint16_t> y, lanes, side;
    std::vector<uint8_t> nb;
    Scratch() : y(kBlock), lanes(kBlock), side(kBlock), nb(kBlock + 16) {}
};

inline uint32_t word_at(const void* in, int dt, size_t i) {
    return dt == 2 ? static_cast<const uint32_t*>(in)[i] : static_cast<const uint16_t*>(in)[i];
}

// Exponent field and stored sign/mantissa byte(s) of one block; y for padding elements is 0.
void front_end(const void* in, int dt, size_t first, uint32_t real, uint32_t padded, int b, int n, uint16_t* y,
               uint16_t* side /* fp16: sign | mantissa bits 9..8 */, uint8_t* sm, uint8_t* smlo) {
    const uint16_t nmask = uint16_t((1u << n) - 1);
    uint32_t i = 0;
    if (dt == 0) {
        const uint16_t* w16 = static_cast<const uint16_t*>(in) + first;
        const __m256i vb = _mm256_set1_epi16(short(b)), vn = _mm256_set1_epi16(short(nmask));
        const __m256i ff = _mm256_set1_epi16(0xFF), s80 = _mm256_set1_epi16(0x80), m7f = _mm256_set1_epi16(0x7F);
        for (; i + 32 <= real; i += 32) {
            const __m256i w0 = _mm256_loadu_si256(reinterpret_cast<const __m256i*>(w16 + i));
            const __m256i w1 = _mm256_loadu_si256(reinterpret_cast<const __m256i*>(w16 + i + 16));
            const __m256i x0 = _mm256_and_si256(_mm256_srli_epi16(w0, 7), ff), x1 = _mm256_and_si256(_mm256_srli_epi16(w1, 7), ff);
            _mm256_storeu_si256(reinterpret_cast<__m256i*>(y + i), _mm256_and_si256(_mm256_sub_epi16(vb, x0), vn));
            _mm256_storeu_si256(reinterpret_cast<__m256i*>(y + i + 16), _mm256_and_si256(_mm256_sub_epi16(vb, x1), vn));
            const __m256i s0 = _mm256_or_si256(_mm256_and_si256(_mm256_srli_epi16(w0, 8), s80), _mm256_and_si256(w0, m7f));
            const __m256i s1 = _mm256_or_si256(_mm256_and_si256(_mm256_srli_epi16(w1, 8), s80), _mm256_and_si256(w1, m7f));
            const __m256i packed = _mm256_permute4x64_epi64(_mm256_packus_epi16(s0, s1), 0xD8);
            _mm256_storeu_si256(reinterpret_cast<__m256i*>(sm + i), packed);
        }
    }
    for (; i < real; ++i) {
        const uint32_t w = word_at(in, dt, first + i);
        uint32_t x;
        if (dt == 0) { x = (w >> 7) & 0xFF; sm[i] = uint8_t(((w >> 8) & 0x80) | (w & 0x7F)); }
        else if (dt == 1) { x = (w >> 10) & 0x1F; sm[i] = uint8_t(w); side[i] = uint16_t(((w >> 13) & 4) | ((w >> 8) & 3)); }
        else { x = (w >> 23) & 0xFF; sm[i] = uint8_t(((w >> 24) & 0x80) | ((w >> 16) & 0x7F)); smlo[2 * i] = uint8_t(w); smlo[2 * i + 1] = uint8_t(w >> 8); }
        y[i] = uint16_t((uint32_t(b) - x) & nmask);
    }
    for (; i < padded; ++i) { y[i] = 0; if (dt == 1) side[i] = 0; }
}

void put32(uint8_t* p, uint32_t v) { memcpy(p, &v, 4); }   // little-endian hosts only (x86)
void put64(uint8_t* p, uint64_t v) { memcpy(p, &v, 8); }

int default_threads() {
    const unsigned hw = std::thread::hardware_concurrency();
    return hw ? int(hw) : 1;
}

}  // namespace

extern "C" {

// Upper bound of the stream length: n = E, m = 1, every group wide.
size_t enec_cpu_max_compressed_size(int dt, size_t count) {
    if (dt < 0 || dt > 2 || (count >> 36)) return 0;
    const Shape s = shape_of(count);
    return layout_of(dt, count, s, exp_bits(dt), 1, s.groups).total;
}

// Returns the stream length, or 0 on an argument error. threads <= 0: all hardware threads.
size_t enec_cpu_compress(const void* in, int dt, size_t count, uint8_t* out, size_t capacity, int threads) {
    if (dt < 0 || dt > 2 || !out || (!in && count) || (count >> 36)) return 0;
    if (capacity < enec_cpu_max_compressed_size(dt, count)) return 0;
    if (threads <= 0) threads = default_threads();
    const int E = exp_bits(dt);
    const Shape s = shape_of(count);
    // phase 1: histogram of the exponent field, one partial histogram per worker
    std::vector<uint64_t> partial(size_t(threads) * 256, 0);
    parallel_blocks(s.nblocks, threads, [&](int t, uint32_t first, uint32_t last) {
        uint32_t h[4][256];
        memset(h, 0, sizeof(h));
        const size_t lo = size_t(first) * kBlock, hi = std::min(count, size_t(last) * kBlock);
        auto flush = [&] {
            for (int x = 0; x < 256; ++x) partial[size_t(t) * 256 + x] += uint64_t(h[0][x]) + h[1][x] + h[2][x] + h[3][x];
            memset(h, 0, sizeof(h));
        };
        size_t since = 0;
        for (size_t i = lo; i < hi; ++i) {
            const uint32_t w = word_at(in, dt, i);
            const uint32_t x = dt == 0 ? (w >> 7) & 0xFF : dt == 1 ? (w >> 10) & 0x1F : (w >> 23) & 0xFF;
            h[i & 3][x] += 1;
            if (++since == (1u << 31)) { flush(); since = 0; }
        }
        flush();
    });
    uint64_t hist[256] = {0};
    for (int t = 0; t < threads; ++t)
        for (int x = 0; x < 256; ++x) hist[x] += partial[size_t(t) * 256 + x];
    int b, n, m;
    choose_params(hist, E, &b, &n, &m);
    const int hbits = n - m;
    const size_t rec_bytes = size_t(2) * hbits;
    // phase 2: every block except the placement of its records, which needs the counts of the blocks before it
    const Layout L0 = layout_of(dt, count, s, n, m, 0);
    std::vector<uint32_t> wide_count(s.nblocks, 0);
    std::vector<uint8_t> staged(size_t(s.groups) * rec_bytes);
    uint8_t* mask = out + L0.mask;
    memset(out + L0.table, 0, L0.low - L0.table);  // table and mask (mask bits are OR-ed in per group)
    parallel_blocks(s.nblocks, threads, [&](int, uint32_t first_block, uint32_t last_block) {
        Scratch sc;
        uint16_t group[kGroup];
        for (uint32_t k = first_block; k < last_block; ++k) {
            const bool tail = k + 1 == s.nblocks;
            const uint32_t real = tail ? s.tail_real : kBlock, padded = tail ? s.tail_padded : kBlock;
            const size_t first = size_t(k) * kBlock;
            front_end(in, dt, first, real, padded, b, n, sc.y.data(), sc.side.data(), out + L0.sm + first,
                      dt == 2 ? out + L0.smlo + 2 * first : nullptr);
            const uint16_t keep = uint16_t((1u << m) - 1);
            for (uint32_t i = 0; i < padded; ++i) sc.lanes[i] = uint16_t(sc.y[i] & keep);
            pack_lanes(sc.lanes.data(), padded, m, sc.nb.data(), out + L0.low + size_t(k) * (kBlock / 8) * m);
            if (dt == 1) pack_lanes(sc.side.data(), padded, 3, sc.nb.data(), out + L0.smhi + size_t(k) * (kBlock / 8) * 3);
            // one group is one 256-bit vector: it is wide when any lane has a bit at or above m
            const __m256i above = _mm256_set1_epi16(short(~keep));
            uint8_t* rec = staged.data() + size_t(k) * kGroupsPerBlock * rec_bytes;
            uint32_t wide = 0;
            for (uint32_t g = 0; g < padded / kGroup; ++g) {
                const __m256i v = _mm256_loadu_si256(reinterpret_cast<const __m256i*>(sc.y.data() + g * kGroup));
                if (_mm256_testz_si256(v, above)) continue;
                const size_t gg = size_t(k) * kGroupsPerBlock + g;   // blocks of a worker are contiguous and a
                mask[gg >> 3] |= uint8_t(1u << (gg & 7));            // block is 128 mask bytes: no shared byte
                _mm256_storeu_si256(reinterpret_cast<__m256i*>(group), _mm256_srl_epi16(v, _mm_cvtsi32_si128(m)));
                pack_lanes(group, kGroup, hbits, sc.nb.data(), rec + size_t(wide) * rec_bytes);
                ++wide;
            }
            wide_count[k] = wide;
        }
    });
    // phase 3: prefix sum of the counts, records to their places, header
    std::vector<uint32_t> before(size_t(s.nblocks) + 1, 0);
    for (uint32_t k = 0; k < s.nblocks; ++k) before[k + 1] = before[k] + wide_count[k];
    const uint32_t wide_total = before[s.nblocks];
    const Layout L = layout_of(dt, count, s, n, m, wide_total);
    parallel_blocks(s.nblocks, threads, [&](int, uint32_t first_block, uint32_t last_block) {
        for (uint32_t k = first_block; k < last_block; ++k) {
            put32(out + L.table + 4 * size_t(k), before[k]);
            if (wide_count[k])
                memcpy(out + L.high + size_t(before[k]) * rec_bytes, staged.data() + size_t(k) * kGroupsPerBlock * rec_bytes,
                       size_t(wide_count[k]) * rec_bytes);
        }
    });
    put32(out + L.table + 4 * size_t(s.nblocks), wide_total);
    // zero the padding behind every section
    auto pad = [&](size_t from, size_t to) { if (to > from) memset(out + from, 0, to - from); };
    pad(L.low + size_t(s.padded) * m / 8, L.smhi);
    if (dt == 1) pad(L.smhi + size_t(s.padded) * 3 / 8, L.sm);
    pad(L.sm + count, L.smlo);
    if (dt == 2) pad(L.smlo + 2 * count, L.high);
    pad(L.high + size_t(wide_total) * rec_bytes, L.total);
    memset(out, 0, kHeader);
    memcpy(out, "ENEC", 4);
    out[4] = 1; out[6] = uint8_t(dt);
    put64(out + 8, count);
    put32(out + 16, kBlock);
    out[20] = uint8_t(b); out[21] = uint8_t(n); out[22] = uint8_t(m); out[23] = uint8_t(kGroup);
    put32(out + 24, s.nblocks);
    put32(out + 28, s.groups);
    put32(out + 32, wide_total);
    put64(out + 40, L.total);
    return L.total;
}

// Returns 0, or -1 when the stream does not describe `count` values of type dt.
int enec_cpu_decompress(const uint8_t* in, size_t in_size, int dt, size_t count, void* out, int threads) {
    if (dt < 0 || dt > 2 || !in || (!out && count) || in_size < kHeader + 16) return -1;
    if (threads <= 0) threads = default_threads();
    uint64_t h_count, h_total;
    uint32_t h_blocks, h_groups, h_wide, h_block;
    memcpy(&h_count, in + 8, 8); memcpy(&h_block, in + 16, 4); memcpy(&h_blocks, in + 24, 4);
    memcpy(&h_groups, in + 28, 4); memcpy(&h_wide, in + 32, 4); memcpy(&h_total, in + 40, 8);
    const int E = exp_bits(dt), b = in[20], n = in[21], m = in[22];
    const Shape s = shape_of(count);
    if (memcmp(in, "ENEC", 4) || in[4] != 1 || in[5] != 0 || in[6] != dt || h_count != count || h_block != kBlock ||
        in[23] != kGroup || n < 1 || n > E || m < 1 || m > n || b >= (1 << E) || h_blocks != s.nblocks ||
        h_groups != s.groups || h_wide > s.groups)
        return -1;
    const Layout L = layout_of(dt, count, s, n, m, h_wide);
    if (h_total != L.total || in_size < L.total) return -1;
    const int hbits = n - m;
    const size_t rec_bytes = size_t(2) * hbits;
    const uint32_t* table = reinterpret_cast<const uint32_t*>(in + L.table);
    int bad = 0;
    parallel_blocks(s.nblocks, threads, [&](int, uint32_t first_block, uint32_t last_block) {
        Scratch sc;
        uint16_t group[kGroup];
        const uint16_t sign = uint16_t(1u << (n - 1)), emask = uint16_t((1u << E) - 1);
        const uint16_t base = uint16_t(b + sign);
        for (uint32_t k = first_block; k < last_block; ++k) {
            const bool tail = k + 1 == s.nblocks;
            const uint32_t real = tail ? s.tail_real : kBlock, padded = tail ? s.tail_padded : kBlock;
            const size_t first = size_t(k) * kBlock;
            uint16_t* y = sc.y.data();
            unpack_lanes(in + L.low + size_t(k) * (kBlock / 8) * m, padded, m, y, sc.nb.data());
            if (dt == 1) unpack_lanes(in + L.smhi + size_t(k) * (kBlock / 8) * 3, padded, 3, sc.side.data(), sc.nb.data());
            uint32_t rank = table[k];
            if (table[k + 1] < rank || table[k + 1] - rank > padded / kGroup || table[k + 1] > h_wide) { bad = 1; continue; }
            for (uint32_t g = 0; g < padded / kGroup; ++g) {
                const size_t gg = size_t(k) * kGroupsPerBlock + g;
                if (!((in[L.mask + (gg >> 3)] >> (gg & 7)) & 1)) continue;
                if (rank >= table[k + 1]) { bad = 1; break; }
                unpack_lanes(in + L.high + size_t(rank) * rec_bytes, kGroup, hbits, group, sc.nb.data());
                for (uint32_t i = 0; i < kGroup; ++i) y[g * kGroup + i] = uint16_t(y[g * kGroup + i] | (group[i] << m));
                ++rank;
            }
            // x = (b - sext_n(y)) mod 2^E with sext_n(y) = (y ^ s) - s, s = 2^(n-1)   (Sec. 5.3)
            const uint8_t* sm = in + L.sm + first;
            if (dt == 0) {
                uint16_t* o = static_cast<uint16_t*>(out) + first;
                for (uint32_t i = 0; i < real; ++i) {
                    const uint16_t x = uint16_t((base - (y[i] ^ sign)) & emask);
                    o[i] = uint16_t(((sm[i] & 0x80) << 8) | (x << 7) | (sm[i] & 0x7F));
                }
            } else if (dt == 1) {
                uint16_t* o = static_cast<uint16_t*>(out) + first;
                const uint16_t* side = sc.side.data();
                for (uint32_t i = 0; i < real; ++i) {
                    const uint16_t x = uint16_t((base - (y[i] ^ sign)) & emask);
                    o[i] = uint16_t(((side[i] & 4) << 13) | (x << 10) | ((side[i] & 3) << 8) | sm[i]);
                }
            } else {
                uint32_t* o = static_cast<uint32_t*>(out) + first;
                const uint16_t* lo = reinterpret_cast<const uint16_t*>(in + L.smlo) + first;
                for (uint32_t i = 0; i < real; ++i) {
                    const uint32_t x = uint32_t(base - (y[i] ^ sign)) & emask;
                    o[i] = (uint32_t(sm[i] & 0x80) << 24) | (x << 23) | (uint32_t(sm[i] & 0x7F) << 16) | lo[i];
                }
            }
        }
    });
    return bad ? -1 : 0;
}

}  // extern "C"
