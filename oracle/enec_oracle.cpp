/*
 * ENEC oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT (see enec_oracle.h).
 *
 * Plain scalar C++17, one thread, no blocking or fusion: every function takes the steps of the paper
 * in the paper's order. Build with -ffp-contract=off so Eq. 4 is evaluated in plain IEEE double.
 *
 * Stream layout (this repository's definition; little-endian; every section starts on a 16-byte
 * boundary and is zero padded):
 *   header 64 B | table u32[nblocks+1] | mask | low plane | (fp16: sm-hi plane) | sm plane |
 *   (fp32: sm-lo plane, mantissa bits 15..0, two bytes per element) | high records
 * Block-wise variant (header byte 7 = 2; Sec. 5.5 run on every block's own histogram): the table is replaced
 * by a block table of 16-byte entries {b, n, m, 0, u32 sum of m over the blocks before, u64 record bytes before},
 * nblocks + 1 of them (the last holds the totals); block k's low plane starts at 2048 x (sum of m before it)
 * and its records at (record bytes before it); header bytes 20..22 are zero.
 */
#include "enec_oracle.h"

#include <cstring>
#include <algorithm>
#include <utility>
#include <vector>

namespace {

constexpr uint32_t kBlock = 16384;  // Sec. 6.4 "Data Block Size": 16,384 elements per block
constexpr uint32_t kGroup = 16;     // Sec. 6.4 "Group Length": L = 16
constexpr size_t kHeaderBytes = 64;

enum { OK = 0, ERR_INVALID_ARG = -1, ERR_UNSUPPORTED_DTYPE = -2, ERR_BUFFER_TOO_SMALL = -3,
       ERR_BAD_STREAM = -4, ERR_PARAMS_NOT_LOSSLESS = -5 };

int exp_bits(int dtype) { return dtype == 1 ? 5 : 8; }  // bf16 and fp32: 8 exponent bits; fp16: 5

bool known_dtype(int dtype) { return dtype >= 0 && dtype <= 2; }

size_t align16(size_t v) { return (v + 15) & ~size_t(15); }

// Number of bits needed to write v (0 for v == 0): floor(log2 v) + 1.
int bit_width(uint64_t v) {
    int w = 0;
    while (v) { ++w; v >>= 1; }
    return w;
}

// ceil(log2 v) for v >= 2, and 0 for v <= 1 (reading of Eq. 1 where the logarithm is undefined).
int ceil_log2(uint64_t v) { return v <= 1 ? 0 : bit_width(v - 1); }

uint32_t next_pow2(uint32_t v) {
    uint32_t p = 1;
    while (p < v) p <<= 1;
    return p;
}

// Padded length of a block holding `real` elements: a power of two (Algorithm 2 needs N = 2^k),
// at least one group.
uint32_t padded_len(uint32_t real) {
    uint32_t p = next_pow2(real);
    return p < kGroup ? kGroup : p;
}

struct Geometry {
    uint32_t nblocks = 0;
    uint32_t tail_real = 0;     // real elements in the last block
    uint32_t tail_padded = 0;   // its padded length
    uint64_t padded_count = 0;  // sum of padded lengths
    uint32_t total_groups = 0;
};

Geometry geometry(size_t count) {
    Geometry g;
    if (count == 0) return g;
    g.nblocks = uint32_t((count + kBlock - 1) / kBlock);
    g.tail_real = uint32_t(count - size_t(g.nblocks - 1) * kBlock);
    g.tail_padded = padded_len(g.tail_real);
    g.padded_count = uint64_t(g.nblocks - 1) * kBlock + g.tail_padded;
    g.total_groups = uint32_t(g.padded_count / kGroup);
    return g;
}

struct Sections {
    size_t unmap, table, mask, low, smhi, sm, smlo, high, total;
};

// Section offsets for stored widths (n, m) and a_total anomalous groups. Streams of the frequency-rank variant
// carry a 256-byte table (rank -> exponent) between the header and the prefix table.
Sections sections(int dtype, size_t count, const Geometry& g, int n, int m, uint64_t a_total, bool ranked = false) {
    Sections s;
    s.unmap = kHeaderBytes;
    s.table = kHeaderBytes + (ranked ? 256 : 0);
    s.mask = s.table + align16(4 * (size_t(g.nblocks) + 1));
    s.low = s.mask + align16((size_t(g.total_groups) + 7) / 8);
    s.smhi = s.low + align16(size_t(g.padded_count) * m / 8);
    s.sm = s.smhi + (dtype == 1 ? align16(size_t(g.padded_count) * 3 / 8) : 0);
    s.smlo = s.sm + align16(count);
    s.high = s.smlo + (dtype == 2 ? align16(count * 2) : 0);
    s.total = s.high + align16(size_t(a_total) * 2 * (n - m));
    return s;
}

// Section offsets of the block-wise variant: low_bytes and high_bytes are the sums over the blocks.
Sections sections_blockwise(int dtype, size_t count, const Geometry& g, uint64_t low_bytes, uint64_t high_bytes) {
    Sections s;
    s.unmap = kHeaderBytes;
    s.table = kHeaderBytes;
    s.mask = s.table + align16(16 * (size_t(g.nblocks) + 1));
    s.low = s.mask + align16((size_t(g.total_groups) + 7) / 8);
    s.smhi = s.low + align16(size_t(low_bytes));
    s.sm = s.smhi + (dtype == 1 ? align16(size_t(g.padded_count) * 3 / 8) : 0);
    s.smlo = s.sm + align16(count);
    s.high = s.smlo + (dtype == 2 ? align16(count * 2) : 0);
    s.total = s.high + align16(size_t(high_bytes));
    return s;
}

void put_u16(uint8_t* p, uint16_t v) { p[0] = uint8_t(v); p[1] = uint8_t(v >> 8); }
void put_u32(uint8_t* p, uint32_t v) { for (int i = 0; i < 4; ++i) p[i] = uint8_t(v >> (8 * i)); }
void put_u64(uint8_t* p, uint64_t v) { for (int i = 0; i < 8; ++i) p[i] = uint8_t(v >> (8 * i)); }
uint16_t get_u16(const uint8_t* p) { return uint16_t(p[0] | (p[1] << 8)); }
uint32_t get_u32(const uint8_t* p) { uint32_t v = 0; for (int i = 0; i < 4; ++i) v |= uint32_t(p[i]) << (8 * i); return v; }
uint64_t get_u64(const uint8_t* p) { uint64_t v = 0; for (int i = 0; i < 8; ++i) v |= uint64_t(p[i]) << (8 * i); return v; }

// ---- Algorithm 2, hierarchical halving bit-packing with byte normalisation ----------------------
// Written as the recursion the text describes: a sub-block of lanes, each carrying `bits` payload bits, is
// folded (the upper half of the lanes moves above the payload of the lower half) until a lane holds at least a
// byte or one lane is left; the low byte of every lane is stored; whatever is above the byte forms the next
// sub-block, which goes through the same procedure.
void normalise_sub_block(std::vector<uint16_t> lanes, int bits, std::vector<uint8_t>& stored) {
    if (bits <= 0) return;
    while (lanes.size() > 1 && bits < 8) {
        const size_t keep = lanes.size() / 2;
        for (size_t lane = 0; lane < keep; ++lane)
            lanes[lane] = uint16_t(lanes[lane] | (lanes[keep + lane] << bits));
        lanes.resize(keep);
        bits *= 2;
    }
    std::vector<uint16_t> overflow;
    overflow.reserve(lanes.size());
    for (uint16_t v : lanes) {
        stored.push_back(uint8_t(v & 0xFF));
        overflow.push_back(uint16_t(v >> 8));
    }
    normalise_sub_block(std::move(overflow), bits - 8, stored);
}

std::vector<uint8_t> alg2_pack(const std::vector<uint16_t>& values, int a) {
    std::vector<uint8_t> stored;
    normalise_sub_block(values, a, stored);
    if (stored.size() % 2 != 0) stored.push_back(0);  // an even number of bytes: whole 16-bit words
    // last pass: 16-bit word i takes byte i as its low byte and byte i + half as its high byte; words are
    // written little-endian
    const size_t half = stored.size() / 2;
    std::vector<uint8_t> stream(stored.size());
    for (size_t i = 0; i < half; ++i) {
        stream[2 * i] = stored[i];
        stream[2 * i + 1] = stored[half + i];
    }
    return stream;
}

// Inverse of Algorithm 2: replay the forward schedule of folds and byte extractions, then undo the
// steps last to first.
std::vector<uint16_t> alg2_unpack(const uint8_t* stream, size_t N, int a) {
    struct Step { bool fold; size_t length; int width; size_t offset; };
    std::vector<Step> steps;
    size_t total_length = 0;
    {
        int width = a;
        size_t length = N;
        while (width > 0) {
            while (length > 1 && width < 8) {
                length /= 2;
                steps.push_back({true, length, width, 0});
                width *= 2;
            }
            steps.push_back({false, length, 0, total_length});
            width -= 8;
            total_length += length;
        }
        if (total_length % 2 != 0) total_length += 1;
    }
    // undo the final fold
    std::vector<uint8_t> normalized_bytes(total_length);
    size_t half = total_length / 2;
    for (size_t i = 0; i < half; ++i) {
        normalized_bytes[i] = stream[2 * i];
        normalized_bytes[i + half] = stream[2 * i + 1];
    }
    std::vector<uint16_t> data(N, 0);
    for (size_t s = steps.size(); s-- > 0;) {
        const Step& st = steps[s];
        if (st.fold) {
            uint16_t low_mask = uint16_t((1u << st.width) - 1);
            for (size_t i = 0; i < st.length; ++i) {
                data[i + st.length] = uint16_t(data[i] >> st.width);
                data[i] = uint16_t(data[i] & low_mask);
            }
        } else {
            for (size_t j = 0; j < st.length; ++j)
                data[j] = uint16_t((data[j] << 8) | normalized_bytes[st.offset + j]);
        }
    }
    return data;
}

// ---- Sec. 5.3 / Eq. 2 transform ---------------------------------------------------------------
uint32_t transform(uint32_t x, int b, int n) {
    uint32_t modulus = 1u << n;
    return (modulus - (x % modulus) + (uint32_t(b) % modulus)) % modulus;  // (2^n - x + b) % 2^n
}

uint32_t inverse_transform(uint32_t y, int b, int n, int E) {
    int32_t v = int32_t(y);
    if (y >> (n - 1)) v -= int32_t(1) << n;  // the top stored bit is the sign (Sec. 5.3)
    int32_t x = b - v;
    return uint32_t(x) & ((1u << E) - 1);
}

// ---- Eq. 1 -------------------------------------------------------------------------------------
int width_eq1(int b, int l, int h, int E) {
    int pos = bit_width(uint64_t(b - l));   // floor(log2(b - l)) + 1, 0 when b == l
    int neg = ceil_log2(uint64_t(h - b));   // ceil(log2(h - b)), 0 when h - b <= 1
    int n = (pos > neg ? pos : neg) + 1;
    if (n < 1) n = 1;
    if (n > E) n = E;  // the field itself has E bits; mod 2^E is already a bijection
    return n;
}

// ---- Sec. 5.5 phases 2 and 3 --------------------------------------------------------------------
void param_search(const uint64_t* hist, int E, int* b_out, int* n_out, int* m_out,
                  uint64_t* cost_out, double* bexp_out) {
    int bins = 1 << E;
    if (cost_out) for (int i = 0; i < bins; ++i) cost_out[i] = UINT64_MAX;
    if (bexp_out) for (int i = 0; i < 9; ++i) bexp_out[i] = 0.0;
    uint64_t total = 0;
    int l = -1, h = -1;
    for (int x = 0; x < bins; ++x) {
        if (hist[x]) { if (l < 0) l = x; h = x; }
        total += hist[x];
    }
    if (total == 0) { *b_out = 0; *n_out = 1; *m_out = 1; return; }

    // Phase 2: exhaustive search over b in [l, h]; minimise sum c[x] * y; ties -> smaller n, then smaller b.
    int best_b = -1, best_n = 0;
    uint64_t best_cost = 0;
    for (int b = l; b <= h; ++b) {
        int n = width_eq1(b, l, h, E);
        uint64_t cost = 0;
        for (int x = l; x <= h; ++x) cost += hist[x] * uint64_t(transform(uint32_t(x), b, n));
        if (cost_out) cost_out[b] = cost;
        if (best_b < 0 || cost < best_cost || (cost == best_cost && n < best_n)) {
            best_b = b; best_n = n; best_cost = cost;
        }
    }
    // Phase 3: threshold m at L = 16 by Eq. 4; ties -> smaller m.
    int best_m = 1;
    double best_bexp = 0.0;
    for (int m = 1; m <= best_n; ++m) {
        uint64_t cnt = 0;
        for (int x = l; x <= h; ++x)
            if (bit_width(transform(uint32_t(x), best_b, best_n)) <= m) cnt += hist[x];
        double p = double(cnt) / double(total);
        double p2 = p * p;
        double p4 = p2 * p2;
        double p8 = p4 * p4;
        double p16 = p8 * p8;
        double saving = double(m - best_n) * p16;
        double bexp = (double(best_n) + 0.0625) + saving;  // 1/L + n + (m - n) p(m)^L
        if (bexp_out) bexp_out[m] = bexp;
        if (m == 1 || bexp < best_bexp) { best_m = m; best_bexp = bexp; }
    }
    *b_out = best_b; *n_out = best_n; *m_out = best_m;
}

// ---- the frequency-rank variant (Sec. 4.2, Algorithm 1: E' = T_freq[E], "the sorted frequency indices serve as
// mapping values"; the ablation's V1 keeps that mapping and adds the one-bit group mask and Algorithm 2) ----
// rank_of[x] = position of exponent x when the occupied exponents are sorted by falling count (ties: smaller
// exponent first); unmap[r] = the exponent of rank r. The stored value of an element is its rank: no base, no
// sign bit, n = bits needed for the largest rank, m by Eq. 4 over the ranks' bit widths.
void rank_mapping(const uint64_t* hist, int E, uint8_t* rank_of, uint8_t* unmap, int* n_out, int* m_out) {
    const int bins = 1 << E;
    std::vector<int> order;
    uint64_t total = 0;
    for (int x = 0; x < bins; ++x) if (hist[x]) { order.push_back(x); total += hist[x]; }
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return hist[a] > hist[b]; });
    std::memset(rank_of, 0, 256);
    std::memset(unmap, 0, 256);
    for (size_t r = 0; r < order.size(); ++r) { rank_of[order[r]] = uint8_t(r); unmap[r] = uint8_t(order[r]); }
    int n = order.size() <= 1 ? 1 : bit_width(uint64_t(order.size() - 1));
    int best_m = 1;
    double best_bexp = 0.0;
    for (int m = 1; m <= n; ++m) {
        uint64_t cnt = 0;
        for (size_t r = 0; r < order.size(); ++r) if (bit_width(uint64_t(r)) <= m) cnt += hist[order[r]];
        double p = total ? double(cnt) / double(total) : 1.0;
        double p2 = p * p;
        double p4 = p2 * p2;
        double p8 = p4 * p4;
        double p16 = p8 * p8;
        double saving = double(m - n) * p16;
        double bexp = (double(n) + 0.0625) + saving;
        if (m == 1 || bexp < best_bexp) { best_m = m; best_bexp = bexp; }
    }
    *n_out = n; *m_out = best_m;
}

// Whether (b, n) reproduces every exponent in [l, h] (n == E always does).
bool params_lossless(int b, int n, int l, int h, int E) {
    if (n == E) return true;
    for (int x = l; x <= h; ++x)
        if (inverse_transform(transform(uint32_t(x), b, n), b, n, E) != uint32_t(x)) return false;
    return true;
}

// Sec. 4.2 "Split". fp32 keeps its 24 sign/mantissa bits as they are, as the text says of all formats; the
// exponent goes the same way as bf16's (Sec. 6.2: "we avoid compressing the mantissa").
void split(uint32_t w, int dtype, uint32_t* x, uint32_t* sm) {
    if (dtype == 2) { *x = (w >> 23) & 0xFF; *sm = ((w >> 8) & 0x800000) | (w & 0x7FFFFF); }
    else if (dtype == 0) { *x = (w >> 7) & 0xFF; *sm = ((w >> 8) & 0x80) | (w & 0x7F); }
    else            { *x = (w >> 10) & 0x1F; *sm = ((w >> 5) & 0x400) | (w & 0x3FF); }
}

uint32_t join(uint32_t x, uint32_t sm, int dtype) {
    if (dtype == 2) return ((sm & 0x800000) << 8) | (x << 23) | (sm & 0x7FFFFF);
    if (dtype == 0) return ((sm & 0x80) << 8) | (x << 7) | (sm & 0x7F);
    return ((sm & 0x400) << 5) | (x << 10) | (sm & 0x3FF);
}

// Element i of a tensor of 16-bit (bf16, fp16) or 32-bit (fp32) words.
uint32_t load_word(const void* in, int dtype, size_t i) {
    return dtype == 2 ? static_cast<const uint32_t*>(in)[i] : static_cast<const uint16_t*>(in)[i];
}

int encode(const void* in, int dtype, size_t count, bool have_params, int b, int n, int m,
           uint8_t* out, size_t capacity, size_t* out_size, bool ranked = false, bool blockwise = false) {
    if (!known_dtype(dtype)) return ERR_UNSUPPORTED_DTYPE;
    if ((!in && count) || !out || !out_size || (count >> 36)) return ERR_INVALID_ARG;
    const int E = exp_bits(dtype);
    const Geometry g = geometry(count);

    // step 1: split; phase 1: histogram of the exponent field
    std::vector<uint8_t> x(count);
    std::vector<uint32_t> sm(count);
    std::vector<uint64_t> hist(size_t(1) << E, 0);
    for (size_t i = 0; i < count; ++i) {
        uint32_t xe, s;
        split(load_word(in, dtype, i), dtype, &xe, &s);
        x[i] = uint8_t(xe); sm[i] = s;
        hist[xe] += 1;
    }
    uint8_t rank_of[256], unmap[256];
    if (blockwise) {
        if (have_params || ranked) return ERR_INVALID_ARG;
        b = 0; n = 1; m = 1;  // every block chooses its own below
    } else if (ranked) {
        if (have_params) return ERR_INVALID_ARG;
        rank_mapping(hist.data(), E, rank_of, unmap, &n, &m);
        b = 0;
    } else if (!have_params) {
        param_search(hist.data(), E, &b, &n, &m, nullptr, nullptr);
    } else {
        if (n < 1 || n > E || m < 1 || m > n || b < 0 || b >= (1 << E)) return ERR_INVALID_ARG;
        int l = -1, h = -1;
        for (int v = 0; v < (1 << E); ++v) if (hist[v]) { if (l < 0) l = v; h = v; }
        if (l >= 0 && !params_lossless(b, n, l, h, E)) return ERR_PARAMS_NOT_LOSSLESS;
    }

    // per block: transform, group flags, low plane, high records
    std::vector<uint32_t> table(size_t(g.nblocks) + 1, 0);
    std::vector<uint8_t> mask((size_t(g.total_groups) + 7) / 8, 0);
    std::vector<uint8_t> low, smhi, high;
    uint16_t low_mask = uint16_t((1u << m) - 1);
    uint32_t a_total = 0;
    std::vector<uint8_t> block_table(blockwise ? 16 * (size_t(g.nblocks) + 1) : 0, 0);
    uint32_t m_before = 0;
    for (uint32_t k = 0; k < g.nblocks; ++k) {
        size_t first = size_t(k) * kBlock;
        uint32_t real = (k + 1 == g.nblocks) ? g.tail_real : kBlock;
        uint32_t np = (k + 1 == g.nblocks) ? g.tail_padded : kBlock;
        if (blockwise) {
            // Sec. 5.5 on the histogram of this block's own (real) elements
            std::vector<uint64_t> block_hist(size_t(1) << E, 0);
            for (uint32_t i = 0; i < real; ++i) block_hist[x[first + i]] += 1;
            param_search(block_hist.data(), E, &b, &n, &m, nullptr, nullptr);
            low_mask = uint16_t((1u << m) - 1);
            uint8_t* e = block_table.data() + 16 * size_t(k);
            e[0] = uint8_t(b); e[1] = uint8_t(n); e[2] = uint8_t(m);
            put_u32(e + 4, m_before);
            put_u64(e + 8, high.size());
            m_before += uint32_t(m);
        }
        std::vector<uint16_t> y(np, 0), hi3(np, 0);  // padding: y = 0
        for (uint32_t i = 0; i < real; ++i) {
            y[i] = ranked ? uint16_t(rank_of[x[first + i]]) : uint16_t(transform(x[first + i], b, n));
            if (dtype == 1) hi3[i] = uint16_t(sm[first + i] >> 8);  // sign | mant[9:8]
        }
        table[k] = a_total;
        std::vector<uint16_t> lowvals(np);
        for (uint32_t i = 0; i < np; ++i) lowvals[i] = uint16_t(y[i] & low_mask);
        std::vector<uint8_t> packed = alg2_pack(lowvals, m);
        low.insert(low.end(), packed.begin(), packed.end());
        if (dtype == 1) {
            std::vector<uint8_t> p3 = alg2_pack(hi3, 3);
            smhi.insert(smhi.end(), p3.begin(), p3.end());
        }
        for (uint32_t gi = 0; gi < np / kGroup; ++gi) {
            uint16_t o = 0;
            for (uint32_t j = 0; j < kGroup; ++j) o = uint16_t(o | y[gi * kGroup + j]);
            if (o >> m) {  // bit width of the group's OR exceeds m
                size_t gg = size_t(k) * (kBlock / kGroup) + gi;
                mask[gg >> 3] = uint8_t(mask[gg >> 3] | (1u << (gg & 7)));
                std::vector<uint16_t> hv(kGroup);
                for (uint32_t j = 0; j < kGroup; ++j) hv[j] = uint16_t(y[gi * kGroup + j] >> m);
                std::vector<uint8_t> rec = alg2_pack(hv, n - m);
                high.insert(high.end(), rec.begin(), rec.end());
                a_total += 1;
            }
        }
    }
    table[g.nblocks] = a_total;
    if (blockwise) {
        uint8_t* e = block_table.data() + 16 * size_t(g.nblocks);
        put_u32(e + 4, m_before);
        put_u64(e + 8, high.size());
    }

    const Sections s = blockwise ? sections_blockwise(dtype, count, g, low.size(), high.size())
                                 : sections(dtype, count, g, n, m, a_total, ranked);
    *out_size = s.total;
    if (capacity < s.total) return ERR_BUFFER_TOO_SMALL;
    std::memset(out, 0, s.total);
    std::memcpy(out, "ENEC", 4);
    put_u16(out + 4, 1);
    out[6] = uint8_t(dtype);
    out[7] = blockwise ? 2 : ranked ? 1 : 0;  // variant: 0 = linear transform, 1 = frequency ranks, 2 = parameters per block
    if (blockwise) { b = 0; n = 0; m = 0; }
    if (ranked) std::memcpy(out + s.unmap, unmap, 256);
    put_u64(out + 8, count);
    put_u32(out + 16, kBlock);
    out[20] = uint8_t(b); out[21] = uint8_t(n); out[22] = uint8_t(m); out[23] = uint8_t(kGroup);
    put_u32(out + 24, g.nblocks);
    put_u32(out + 28, g.total_groups);
    put_u32(out + 32, a_total);
    put_u64(out + 40, s.total);
    if (blockwise) std::memcpy(out + s.table, block_table.data(), block_table.size());
    else for (size_t i = 0; i < table.size(); ++i) put_u32(out + s.table + 4 * i, table[i]);
    if (!mask.empty()) std::memcpy(out + s.mask, mask.data(), mask.size());
    if (!low.empty()) std::memcpy(out + s.low, low.data(), low.size());
    if (!smhi.empty()) std::memcpy(out + s.smhi, smhi.data(), smhi.size());
    if (dtype == 2) {
        // fp32: sign | mantissa bits 22..16 in the byte plane, mantissa bits 15..0 in the two-byte plane
        for (size_t i = 0; i < count; ++i) {
            out[s.sm + i] = uint8_t(sm[i] >> 16);
            put_u16(out + s.smlo + 2 * i, uint16_t(sm[i] & 0xFFFF));
        }
    } else {
        for (size_t i = 0; i < count; ++i) out[s.sm + i] = uint8_t(sm[i] & 0xFF);
    }
    if (!high.empty()) std::memcpy(out + s.high, high.data(), high.size());
    return OK;
}

int decode(const uint8_t* in, size_t in_size, int dtype, size_t count, void* out) {
    if (!known_dtype(dtype)) return ERR_UNSUPPORTED_DTYPE;
    if (!in || (!out && count)) return ERR_INVALID_ARG;
    if (in_size < kHeaderBytes + 16) return ERR_BAD_STREAM;
    if (std::memcmp(in, "ENEC", 4) != 0 || get_u16(in + 4) != 1) return ERR_BAD_STREAM;
    if (in[6] != dtype || get_u64(in + 8) != count || get_u32(in + 16) != kBlock || in[23] != kGroup)
        return ERR_BAD_STREAM;
    const int E = exp_bits(dtype);
    int b = in[20], n = in[21], m = in[22];
    if (in[7] > 2) return ERR_BAD_STREAM;
    const bool ranked = in[7] == 1, blockwise = in[7] == 2;
    if (!blockwise && (n < 1 || n > E || m < 1 || m > n || b >= (1 << E))) return ERR_BAD_STREAM;
    if (blockwise && (b || n || m)) return ERR_BAD_STREAM;
    const Geometry g = geometry(count);
    const uint32_t a_total = get_u32(in + 32);
    if (get_u32(in + 24) != g.nblocks || get_u32(in + 28) != g.total_groups) return ERR_BAD_STREAM;
    Sections s;
    if (blockwise) {
        // the block table's last entry holds the totals that fix the section sizes; the entries must chain
        const size_t table_bytes = 16 * (size_t(g.nblocks) + 1);
        if (in_size < kHeaderBytes + table_bytes) return ERR_BAD_STREAM;
        const uint8_t* t = in + kHeaderBytes;
        uint64_t m_sum = 0, high_sum = 0, low_sum = 0, wide_sum = 0;
        for (uint32_t k = 0; k < g.nblocks; ++k) {
            const uint8_t* e = t + 16 * size_t(k);
            const int bb = e[0], nn = e[1], mm = e[2];
            if (nn < 1 || nn > E || mm < 1 || mm > nn || bb >= (1 << E) || e[3]) return ERR_BAD_STREAM;
            if (get_u32(e + 4) != m_sum || get_u64(e + 8) != high_sum) return ERR_BAD_STREAM;
            const uint64_t next_high = get_u64(e + 24);
            const uint64_t rec = uint64_t(2) * (nn - mm);
            if (next_high < high_sum || (rec == 0 ? next_high != high_sum : (next_high - high_sum) % rec != 0)) return ERR_BAD_STREAM;
            wide_sum += rec ? (next_high - high_sum) / rec : 0;
            const uint32_t np = (k + 1 == g.nblocks) ? g.tail_padded : kBlock;
            low_sum += uint64_t(np) * mm / 8;
            m_sum += mm;
            high_sum = next_high;
        }
        const uint8_t* last = t + 16 * size_t(g.nblocks);
        if (last[0] || last[1] || last[2] || last[3] || get_u32(last + 4) != m_sum || get_u64(last + 8) != high_sum ||
            wide_sum != a_total)
            return ERR_BAD_STREAM;
        s = sections_blockwise(dtype, count, g, low_sum, high_sum);
    } else {
        s = sections(dtype, count, g, n, m, a_total, ranked);
    }
    if (get_u64(in + 40) != s.total || in_size < s.total) return ERR_BAD_STREAM;
    if (!blockwise && get_u32(in + s.table + 4 * size_t(g.nblocks)) != a_total) return ERR_BAD_STREAM;

    size_t rec_bytes = blockwise ? 0 : size_t(2) * (n - m);
    for (uint32_t k = 0; k < g.nblocks; ++k) {
        size_t first = size_t(k) * kBlock;
        uint32_t real = (k + 1 == g.nblocks) ? g.tail_real : kBlock;
        uint32_t np = (k + 1 == g.nblocks) ? g.tail_padded : kBlock;
        size_t low_at = s.low + size_t(k) * kBlock * m / 8;
        size_t high_at = s.high;     // of record number 0 (per tensor) or of the block's first record (per block)
        uint32_t rank, next;         // records before this block and before the next one, in the units of high_at
        if (blockwise) {
            const uint8_t* e = in + s.table + 16 * size_t(k);
            b = e[0]; n = e[1]; m = e[2];
            rec_bytes = size_t(2) * (n - m);
            low_at = s.low + size_t(2048) * get_u32(e + 4);
            high_at = s.high + get_u64(e + 8);
            rank = 0;
            next = rec_bytes ? uint32_t((get_u64(e + 24) - get_u64(e + 8)) / rec_bytes) : 0;
        } else {
            rank = get_u32(in + s.table + 4 * size_t(k));
            next = get_u32(in + s.table + 4 * size_t(k + 1));
        }
        std::vector<uint16_t> y = alg2_unpack(in + low_at, np, m);
        std::vector<uint16_t> hi3;
        if (dtype == 1) hi3 = alg2_unpack(in + s.smhi + size_t(k) * kBlock * 3 / 8, np, 3);
        for (uint32_t gi = 0; gi < np / kGroup; ++gi) {
            size_t gg = size_t(k) * (kBlock / kGroup) + gi;
            if ((in[s.mask + (gg >> 3)] >> (gg & 7)) & 1) {
                if (rank >= next || n == m) return ERR_BAD_STREAM;
                std::vector<uint16_t> hv = alg2_unpack(in + high_at + size_t(rank) * rec_bytes, kGroup, n - m);
                for (uint32_t j = 0; j < kGroup; ++j)
                    y[gi * kGroup + j] = uint16_t(y[gi * kGroup + j] | (hv[j] << m));
                rank += 1;
            }
        }
        if (rank != next) return ERR_BAD_STREAM;  // table must agree with the mask's popcount
        for (uint32_t i = 0; i < real; ++i) {
            uint32_t xe = ranked ? in[s.unmap + (y[i] & 0xFF)] : inverse_transform(y[i], b, n, E);
            uint32_t smv = in[s.sm + first + i];
            if (dtype == 1) smv |= uint32_t(hi3[i]) << 8;
            if (dtype == 2) {
                smv = (smv << 16) | get_u16(in + s.smlo + 2 * (first + i));
                static_cast<uint32_t*>(out)[first + i] = join(xe, smv, dtype);
            } else {
                static_cast<uint16_t*>(out)[first + i] = uint16_t(join(xe, smv, dtype));
            }
        }
    }
    return OK;
}

}  // namespace

extern "C" {

void enec_oracle_split(uint32_t w, int dtype, uint32_t* x, uint32_t* sm) { split(w, dtype, x, sm); }
uint32_t enec_oracle_join(uint32_t x, uint32_t sm, int dtype) { return join(x, sm, dtype); }
int enec_oracle_width_eq1(int b, int l, int h, int E) { return width_eq1(b, l, h, E); }
uint32_t enec_oracle_transform(uint32_t x, int b, int n) { return transform(x, b, n); }
uint32_t enec_oracle_inverse_transform(uint32_t y, int b, int n, int E) { return inverse_transform(y, b, n, E); }

void enec_oracle_param_search(const uint64_t* hist, int E, int* b, int* n, int* m, uint64_t* cost_out,
                              double* bexp_out) {
    param_search(hist, E, b, n, m, cost_out, bexp_out);
}

size_t enec_oracle_alg2_pack(const uint16_t* data, size_t N, int a, uint8_t* out) {
    std::vector<uint8_t> s = alg2_pack(std::vector<uint16_t>(data, data + N), a);
    std::memcpy(out, s.data(), s.size());
    return s.size();
}

void enec_oracle_alg2_unpack(const uint8_t* in, size_t N, int a, uint16_t* out) {
    std::vector<uint16_t> d = alg2_unpack(in, N, a);
    std::memcpy(out, d.data(), N * sizeof(uint16_t));
}

size_t enec_oracle_max_compressed_size(int dtype, size_t count) {
    if (!known_dtype(dtype) || (count >> 36)) return 0;
    const int E = exp_bits(dtype);
    const Geometry g = geometry(count);
    size_t worst = 0;  // widest stored width, every group anomalous, every split m
    for (int m = 1; m <= E; ++m) {
        size_t t = sections(dtype, count, g, E, m, g.total_groups).total;
        if (t > worst) worst = t;
    }
    return worst;
}

int enec_oracle_compress(const void* in, int dtype, size_t count, void* out, size_t capacity, size_t* out_size) {
    return encode(in, dtype, count, false, 0, 0, 0,
                  static_cast<uint8_t*>(out), capacity, out_size);
}

int enec_oracle_compress_with_params(const void* in, int dtype, size_t count, int b, int n, int m, void* out,
                                     size_t capacity, size_t* out_size) {
    return encode(in, dtype, count, true, b, n, m,
                  static_cast<uint8_t*>(out), capacity, out_size);
}

// The frequency-rank variant stores its 256-byte table on top of the same sections.
size_t enec_oracle_max_compressed_size_ranked(int dtype, size_t count) {
    const size_t base = enec_oracle_max_compressed_size(dtype, count);
    return base ? base + 256 : 0;
}

int enec_oracle_compress_ranked(const void* in, int dtype, size_t count, void* out, size_t capacity, size_t* out_size) {
    return encode(in, dtype, count, false, 0, 0, 0, static_cast<uint8_t*>(out), capacity, out_size, true);
}

// The block-wise variant: Sec. 5.5 on every block's own histogram; a 16-byte entry per block in place of the
// prefix table. Worst case: the per-tensor worst case with the larger table (a block's low plane and records
// together never exceed its elements times the exponent width, whatever its m).
size_t enec_oracle_max_compressed_size_blockwise(int dtype, size_t count) {
    if (!known_dtype(dtype) || (count >> 36)) return 0;
    const int E = exp_bits(dtype);
    const Geometry g = geometry(count);
    size_t worst = 0;
    for (int m = 1; m <= E; ++m) {
        const Sections s = sections_blockwise(dtype, count, g, size_t(g.padded_count) * m / 8,
                                              size_t(g.total_groups) * 2 * (E - m));
        if (s.total > worst) worst = s.total;
    }
    return worst + 32;  // per-block m can leave both variable sections with up to 15 padding bytes each
}

int enec_oracle_compress_blockwise(const void* in, int dtype, size_t count, void* out, size_t capacity, size_t* out_size) {
    return encode(in, dtype, count, false, 0, 0, 0, static_cast<uint8_t*>(out), capacity, out_size, false, true);
}

int enec_oracle_decompress(const void* in, size_t in_size, int dtype, size_t count, void* out) {
    return decode(static_cast<const uint8_t*>(in), in_size, dtype, count, out);
}

}  // extern "C"
