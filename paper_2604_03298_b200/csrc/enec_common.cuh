// Shared definitions of the CUDA codec: stream format, geometry, packed-byte helpers, async-copy and
// mbarrier wrappers. Used only by the CUDA library (the CPU oracle has its own, separate code).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "enec.h"

namespace enec {

constexpr uint32_t kBlockElems = 16384;  // elements per block (Sec. 6.4 "Data Block Size")
constexpr uint32_t kGroupElems = 16;     // L (Sec. 6.4 "Group Length")
constexpr uint32_t kGroupsPerBlock = kBlockElems / kGroupElems;
constexpr uint32_t kHeaderBytes = 64;
constexpr uint32_t kMagic = 0x43454E45u;  // "ENEC" little-endian
constexpr uint32_t kVersion = 1;

// 64-byte stream header (little-endian, natural alignment).
struct alignas(16) Header {
    uint32_t magic;         //  0
    uint16_t version;       //  4
    uint8_t dtype;          //  6
    uint8_t variant;        //  7: 0 = linear transform (Sec. 5.3), 1 = frequency ranks (Sec. 4.2, Algorithm 1),
                            //     2 = linear transform with parameters per block (block table)
    uint64_t count;         //  8
    uint32_t block;         // 16
    uint8_t b, n, m, L;     // 20..23
    uint32_t nblocks;       // 24
    uint32_t total_groups;  // 28
    uint32_t a_total;       // 32
    uint32_t pad1;          // 36
    uint64_t total_bytes;   // 40
    uint64_t pad2[2];       // 48
};
static_assert(sizeof(Header) == 64, "header is 64 bytes");

__host__ __device__ constexpr bool known_dtype(int dt) { return dt == ENEC_BF16 || dt == ENEC_FP16 || dt == ENEC_FP32; }
__host__ __device__ constexpr int exp_bits(int dt) { return dt == ENEC_FP16 ? 5 : 8; }
__host__ __device__ constexpr int elem_bytes(int dt) { return dt == ENEC_FP32 ? 4 : 2; }
__host__ __device__ inline uint64_t align16(uint64_t v) { return (v + 15) & ~uint64_t(15); }

struct Geometry {
    uint32_t nblocks;
    uint32_t tail_real;    // real elements of the last block
    uint32_t tail_padded;  // power of two >= max(16, tail_real)
    uint64_t padded_count;
    uint32_t total_groups;
};

__host__ __device__ inline Geometry make_geometry(uint64_t count) {
    Geometry g{0, 0, 0, 0, 0};
    if (count == 0) return g;
    g.nblocks = uint32_t((count + kBlockElems - 1) / kBlockElems);
    g.tail_real = uint32_t(count - uint64_t(g.nblocks - 1) * kBlockElems);
    uint32_t p = kGroupElems;
    while (p < g.tail_real) p <<= 1;
    g.tail_padded = p;
    g.padded_count = uint64_t(g.nblocks - 1) * kBlockElems + p;
    g.total_groups = uint32_t(g.padded_count / kGroupElems);
    return g;
}

constexpr uint32_t kRankTableBytes = 256;  // frequency-rank variant: rank -> exponent, behind the header

struct Sections {
    uint64_t unmap, table, mask, low, smhi, sm, smlo, high, total;
};

__host__ __device__ inline Sections make_sections(int dt, uint64_t count, const Geometry& g, int n, int m,
                                                  uint64_t a_total, bool ranked = false) {
    Sections s;
    s.unmap = kHeaderBytes;
    s.table = kHeaderBytes + (ranked ? kRankTableBytes : 0);
    s.mask = s.table + align16(4 * (uint64_t(g.nblocks) + 1));
    s.low = s.mask + align16((uint64_t(g.total_groups) + 7) / 8);
    s.smhi = s.low + align16(g.padded_count * uint64_t(m) / 8);
    s.sm = s.smhi + (dt == ENEC_FP16 ? align16(g.padded_count * 3 / 8) : 0);
    s.smlo = s.sm + align16(count);  // fp32 only: mantissa bits 15..0, two bytes per element
    s.high = s.smlo + (dt == ENEC_FP32 ? align16(count * 2) : 0);
    s.total = s.high + align16(a_total * 2 * uint64_t(n - m));
    return s;
}

// ---- device helpers -------------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return uint32_t(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after about a second and returns false; never spins forever.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < (1u << 22); ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (it > 32) __nanosleep(128);
    }
    return false;
}
// Bounded wait of any number of threads: each try suspends the thread for up to 20 us or until the phase
// completes, and there are at most 2^16 tries (about a second); also gives up when the CTA aborts.
__device__ __forceinline__ bool suspended_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    for (uint32_t it = 0; it < (1u << 16); ++it) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity), "r"(20000u)
            : "memory");
        if (ok) return true;
        if (*abort_flag) return false;
    }
    return false;
}

// Bulk asynchronous copy global -> this CTA's shared memory; completes on `bar` with `bytes` transferred.
// dst, src 16-byte aligned; bytes a positive multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// Asks for `bytes` of global memory to be brought into L2 (no destination, nothing to wait for).
// src 16-byte aligned; bytes a positive multiple of 16.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    return __byte_perm(a, b, sel);
}
__host__ __device__ constexpr uint32_t rep4(uint32_t byte) { return (byte & 0xFFu) * 0x01010101u; }

// Shared-memory accesses by 32-bit shared address (keeps address arithmetic in 32 bits).
__device__ __forceinline__ uint4 lds128(uint32_t a) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a));
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t a) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds32(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds16(uint32_t a) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ uint32_t lds8(uint32_t a) {
    uint32_t v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t a, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}

__device__ __forceinline__ void sts64(uint32_t a, uint2 v) {
    asm volatile("st.shared.v2.u32 [%0], {%1, %2};" ::"r"(a), "r"(v.x), "r"(v.y) : "memory");
}
__device__ __forceinline__ void sts8(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u8 [%0], %1;" ::"r"(a), "r"(v) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t a, uint32_t v) {
    asm volatile("st.shared.u16 [%0], %1;" ::"r"(a), "h"(uint16_t(v)) : "memory");
}

// Schedule of Algorithm 2 for fields of w bits: number of halvings until a lane holds at least a byte,
// and the bit reversal that orders the folded fields inside a lane.
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

// Programmatic dependent launch. A kernel launched with programmatic stream serialisation may start
// while the kernel before it in the stream is still running: pdl_wait() blocks until that kernel has
// finished and its memory is visible (it returns at once under an ordinary launch); everything that
// touches global memory comes after it. pdl_launch_dependents() lets the next kernel of the stream be
// scheduled into SM resources as they free up, so its launch latency hides behind this kernel's tail.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void report(int* status, int code) {
    if (status) atomicCAS(status, 0, code);
}

#endif  // __CUDACC__

}  // namespace enec
