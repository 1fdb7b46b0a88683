/*
 * ENEC oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, single-threaded, scalar CPU encoder/decoder of the ENEC codec (block-based fixed-length
 * lossless coding of bf16/fp16 weights), written step by step from the paper. It exists to check the
 * CUDA library and to be timed as a CPU baseline. Only tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it; the product (the CUDA library) shares no code with it.
 *
 * Pinned by the CPU test-suite: Sec. 5.3 worked example, Eq. 1 hand values, Algorithm 2 brute force and
 * library special cases, closed-form sizes, hand-built streams, all 2^16 bit patterns.
 * Parity unpinned: the byte layout of the authors' own compressed files (the stream-layout figure is
 * not available); the layout here is this repository's own definition.
 */
#ifndef ENEC_ORACLE_H
#define ENEC_ORACLE_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* dtype: 0 = bf16, 1 = fp16, 2 = fp32 (32-bit words). Status: 0 ok, negative = error (same numbering as the CUDA library). */

/* Sec. 4.2 "Split": exponent field and sign/mantissa remainder of one word (16 bits, or 32 for fp32). */
void enec_oracle_split(uint32_t w, int dtype, uint32_t* x, uint32_t* sm);
uint32_t enec_oracle_join(uint32_t x, uint32_t sm, int dtype);

/* Eq. 1: stored width n (sign bit included) for mapping parameter b and occupied range [l, h]. */
int enec_oracle_width_eq1(int b, int l, int h, int E);
/* Eq. 2: y = (b - x) mod 2^n.  Inverse: x = (b - sext_n(y)) mod 2^E. */
uint32_t enec_oracle_transform(uint32_t x, int b, int n);
uint32_t enec_oracle_inverse_transform(uint32_t y, int b, int n, int E);

/* Sec. 5.5 phases 2 and 3 on a 2^E-bin histogram. cost_out[b] = sum c[x]*y (Eq. 3 times N) for every
 * candidate b (others left at UINT64_MAX); bexp_out[m] = Eq. 4 at L = 16 for m in 1..n (index 0 unused). */
void enec_oracle_param_search(const uint64_t* hist, int E, int* b, int* n, int* m,
                              uint64_t* cost_out /* [2^E] or NULL */, double* bexp_out /* [9] or NULL */);

/* Algorithm 2 and its inverse. N a power of two, 0 < a <= 8. pack returns the byte count written. */
size_t enec_oracle_alg2_pack(const uint16_t* data, size_t N, int a, uint8_t* out);
void enec_oracle_alg2_unpack(const uint8_t* in, size_t N, int a, uint16_t* out);

/* Whole codec over host memory. */
size_t enec_oracle_max_compressed_size(int dtype, size_t count);
/* The frequency-rank variant (Sec. 4.2, Algorithm 1; the ablation's V1): stored value = rank of the exponent by
 * falling frequency; header byte 7 = 1; a 256-byte rank -> exponent table follows the header. */
size_t enec_oracle_max_compressed_size_ranked(int dtype, size_t count);
int enec_oracle_compress_ranked(const void* in, int dtype, size_t count, void* out, size_t capacity, size_t* out_size);

/* The block-wise variant (Sec. 5.5 run on every block's own histogram): header byte 7 = 2; a block table of
 * 16-byte entries {b, n, m, 0, u32 sum of m before, u64 record bytes before} replaces the prefix table. */
size_t enec_oracle_max_compressed_size_blockwise(int dtype, size_t count);
int enec_oracle_compress_blockwise(const void* in, int dtype, size_t count, void* out, size_t capacity, size_t* out_size);

int enec_oracle_compress(const void* in, int dtype, size_t count, void* out, size_t capacity,
                         size_t* out_size);
int enec_oracle_compress_with_params(const void* in, int dtype, size_t count, int b, int n, int m,
                                     void* out, size_t capacity, size_t* out_size);
int enec_oracle_decompress(const void* in, size_t in_size, int dtype, size_t count, void* out);

#ifdef __cplusplus
}
#endif
#endif
