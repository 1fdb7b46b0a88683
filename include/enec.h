/*
 * libenec -- ENEC lossless codec for bf16/fp16 (and fp32) model weights on NVIDIA B200 (sm_100a).
 *
 * Block-based fixed-length coding: every 16-bit value is split into its exponent field and its
 * sign/mantissa bits (Sec. 4.2, Algorithm 1 "Split"); exponents go through the branch-free integer
 * transform y = (b - x) mod 2^n (Sec. 5.3, Eq. 2); each group of L = 16 transformed exponents is stored
 * with m bits per element, or with n bits when its OR needs more than m (Sec. 5.2); bits are packed with
 * hierarchical halving bit-packing (Algorithm 2); a prefix sum over the per-block counts of wide groups
 * gives every block's offset in the variable-length part of the stream (Sec. 5.1, Sec. 5.4); (b, n, m) are
 * chosen per tensor from the exponent histogram (Sec. 5.5, Eq. 1, 3, 4). fp32 values (32-bit words) take the same
 * path as bf16 with their high halves; their low halves are stored as they are (Sec. 6.2: the mantissa is not
 * compressed). `count` is always a number of elements.
 *
 * All pointers named d_* are DEVICE pointers, 16-byte aligned, owned by the caller. Every call only
 * enqueues work on `stream` and returns; nothing synchronises with the host. The current device's ordinal
 * must be below 64 (ENEC_ERR_CUDA otherwise). Errors the host can see
 * (null or misaligned pointers, unknown dtype, count >= 2^36, capacity below enec_max_compressed_size)
 * are returned at once. Errors only the device can see (damaged stream, parameters that are not
 * lossless, a wait that ran out) are written to *d_status if d_status is not NULL: the first error wins,
 * the value is one of enec_status, and it stays 0 when the call succeeded. The caller zeroes *d_status.
 * A kernel that finds an error stops touching the output; it never reads or writes out of range.
 *
 * The library keeps one small device scratch area per (device, stream) for the compressor (histogram
 * and control words); it is allocated on the first compress call on that stream and kept until exit.
 * The area carries state from one compress call on the stream to the next (that is what saves clearing it
 * every call), so: compress calls on ONE stream are issued by one host thread at a time, and
 * enec_compress / enec_compress_with_params / enec_compress_batched on a stream that is being captured into a
 * CUDA graph return ENEC_ERR_INVALID_ARG (a replay would not see the state). Decompression can be captured: what
 * it keeps per (device, stream) is one word that hands out the blocks of tensors of about 2^28 elements or more (allocated
 * with the first such call on the stream, numbered per launch, never relied on by a later call; if it cannot be
 * allocated the call does without it), and a call on a
 * capturing stream does without it; a batched call of more than 16 tensors is then recorded as one launch per 16 tensors, since
 * a longer list would have to pass through host and scratch memory that a replay cannot rely on.
 */
#ifndef ENEC_H
#define ENEC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum { ENEC_BF16 = 0, ENEC_FP16 = 1, ENEC_FP32 = 2 } enec_dtype;

typedef enum {
    ENEC_OK = 0,
    ENEC_ERR_INVALID_ARG = -1,
    ENEC_ERR_UNSUPPORTED_DTYPE = -2,
    ENEC_ERR_BUFFER_TOO_SMALL = -3,
    ENEC_ERR_BAD_STREAM = -4,
    ENEC_ERR_PARAMS_NOT_LOSSLESS = -5,
    ENEC_ERR_TIMEOUT = -6,
    ENEC_ERR_CUDA = -7,
    ENEC_ERR_TOO_LARGE = -8
} enec_status;

/* Same type as cudaStream_t; spelled out so that this header needs no CUDA header. */
typedef struct CUstream_st* enec_stream_t;

/*
 * Upper bound, in bytes, of the stream enec_compress writes for `count` elements of `dt`: the stream
 * layout (64-byte header, per-block prefix table, group mask, low plane, fp16 sign/mantissa-high plane,
 * sign/mantissa byte plane, wide-group records; every section padded to 16 bytes) with n = exponent
 * width, every group wide, maximised over m. Pure host function. Returns 0 for an unknown dtype or
 * count >= 2^36.
 */
size_t enec_max_compressed_size(enec_dtype dt, size_t count);

/*
 * Compress `count` elements of type `dt` at d_in into d_out (Sec. 5.1 compression flow: split, histogram and
 * parameter choice of Sec. 5.5, transform of Sec. 5.3, group widths of Sec. 5.2, Algorithm 2 packing,
 * block-offset prefix sum). out_capacity must be at least enec_max_compressed_size(dt, count).
 * d_out_size (device, 8-byte aligned, may be NULL) receives the stream length, which is also in the
 * stream header. count == 0 is valid and gives a header-plus-table stream of 80 bytes.
 */
enec_status enec_compress(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                          size_t* d_out_size, int* d_status, enec_stream_t stream);

/*
 * As enec_compress, with the caller's (b, n, m) instead of the search of Sec. 5.5 (the paper's offline
 * tuned mode, Sec. 6 "Compression Configurations"). 0 <= b < 2^E, 1 <= m <= n <= E (E = 8 for bf16,
 * 5 for fp16). If some exponent of the tensor does not survive (b, n) the device reports
 * ENEC_ERR_PARAMS_NOT_LOSSLESS in *d_status and writes no stream.
 */
enec_status enec_compress_with_params(const void* d_in, enec_dtype dt, size_t count, int b, int n, int m,
                                      void* d_out, size_t out_capacity, size_t* d_out_size, int* d_status,
                                      enec_stream_t stream);

/*
 * Decompress the stream at d_in (in_size bytes) into `count` elements of type `dt` at d_out (Sec. 5.1
 * decompression flow: mask -> prefix sums -> unpack low and high parts -> inverse transform -> rejoin
 * with sign/mantissa). dt and count must match the stream header, else ENEC_ERR_BAD_STREAM is reported in
 * *d_status. The result is bit-identical to the tensor that was compressed.
 */
enec_status enec_decompress(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                            int* d_status, enec_stream_t stream);

/*
 * The frequency-rank variant of enec_compress, kept for the ablation (Sec. 4.2, Algorithm 1 "E' = T_freq[E]";
 * Sec. 6.6 calls the version with this mapping, the one-bit group mask and Algorithm 2 "V1"): the stored value
 * of an element is the rank of its exponent when the tensor's exponents are sorted by falling count (ties:
 * smaller exponent first), n is the bit width of the largest rank and m follows Eq. 4; there is no base b and
 * no sign bit. The stream has header byte 7 = 1 and a 256-byte table (rank -> exponent) between the header and
 * the prefix table; everything else is laid out as by enec_compress. out_capacity must be at least
 * enec_max_compressed_size_ranked(dt, count) (256 bytes more than enec_max_compressed_size).
 * Such a stream is decoded by enec_decompress_ranked (same arguments as enec_decompress); each of the two
 * decompress calls reports ENEC_ERR_BAD_STREAM in *d_status for the other kind of stream, and
 * enec_decompress_batched takes streams of enec_compress only.
 */
size_t enec_max_compressed_size_ranked(enec_dtype dt, size_t count);
enec_status enec_compress_ranked(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                                 size_t* d_out_size, int* d_status, enec_stream_t stream);
enec_status enec_decompress_ranked(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                                   int* d_status, enec_stream_t stream);

/*
 * The block-wise variant of enec_compress, kept for the ablation: the search of Sec. 5.5 (Eq. 1-5) runs on the
 * exponent histogram of every 16384-element block instead of the tensor's, so each block is coded with its own
 * (b, n, m). (Sec. 6.4 and Table 6 measure how little is lost by sharing parameters; this variant measures the
 * other end of that trade on the GPU.) The stream has header byte 7 = 2 and header bytes 20..22 zero; in place of
 * the prefix table it carries a block table of 16-byte entries, one per block plus one with the totals:
 *   byte 0 b, byte 1 n, byte 2 m, byte 3 zero,
 *   bytes 4..7   u32: sum of m over the blocks before (the block's low plane starts 2048 x that many bytes into
 *                the low-plane section),
 *   bytes 8..15  u64: bytes of wide-group records before the block's first record;
 * header bytes 32..35 hold the number of wide groups of the tensor. Every other section is laid out as by
 * enec_compress. out_capacity must be at least enec_max_compressed_size_blockwise(dt, count). The arguments,
 * the scratch rule, the stream-capture rule (refused with ENEC_ERR_INVALID_ARG) and the error behaviour are those
 * of enec_compress. Such a stream is decoded by enec_decompress_blockwise (same arguments as enec_decompress);
 * every decompress call reports ENEC_ERR_BAD_STREAM in *d_status for a stream of another variant.
 */
size_t enec_max_compressed_size_blockwise(enec_dtype dt, size_t count);
enec_status enec_compress_blockwise(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                                    size_t* d_out_size, int* d_status, enec_stream_t stream);
enec_status enec_decompress_blockwise(const void* d_in, size_t in_size, enec_dtype dt, size_t count, void* d_out,
                                      int* d_status, enec_stream_t stream);

/* One tensor of a batch. All pointers are device pointers. */
typedef struct {
    const void* d_in;    /* decompress: stream; compress: raw values            */
    void* d_out;         /* decompress: raw values; compress: stream            */
    size_t count;        /* elements                                            */
    size_t size;         /* decompress: stream bytes; compress: output capacity */
} enec_batch_item;

/*
 * Decompress n_items streams of one dtype with a single launch (one entry per tensor, in HOST memory;
 * the call copies the descriptors to the device on `stream`; the paper's interface has no batch, and host
 * arrays spare the caller a device copy of its own). Meant for checkpoints made of many small tensors, where
 * one launch per tensor would be launch-bound. Same per-tensor semantics as enec_decompress, for tensors
 * without elements too (their 80-byte streams are checked); *d_status holds the first error of any tensor.
 */
enec_status enec_decompress_batched(const enec_batch_item* h_items, int n_items, enec_dtype dt, int* d_status,
                                    enec_stream_t stream);

/*
 * Compress n_items tensors of one dtype with two launches (the histograms and parameter searches of all
 * tensors, then the encode of all their blocks), each tensor into a stream of its own exactly as
 * enec_compress would write it. Entries in HOST memory: d_in = values, d_out = stream buffer, count =
 * elements, size = capacity of d_out (at least enec_max_compressed_size(dt, count)). d_out_sizes (device
 * array of n_items 8-byte words, may be NULL) receives the stream lengths. Meant for checkpoints made of
 * many small tensors; the same conventions as enec_decompress_batched. Output buffers must not overlap.
 */
enec_status enec_compress_batched(const enec_batch_item* h_items, int n_items, enec_dtype dt, size_t* d_out_sizes,
                                  int* d_status, enec_stream_t stream);

/*
 * enec_compress for callers that must not allocate device memory. (The paper has no counterpart: this is
 * a property of this library's interface, not of the codec.)
 *
 * enec_compress keeps its working memory (a histogram, a few control words and one 8-byte word per
 * 16384-value block) in an area it allocates with cudaMalloc the first time a stream is used, and again
 * when a larger tensor arrives. Some callers cannot have that: code that runs inside a memory pool or a
 * caching allocator which owns all device memory and must see every allocation, code in a phase where a
 * cudaMalloc would stall other streams (it synchronises the device), and services that have handed the
 * whole device budget to something else. For them this entry point takes its working memory from a
 * fixed array inside the library image (ENEC_NOALLOC_SCRATCH_BYTES, about 0.5 MB, present on every GPU
 * that loads the library for as long as the process lives) and makes no cudaMalloc or cudaFree call of its
 * own, nor a call of a library routine that allocates (what the driver does when it first loads a kernel's
 * code is outside the library's hands); enec_allocation_count() lets a caller check.
 *
 * Same arguments, stream format and output as enec_compress (the two write identical bytes). Limits and
 * rules that differ:
 *   - count may be at most ENEC_NOALLOC_MAX_COUNT (2^30 values, 2 GiB of bf16); more is refused with
 *     ENEC_ERR_TOO_LARGE before anything is enqueued. Split larger tensors or use enec_compress.
 *   - All calls on a device share the one array, whatever their stream. Each call begins by clearing the
 *     part it uses, so calls that follow one another on a stream are fine; two calls whose work overlaps
 *     on the GPU (different streams without an ordering between them) corrupt each other's state.
 *   - The first call on each device looks up the array's device address, with that device current. Make
 *     that first call outside any stream capture.
 */
#define ENEC_NOALLOC_MAX_COUNT ((size_t)1 << 30)
#define ENEC_NOALLOC_SCRATCH_BYTES (8192 + (ENEC_NOALLOC_MAX_COUNT / 16384) * 8)
enec_status enec_compress_noalloc(const void* d_in, enec_dtype dt, size_t count, void* d_out, size_t out_capacity,
                                  size_t* d_out_size, int* d_status, enec_stream_t stream);

/* Number of kernels the library has launched in this process (all entry points, all streams). */
uint64_t enec_launch_count(void);

/* Number of cudaMalloc calls the library has made in this process (scratch areas; never freed before exit). */
uint64_t enec_allocation_count(void);

/* Library version: 10000 * major + 100 * minor + patch. */
int enec_version(void);

#ifdef __cplusplus
}
#endif
#endif /* ENEC_H */
