/*
 * llms.h - C ABI of the B200 chunk-wise KV-cache codec and tolerance score.
 *
 * The library implements the data-parallel part of context switching in LLMS
 * ("LLM as a System Service on Mobile Devices", arXiv 2403.11805): per-chunk
 * quantize + bit-pack on swap-out, unpack + dequantize on swap-in, the per-chunk
 * information density that ranks chunks, the rank -> bit-width rule, the LCTRU
 * eviction order and the copy of packed records to and from pinned host memory.
 *
 * Conventions
 *  - Every function returns LLMS_OK (0) or a negative llms_status.  Arguments are
 *    checked on the host before anything is enqueued; after an argument error
 *    nothing has been launched or written.
 *  - "device" pointers are CUDA device addresses of the current device, "host"
 *    pointers are ordinary host addresses, "pinned" means page-locked host memory.
 *  - The library never allocates or frees device or pinned memory.  Scratch
 *    ("workspace") is passed in by the caller.
 *  - Device work is enqueued on the given stream (a cudaStream_t passed as void*;
 *    NULL is the legacy default stream) and the call returns without synchronising.
 *    Host arrays passed in are consumed before the call returns unless stated.
 *  - fp16 values are IEEE binary16; multi-byte fields in records are little-endian.
 *
 * KV layout.  Element (l, s, h, t, c) - layer, 0 = K / 1 = V, KV head, token,
 * channel - lives at  l*stride_l + s*stride_s + h*stride_h + t*head_dim + c
 * (strides in elements).  A *chunk* i is tokens [i*chunk_len, (i+1)*chunk_len) of
 * every layer, of K and V, of every head (Sec. 3.1: chunks hold the same number of
 * tokens and carry one compression ratio each); floor(n_tokens / chunk_len)
 * chunks exist and a shorter tail is not a chunk.  A *slab* is the chunk's
 * chunk_len*head_dim contiguous elements of one (l, s, h); slabs are numbered
 * s_idx = (l*2 + s)*n_kv_heads + h.  A descriptor may equally describe a pool of
 * chunk slots: chunk ids are then slot numbers.
 *
 * Record of one chunk at bit-width b (Sec. 3.2 "Compressing chunks": linear
 * quantization to a lower bit-width; Sec. 4: sub-byte codes packed with bit shifts):
 *     [ n_groups x { u16 scale (fp16 bits), u16 zero-point (fp16 bits) } ]
 *     zero bytes up to a multiple of 16
 *     [ codes: element e of the chunk, in memory order (slab, token, channel),
 *       occupies bits [e*b, (e+1)*b) of a little-endian bit stream ]
 *     zero bytes up to a multiple of 256
 * quant_mode 0: a group is group_size consecutive channels of one token of one
 * slab (group index = (s_idx*chunk_len + t)*(head_dim/group_size) + j).
 * quant_mode 1: a group is one channel of one slab across the chunk's tokens
 * (group index = s_idx*head_dim + c), the paper's "channel-wise" wording.
 * Per group, in binary32 with IEEE round-to-nearest and no fused operations:
 *     zero = min x (stored as +0 when it is a zero);  scale = fp16((max x - min x) / (2^b - 1)), 65504 if larger;
 *     code = min(2^b - 1, rint((x - zero) * (1 / scale)))  (ties to even; all codes 0 when scale == 0);
 *     decoded value = fp16(clamp(zero + code*scale, -65504, 65504)).
 * Inputs must be finite.
 */
#ifndef LLMS_H
#define LLMS_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum llms_status {
    LLMS_OK = 0,
    LLMS_ERR_INVALID_ARG = -1,   /* null pointer, non-positive size, id out of range, duplicate chunk id */
    LLMS_ERR_BAD_BITS = -2,      /* a bit-width other than 1, 2, 4, 8 */
    LLMS_ERR_MISALIGNED = -3,    /* pointer, stride or offset not aligned as required */
    LLMS_ERR_BUF_TOO_SMALL = -4, /* output buffer or workspace smaller than needed */
    LLMS_ERR_CUDA = -5,          /* a CUDA runtime call failed (see llms_last_cuda_error) */
    LLMS_ERR_TIMEOUT = -6,       /* llms_wait ran out of time */
    LLMS_ERR_CORRUPT = -7,       /* a record's checksum does not match */
    LLMS_ERR_UNSUPPORTED = -8    /* valid in the format but not implemented by the kernels */
} llms_status;

/* Shape of a KV tensor (or slot pool) and of the codec applied to it.
 * Requirements of the codec kernels: head_dim a multiple of 16; for quant_mode 0,
 * group_size a power of two in [16, 512] dividing head_dim; strides multiples of 8
 * elements; n_q_heads a multiple of n_kv_heads. */
typedef struct llms_kv_desc {
    int32_t n_layers, n_kv_heads, n_q_heads, head_dim;
    int32_t n_tokens, chunk_len, group_size, quant_mode;
    int64_t stride_l, stride_s, stride_h;
} llms_kv_desc;

/* One record of a swap buffer: where it is and what is in it (32 bytes). */
typedef struct llms_chunk_meta {
    uint32_t chunk_id;  /* chunk (slot) the record was made from */
    uint32_t bits;      /* 1, 2, 4 or 8 */
    uint64_t offset;    /* byte offset of the record in its swap buffer, multiple of 256 */
    uint64_t nbytes;    /* record size, multiple of 256 */
    uint32_t n_groups;
    uint32_t checksum;  /* sum of the record's little-endian u32 words, mod 2^32 */
} llms_chunk_meta;

/* One row of the host-side chunk table that the LCTRU order is taken over. */
typedef struct llms_chunk_state {
    uint32_t ctx_id, chunk_id, bits;
    uint32_t resident;  /* non-zero: in device memory */
    uint32_t locked;    /* non-zero: its context is being served (working-set lock) */
    uint32_t pad_;
    uint64_t last_access_step;
} llms_chunk_state;

const char *llms_strerror(int status);
/* Text of the last CUDA error a call of this thread ran into ("" if none). */
const char *llms_last_cuda_error(void);

/* ------------------------------------------------------------------ sizes (host only) */

/* Record layout at `bits`: byte offset of the code stream inside the record and the
 * padded record size (see the layout above).  Either output may be NULL. */
int llms_record_layout(const llms_kv_desc *desc, int bits, uint64_t *codes_offset, uint64_t *nbytes);
int llms_record_bytes(const llms_kv_desc *desc, int bits, uint64_t *nbytes);
/* Sum of the record sizes of n chunks with the given bit-widths (host array). */
int llms_compressed_size(const llms_kv_desc *desc, const uint8_t *bits, int n, uint64_t *nbytes);
/* Device scratch needed by llms_compress_chunks / llms_decompress_chunks for n chunks. */
int llms_codec_workspace_bytes(int n, uint64_t *nbytes);

/* ------------------------------------------------------------------ swap-out: quantize + pack */

/* Reclaim's compression half (Sec. 3.1 primitives; Sec. 3.2; Sec. 4).
 * For i < n: chunk chunk_ids[i] of `kv` is quantized at bits[i] bits and its record is laid
 * down in out_buf at the running offset (records in list order, each 256-byte aligned).
 *   kv         device, fp16, 16-byte aligned, read only
 *   chunk_ids  host, n distinct ids < floor(n_tokens/chunk_len)
 *   bits       host, n values from {1, 2, 4, 8}
 *   out_buf    device, 256-byte aligned, out_bytes >= llms_compressed_size(...); every byte of
 *              every record, padding included, is written
 *   meta       host, n entries, filled before return except `checksum`, which the device
 *              computes: it reaches meta[] in stream order, so it is valid once the stream has
 *              been synchronised.  Into pinned (page-locked) memory a kernel stores it, which
 *              neither blocks the call nor waits for copies other streams have in flight; into
 *              pageable memory it is copied, and the call may block until the kernel is done
 *   workspace  device, 16-byte aligned, llms_codec_workspace_bytes(n); may be reused by the
 *              next call on the same stream
 * n == 0 is valid and does nothing. */
int llms_compress_chunks(const llms_kv_desc *desc, const void *kv, const uint32_t *chunk_ids,
                         const uint8_t *bits, int n, void *out_buf, uint64_t out_bytes,
                         llms_chunk_meta *meta, void *workspace, uint64_t workspace_bytes, void *stream);

/* llms_compress_chunks without a workspace argument, for callers that cannot obtain device scratch:
 * a service that handed all device memory to its KV pool at start-up (an allocation would fail, or
 * would stall inference because cudaMalloc synchronises the device), or code running where the CUDA
 * allocator must not be entered at all.  The paper has no counterpart to this call; it is a
 * convenience of this library.  The chunk table lives in a fixed array inside the library image
 * (about 64 KiB, present on every GPU that loads the library until the process exits), which limits
 * one call to LLMS_STATIC_MAX_CHUNKS chunks: a larger n returns LLMS_ERR_BUF_TOO_SMALL and nothing
 * is launched.  No device memory is allocated or freed.  All other arguments, results and errors
 * are those of llms_compress_chunks.
 * The first call on each device looks up the array's device address (with that device current);
 * make that first call outside of any stream capture.  Every call on a device uses the same array
 * and overwrites what the previous call left in it, so two calls whose GPU work may overlap (different
 * streams, different threads) race on it: order them on one stream or with events. */
#define LLMS_STATIC_MAX_CHUNKS 1024
int llms_compress_chunks_static(const llms_kv_desc *desc, const void *kv, const uint32_t *chunk_ids,
                                const uint8_t *bits, int n, void *out_buf, uint64_t out_bytes,
                                llms_chunk_meta *meta, void *stream);

/* ------------------------------------------------------------------ swap-in: unpack + dequantize */

/* Load's decompression half.  Record i (meta[i], inside `buf`) is decoded into chunk slot
 * dst_chunk_ids[i] of kv_out (dst_chunk_ids == NULL: meta[i].chunk_id).  Other chunks of kv_out
 * are not touched.  While decoding, each record's checksum is recomputed; the number of
 * records whose sum differs from meta[i].checksum is left in the workspace and can be read
 * with llms_codec_corrupt_count (decoded values of such a record are still written).
 *   buf        device, 256-byte aligned, buf_bytes long: a record that does not lie inside it
 *              (meta[i].offset + meta[i].nbytes > buf_bytes) is refused with LLMS_ERR_BUF_TOO_SMALL
 *              before anything is launched, so a stale or damaged meta table cannot turn into a read
 *              outside the buffer;  meta, dst_chunk_ids  host;  kv_out  device fp16
 * Everything in meta, the expected checksums included, is read when the call is made. */
int llms_decompress_chunks(const llms_kv_desc *desc, const void *buf, uint64_t buf_bytes, const llms_chunk_meta *meta,
                           const uint32_t *dst_chunk_ids, int n, void *kv_out,
                           void *workspace, uint64_t workspace_bytes, void *stream);

/* The same with the expected checksums taken in stream order: meta must lie in page-locked (pinned) host
 * memory (else LLMS_ERR_INVALID_ARG); sizes, offsets and bit-widths are read when the call is made, but
 * meta[i].checksum is read by the device itself when the check runs on `stream`.  Such a call may follow,
 * on the same stream and without a synchronisation in between, the llms_compress_chunks call that is still
 * producing those checksums into the same array.  The host must neither free nor change the array (a new
 * llms_compress_chunks into it changes it) until the stream has passed this call. */
int llms_decompress_chunks_ordered(const llms_kv_desc *desc, const void *buf, uint64_t buf_bytes, const llms_chunk_meta *meta,
                                   const uint32_t *dst_chunk_ids, int n, void *kv_out,
                                   void *workspace, uint64_t workspace_bytes, void *stream);

/* Synchronises `stream`, then reports on the last llms_decompress_chunks that used this workspace:
 * LLMS_ERR_CORRUPT if a decoded record's checksum did not match, else LLMS_OK; *n_corrupt (host, may
 * be NULL) receives the number of such records. */
int llms_codec_corrupt_count(const void *workspace, uint32_t *n_corrupt, void *stream);

/* ------------------------------------------------------------------ tolerance score (Eq. 1) */

/* Information density D_i of every chunk (Sec. 3.2 Eq. 1): the attention matrix
 * A = softmax(mask(Q K^T / sqrt(head_dim))) of the last W query positions (row r sits at token
 * position n_tokens - W + r and sees columns 0..that position) is averaged down each column over
 * the rows that see it, then over heads, layers and the chunk's tokens.  W = n_tokens gives the
 * paper's full lower-triangular matrix.  Query head h reads KV head h / (n_q_heads/n_kv_heads).
 *   kv      device fp16 (only K, the s = 0 half, is read)
 *   q_win   device fp16 [n_layers][n_q_heads][W][head_dim], contiguous, 16-byte aligned
 *   scores  device fp32 [floor(n_tokens/chunk_len)]
 *   workspace device, llms_tolerance_workspace_bytes(desc, W) */
int llms_tolerance_workspace_bytes(const llms_kv_desc *desc, int W, uint64_t *nbytes);
int llms_chunk_tolerance(const llms_kv_desc *desc, const void *kv, const void *q_win, int W,
                         float *scores, void *workspace, uint64_t workspace_bytes, void *stream);
/* The same reduction from attention probabilities that inference already produced:
 *   probs   device fp32 [n_layers][n_q_heads][W][n_tokens]; entries above the causal boundary
 *           (col > n_tokens - W + r) are ignored. */
int llms_chunk_tolerance_from_probs(const llms_kv_desc *desc, const float *probs, int W,
                                    float *scores, void *workspace, uint64_t workspace_bytes, void *stream);

/* ------------------------------------------------------------------ policy (host only) */

/* Eq. 2: rank chunks by density and map rank to a bit-width.  order_out (may be NULL) receives
 * chunk indices, densest first, ties to the lower index.  With frac = {f8, f4, f2} (sum 1):
 * the first n8 = floor(f8*n + 1/2) chunks of that order keep 8 bits, up to
 * floor((f8+f4)*n + 1/2) get 4, the rest 2 - low density means high tolerance means fewer bits. */
int llms_assign_bits(const float *scores, int n, const float frac[3], uint8_t *bits_out, uint32_t *order_out);

/* Eq. 2 for another level set (Sec. 3.2: the method is not tied to 8/4/2 - atop a 4-bit cache it offers 2 and
 * 1 bit).  levels = {top, middle, low} bit-widths from {8, 4, 2, 1}, strictly decreasing; frac = the shares
 * of chunks per level, in that order; everything else as llms_assign_bits, which is this call with
 * levels {8, 4, 2}; llms_optimize_thresholds_levels finds the shares for such a set. */
int llms_assign_levels(const float *scores, int n, const float frac[3], const uint8_t levels[3],
                       uint8_t *bits_out, uint32_t *order_out);

/* Eq. 3: the shares of chunks per level that maximise the context's information under a global average
 * ratio, for the levels {8/8, 4/8, 2/8} (Sec. 3.2: one free variable is left).  A chunk at level w keeps
 * weight ratio_w of its density (the printed weight 1/ratio_w would reward compressing the densest chunks most and
 * is read as a misprint).
 * ratio_global in [0.25, 1] is relative to 8 bits: f8 + f4/2 + f2/4 = ratio_global, hence
 * f2 = 2*f8 + 2 - 4*ratio_global.  Every count n8 of 8-bit chunks is tried on the density-ordered list
 * (n2 = floor(2*n8 + (2 - 4*ratio_global)*n + 1/2), n4 the rest); the best wins, the smaller n8 on a tie.
 * frac_out = {n8, n4, n2} / n, ready for llms_assign_bits.  scores: host, n > 0 values. */
int llms_optimize_thresholds(const float *scores, int n, float ratio_global, float frac_out[3]);

/* Eq. 3 for any level set {top, middle, low} (strictly decreasing bit-widths from {8, 4, 2, 1}).  With
 * r1 = middle/top and r2 = low/top, ratio_global in [r2, 1] is relative to the top level:
 * f_top + r1*f_mid + r2*f_low = ratio_global, hence f_low = ((1 - r1)*f_top + r1 - ratio_global) / (r1 - r2);
 * n_low = floor(that * n + 1/2) for every count n_top, weights 1, r1, r2, the best wins, the smaller n_top on a
 * tie.  LLMS_ERR_INVALID_ARG when no count triple meets the ratio (possible for a handful of chunks only).
 * llms_optimize_thresholds is this call with levels {8, 4, 2}. */
int llms_optimize_thresholds_levels(const float *scores, int n, float ratio_global, const uint8_t levels[3],
                                    float frac_out[3]);

/* Sec. 3.4 (ii): eviction order over the rows that are resident and not locked - the 8-bit
 * sub-queue first, then 4, then 2 ("heavy chunks first"), least recently used first inside a
 * sub-queue, ties by (ctx_id, chunk_id).  order_out (n entries) receives row indices; the return
 * value is their count, or a negative status. */
int llms_lctru_order(const llms_chunk_state *table, int n, uint32_t *order_out);

/* ------------------------------------------------------------------ a whole context in one call */

/* The compression half of swapping a context out (Sec. 3.2, "Compressing chunks": density of every
 * chunk, its rank, its level, then quantization) as one call: llms_chunk_tolerance on K and the query
 * window, llms_assign_levels on the scores, then llms_compress_chunks over all chunks in index order
 * (chunk_ids 0 .. n-1).  Results are those of the three calls made one after the other.
 *   scores_dev   device fp32 [n_chunks];  scores_host  host fp32 [n_chunks]
 *   bits_out     host, n_chunks bytes: the level each chunk got
 *   after_scores optional cudaEvent_t, recorded on `stream` behind the score kernels and whatever
 *                brings scores, levels and meta to the host
 *   everything else as in the three calls.
 * Stream-ordered form: when scores_host, bits_out and meta all lie in page-locked memory (and the
 * context has at most 4096 chunks), a kernel ranks the chunks, assigns the levels and lays the
 * encoder's chunk table down on the device, and stores scores, levels and meta (sizes, offsets)
 * into the three host arrays itself: the call returns without synchronising, and the three arrays
 * are valid once after_scores has completed (meta[].checksum once the whole call has).  A call that
 * needs meta on the host - llms_decompress_chunks, llms_swap_out - waits for that event first
 * (llms_wait), while the encoder is still running.
 * Otherwise the ranking is a host step: the call synchronises `stream` once, when the scores have
 * reached the host, and the arrays are filled when it returns (checksums as in llms_compress_chunks).
 * All arguments, the room in out_buf included (the number of chunks per level follows from frac and
 * n_chunks alone), are checked before the first launch. */
int llms_compress_context(const llms_kv_desc *desc, const void *kv, const void *q_win, int W,
                          const float frac[3], const uint8_t levels[3],
                          float *scores_dev, float *scores_host, uint8_t *bits_out,
                          void *out_buf, uint64_t out_bytes, llms_chunk_meta *meta,
                          void *tolerance_workspace, uint64_t tolerance_workspace_bytes,
                          void *codec_workspace, uint64_t codec_workspace_bytes,
                          void *after_scores, void *stream);

/* ------------------------------------------------------------------ swap copies */

/* Copy n records between a device swap buffer and a pinned host arena on `side_stream`
 * (Sec. 3.1 Reclaim / Load, with pinned host memory in the place of the paper's disk; Sec. 4:
 * an I/O thread of its own).  Record i sits at meta[i].offset in the device buffer and at
 * host_offsets[i] in the arena (host_offsets == NULL: the same offsets).  Runs of records
 * adjacent on both sides travel as one copy.  If `after` (a cudaEvent_t) is not NULL the side
 * stream first waits for it - record it on the stream that produced (swap-out) or last used
 * (swap-in) the device buffer.  If `done` is not NULL it is recorded on the side stream after
 * the last copy.  dev_bytes and host_bytes are the sizes of the device buffer and of the arena: a
 * record that ends beyond either is refused with LLMS_ERR_BUF_TOO_SMALL before any copy is queued. */
int llms_swap_out(const void *dev_buf, uint64_t dev_bytes, const llms_chunk_meta *meta, int n, void *pinned_dst,
                  uint64_t host_bytes, const uint64_t *host_offsets, void *side_stream, void *after, void *done);
int llms_swap_in(const void *pinned_src, uint64_t host_bytes, const uint64_t *host_offsets, const llms_chunk_meta *meta,
                 int n, void *dev_buf, uint64_t dev_bytes, void *side_stream, void *after, void *done);
/* Poll a cudaEvent_t until it has completed or timeout_ms has passed (LLMS_ERR_TIMEOUT). */
int llms_wait(void *event, uint32_t timeout_ms);

/* ------------------------------------------------------------------ checked build */

/* Not a step of the method (the paper has no counterpart).  The library can be built a second time with a bounds check
 * in front of every access the group-wise codec kernels make to the KV tensor and the swap buffer (a file of its
 * own, for tests; see the package's build module).  In that build this call waits for the device and reports how many
 * accesses fell outside the two buffers of their call since the library was loaded (they were skipped) and the address
 * of the first one; in the ordinary build it sets *compiled_in = 0 and the other two to 0.  The checked build keeps
 * one pair of ranges per device: its codec calls must not overlap on different streams.  All three pointers are host
 * pointers and must not be NULL (LLMS_ERR_INVALID_ARG). */
int llms_debug_bounds(uint32_t *compiled_in, uint32_t *violations, uint64_t *first_address);

/* ------------------------------------------------------------------ measurement aid */

/* Not a step of the method (the paper has no counterpart): a plain streaming kernel with the codec kernels' access
 * shape - every load or store instruction of a warp covers 1 KiB of consecutive bytes in 256-bit accesses - that reads
 * read_kib KiB from src and writes write_kib KiB to dst per warp iteration, `iters` iterations in all.  Timing it
 * tells what the memory system gives a stream of that read:write mix, the yardstick for the encoder (about 4:1) and
 * the decoder (about 1:4).  Mixes: (4,0) read only, (0,4) write only, (4,1), (1,4), (2,2); others return
 * LLMS_ERR_UNSUPPORTED.  src and dst are device pointers, 32-byte aligned, of at least iters*read_kib KiB and
 * iters*write_kib KiB (LLMS_ERR_BUF_TOO_SMALL otherwise, before any launch); dst is overwritten with arbitrary bytes. */
int llms_stream_probe(const void *src, uint64_t src_bytes, void *dst, uint64_t dst_bytes, uint64_t iters,
                      int read_kib, int write_kib, void *stream);

/* The same stream with a chosen work split (no counterpart in the paper either): 0 = a warp per iteration, CTAs handed
 * out in address order as earlier ones leave (what llms_stream_probe runs, the fastest plain stream found); 1 = two
 * resident CTAs per SM, warp w takes iterations w, w + W, ... (the split the codec kernels had at first); 2 = two
 * resident CTAs per SM whose warps draw batches of two iterations from 16 counters (the codec kernels' split now; the
 * counters live in the library, so calls with split 2 on one device must not overlap).  Other values:
 * LLMS_ERR_INVALID_ARG.  Arguments and errors otherwise as llms_stream_probe. */
int llms_stream_probe_split(const void *src, uint64_t src_bytes, void *dst, uint64_t dst_bytes, uint64_t iters,
                            int read_kib, int write_kib, int split, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* LLMS_H */
