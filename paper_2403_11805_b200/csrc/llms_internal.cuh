// Shared host-side helpers of the library: argument checks, record layout arithmetic, CUDA error capture.
#pragma once

#include <cuda_runtime.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "llms.h"

namespace llms {

void set_cuda_error(cudaError_t e, const char *where);

#define LLMS_CUDA_TRY(expr)                                   \
    do {                                                      \
        cudaError_t e__ = (expr);                             \
        if (e__ != cudaSuccess) {                             \
            ::llms::set_cuda_error(e__, #expr);               \
            return LLMS_ERR_CUDA;                             \
        }                                                     \
    } while (0)

// Programmatic dependent launch: `kernel` may be set up on the GPU while the kernel before it on the stream is still
// finishing, once all CTAs of that kernel have called grid_launch_dependents() (or left).  The launched kernel must
// call grid_dependency_wait() before it touches anything its predecessor wrote: that returns when the predecessor has
// completed and its writes are visible.  Both calls do nothing in a kernel that was launched the ordinary way.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#ifdef __CUDACC__
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif

inline uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }
inline bool aligned(const void *p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

inline int64_t slabs_per_chunk(const llms_kv_desc &d) { return (int64_t)d.n_layers * 2 * d.n_kv_heads; }
inline int64_t slab_elems(const llms_kv_desc &d) { return (int64_t)d.chunk_len * d.head_dim; }
inline int n_chunks(const llms_kv_desc &d) { return d.n_tokens / d.chunk_len; }
inline uint64_t groups_per_slab(const llms_kv_desc &d)
{
    return d.quant_mode == 0 ? (uint64_t)d.chunk_len * (d.head_dim / d.group_size) : (uint64_t)d.head_dim;
}
inline uint64_t groups_per_chunk(const llms_kv_desc &d) { return (uint64_t)slabs_per_chunk(d) * groups_per_slab(d); }

// Shape checks common to every entry point.
int check_desc(const llms_kv_desc *d);
// Shape + alignment checks for the codec kernels (vector loads need 16-byte aligned slabs).
int check_desc_codec(const llms_kv_desc *d);
inline int check_bits(int b) { return (b == 1 || b == 2 || b == 4 || b == 8) ? LLMS_OK : LLMS_ERR_BAD_BITS; }

// Number of SMs of the current device (cached per device).
int sm_count();

// The device's view of a host pointer if it is page-locked memory the device can access, else NULL.
void *device_view_of_pinned(const void *host_ptr);

// llms_chunk_tolerance with a second destination: scores_live, when not NULL, is a device-visible address (page-locked
// host memory) into which the last kernel also stores the scores, so that no copy has to follow the kernels.
int chunk_tolerance_impl(const llms_kv_desc *desc, const void *kv, const void *q_win, int W, float *scores,
                         float *scores_live, void *workspace, uint64_t workspace_bytes, void *stream);

// The encoder over chunk tables already present in the workspace (see codec.cu), and the argument checks of the
// compress call that do not depend on the chunk list.
int compress_planned(const llms_kv_desc *desc, const void *kv, int n, const int count[4], void *out_buf, uint64_t out_bytes,
                     llms_chunk_meta *meta, void *workspace, void *stream);
int check_compress_args(const llms_kv_desc *desc, int n, const void *kv, const void *out_buf, const void *workspace,
                        uint64_t workspace_bytes);

// Device-side copy of the per-chunk table, kept in the workspace.
struct ChunkEntry {          // same bytes as llms_chunk_meta
    uint32_t chunk_id, bits;
    uint64_t offset, nbytes;
    uint32_t n_groups, checksum;
};
static_assert(sizeof(ChunkEntry) == sizeof(llms_chunk_meta) && sizeof(ChunkEntry) == 32, "meta layout");

// One chunk of a codec launch, in the order the launch walks them (chunks grouped by bit-width).
struct UnitEntry {
    uint32_t chunk_id;  // source / destination chunk (slot) in the KV tensor
    uint32_t entry;     // index into the caller-ordered entry table (checksums)
    uint64_t rec_off;   // byte offset of the record in the swap buffer
};
static_assert(sizeof(UnitEntry) == 16, "table layout");

// Workspace of the codec calls:
// [header][n entries][n 16-byte unit-table rows][n entry indices grouped by bit-width][n recomputed sums].  Header: a
// status word, a spare word and a count of finished CTAs, then, from byte 128 on, the counters from which the codec
// kernels' warps draw their work (four bit-widths x 16 counters, one per 128 bytes).  The header starts every call
// as zeros; everything up to the sums is written by one host-to-device copy per call.
constexpr uint64_t kWsFeedOffset = 128;
constexpr uint64_t kWsFeedBytes = 4 * 16 * 128;
constexpr uint64_t kWsEntriesOffset = kWsFeedOffset + kWsFeedBytes;
constexpr uint64_t kWsBytesPerChunk = sizeof(ChunkEntry) + 16 + 4 + 4;
__host__ __device__ inline uint64_t ws_table_offset(int n) { return kWsEntriesOffset + (uint64_t)n * sizeof(ChunkEntry); }
__host__ __device__ inline uint64_t ws_order_offset(int n) { return ws_table_offset(n) + (uint64_t)n * 16; }
__host__ __device__ inline uint64_t ws_sums_offset(int n) { return ws_order_offset(n) + (uint64_t)n * 4; }
inline uint64_t ws_total(int n) { return round_up(kWsEntriesOffset + (uint64_t)n * kWsBytesPerChunk, 16); }

}  // namespace llms
