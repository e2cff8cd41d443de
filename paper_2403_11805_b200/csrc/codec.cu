// Chunk codec kernels for sm_100a: group quantize + bit-pack (swap-out) and unpack + dequantize (swap-in).
//
// Work item = one slab (chunk_len*head_dim contiguous fp16 of one chunk, layer, K/V, head).  One warp
// takes a slab at a time from a persistent grid.  A lane owns 16 consecutive elements (32 bytes of
// fp16), so a group of G channels is G/16 neighbouring lanes: min/max take log2(G/16) xor-shuffles,
// a lane's packed codes are 4/8/16 contiguous bytes at 2/4/8 bits, and the warp's stores are contiguous.
// The bit-width is uniform per chunk, hence per warp.
//
// The arithmetic is fixed by the record format (see llms.h): every binary32 operation is written with a
// round-to-nearest intrinsic so that nothing is contracted into an FMA or replaced by an approximation.
#include <vector>

#include "llms_internal.cuh"

namespace llms {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kElemsPerLane = 16;
constexpr int kElemsPerWarpIter = 32 * kElemsPerLane;  // 512 elements = 1 KiB of fp16

struct CodecArgs {
    const __half *kv_in;   // compress: source
    __half *kv_out;        // decompress: destination
    uint8_t *buf;          // swap buffer (written by compress, read by decompress)
    ChunkEntry *entries;   // n entries in the workspace
    uint32_t *sums;        // decompress: recomputed checksums
    int n;
    int n_slabs;           // slabs per chunk
    int slab_elems;        // chunk_len * head_dim
    int groups_per_slab;
    int n_kv_heads;
    uint32_t codes_off;    // byte offset of the code stream in a record
    uint32_t params_bytes; // 4 * n_groups
    int64_t stride_l, stride_s, stride_h, chunk_stride;
};

__device__ __forceinline__ int64_t slab_offset(const CodecArgs &a, int s_idx, uint32_t chunk)
{
    const int h = s_idx % a.n_kv_heads;
    const int ls = s_idx / a.n_kv_heads;
    return (int64_t)(ls >> 1) * a.stride_l + (int64_t)(ls & 1) * a.stride_s + (int64_t)h * a.stride_h +
           (int64_t)chunk * a.chunk_stride;
}

__device__ __forceinline__ __half2 as_h2(uint32_t u) { return *reinterpret_cast<__half2 *>(&u); }
__device__ __forceinline__ uint32_t as_u32(__half2 h) { return *reinterpret_cast<uint32_t *>(&h); }

// ---------------------------------------------------------------------------------------------- quantize

// Quantize the lane's 16 values and pack them: BITS/2 words.
template <int BITS>
__device__ __forceinline__ void quantize_pack16(const uint32_t (&w)[8], float zero, float inv, uint32_t (&out)[BITS / 2])
{
    constexpr float kQmax = (float)((1 << BITS) - 1);
    uint32_t q[16];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const float2 f = __half22float2(as_h2(w[k]));
        const float v0 = fminf(__fmul_rn(__fsub_rn(f.x, zero), inv), kQmax);
        const float v1 = fminf(__fmul_rn(__fsub_rn(f.y, zero), inv), kQmax);
        q[2 * k] = (uint32_t)__float2int_rn(v0);  // round half to even; v >= 0 always because zero is the minimum
        q[2 * k + 1] = (uint32_t)__float2int_rn(v1);
    }
    constexpr int kPerWord = 32 / BITS;
#pragma unroll
    for (int j = 0; j < BITS / 2; ++j) {
        uint32_t word = 0;
#pragma unroll
        for (int k = 0; k < kPerWord; ++k) word |= q[j * kPerWord + k] << (k * BITS);
        out[j] = word;
    }
}

template <int BITS>
__device__ __forceinline__ void store_codes(uint8_t *p, const uint32_t (&c)[BITS / 2])
{
    if constexpr (BITS == 8) *reinterpret_cast<uint4 *>(p) = make_uint4(c[0], c[1], c[2], c[3]);
    else if constexpr (BITS == 4) *reinterpret_cast<uint2 *>(p) = make_uint2(c[0], c[1]);
    else *reinterpret_cast<uint32_t *>(p) = c[0];
}

// One slab by one warp.  Returns this lane's share of the checksum.
template <int BITS, int LPG>
__device__ __forceinline__ uint32_t compress_slab(const CodecArgs &a, const __half *__restrict__ src, uint8_t *__restrict__ rec,
                                                  int s_idx, int lane)
{
    constexpr float kQmax = (float)((1 << BITS) - 1);
    constexpr int kLaneBytes = kElemsPerLane * BITS / 8;
    uint32_t *params = reinterpret_cast<uint32_t *>(rec) + (int64_t)s_idx * a.groups_per_slab;
    uint8_t *codes = rec + a.codes_off + (int64_t)s_idx * a.slab_elems * BITS / 8;
    uint32_t sum = 0;
    for (int e0 = lane * kElemsPerLane; e0 - lane * kElemsPerLane < a.slab_elems; e0 += kElemsPerWarpIter) {
        const bool active = e0 < a.slab_elems;  // inactive lanes form whole inactive groups
        uint32_t w[8];
        if (active) {
            const uint4 lo = __ldg(reinterpret_cast<const uint4 *>(src + e0));
            const uint4 hi = __ldg(reinterpret_cast<const uint4 *>(src + e0) + 1);
            w[0] = lo.x; w[1] = lo.y; w[2] = lo.z; w[3] = lo.w;
            w[4] = hi.x; w[5] = hi.y; w[6] = hi.z; w[7] = hi.w;
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) w[k] = 0;
        }
        // min and max of the lane's 16 values, two at a time
        __half2 mn2 = as_h2(w[0]), mx2 = as_h2(w[0]);
#pragma unroll
        for (int k = 1; k < 8; ++k) {
            mn2 = __hmin2(mn2, as_h2(w[k]));
            mx2 = __hmax2(mx2, as_h2(w[k]));
        }
        // (min, -max) in one register: a single min per shuffle step reduces both
        __half2 mm = __halves2half2(__hmin(__low2half(mn2), __high2half(mn2)),
                                    __hneg(__hmax(__low2half(mx2), __high2half(mx2))));
#pragma unroll
        for (int m = LPG / 2; m > 0; m >>= 1) mm = __hmin2(mm, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mm), m)));
        // adding +0 turns a -0 minimum or maximum into +0 and changes nothing else
        const float zero = __fadd_rn(__low2float(mm), 0.0f);
        const float top = __fadd_rn(-__high2float(mm), 0.0f);
        const __half scale_h = __float2half_rn(__fdiv_rn(__fsub_rn(top, zero), kQmax));
        const float scale = __half2float(scale_h);
        const float inv = scale == 0.0f ? 0.0f : __frcp_rn(scale);  // inv = 0 makes every code 0
        uint32_t c[BITS / 2];
        quantize_pack16<BITS>(w, zero, inv, c);
        if (active) {
            store_codes<BITS>(codes + (int64_t)(e0 / kElemsPerLane) * kLaneBytes, c);
#pragma unroll
            for (int j = 0; j < BITS / 2; ++j) sum += c[j];
            if ((lane & (LPG - 1)) == 0) {
                const uint32_t p = (uint32_t)__half_as_ushort(scale_h) | ((uint32_t)__half_as_ushort(__float2half_rn(zero)) << 16);
                params[e0 / (kElemsPerLane * LPG)] = p;
                sum += p;
            }
        }
    }
    return sum;
}

// Zero the two padding runs of a record (after the parameter block, after the code stream).
__device__ __forceinline__ void zero_padding(const CodecArgs &a, uint8_t *rec, const ChunkEntry &e, int lane)
{
    for (uint32_t i = a.params_bytes + lane; i < a.codes_off; i += 32) rec[i] = 0;
    const uint64_t codes_end = a.codes_off + (uint64_t)a.n_slabs * a.slab_elems * e.bits / 8;
    for (uint64_t i = codes_end + lane; i < e.nbytes; i += 32) rec[i] = 0;
}

template <int LPG>
__global__ void __launch_bounds__(kThreads) compress_kernel(const CodecArgs a)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kWarpsPerBlock;
    const int64_t total = (int64_t)a.n * a.n_slabs;
    for (int64_t item = warp; item < total; item += n_warps) {
        const int i = (int)(item / a.n_slabs);
        const int s_idx = (int)(item - (int64_t)i * a.n_slabs);
        const ChunkEntry e = a.entries[i];
        const __half *src = a.kv_in + slab_offset(a, s_idx, e.chunk_id);
        uint8_t *rec = a.buf + e.offset;
        uint32_t sum;
        if (e.bits == 8) sum = compress_slab<8, LPG>(a, src, rec, s_idx, lane);
        else if (e.bits == 4) sum = compress_slab<4, LPG>(a, src, rec, s_idx, lane);
        else sum = compress_slab<2, LPG>(a, src, rec, s_idx, lane);
        if (s_idx == 0) zero_padding(a, rec, e, lane);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.entries[i].checksum, sum);
    }
}

// ---------------------------------------------------------------------------------------------- dequantize

template <int BITS>
__device__ __forceinline__ void load_codes(const uint8_t *p, uint32_t (&c)[BITS / 2])
{
    if constexpr (BITS == 8) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(p));
        c[0] = v.x; c[1] = v.y; c[2] = v.z; c[3] = v.w;
    } else if constexpr (BITS == 4) {
        const uint2 v = __ldg(reinterpret_cast<const uint2 *>(p));
        c[0] = v.x; c[1] = v.y;
    } else {
        c[0] = __ldg(reinterpret_cast<const uint32_t *>(p));
    }
}

__device__ __forceinline__ float decode(uint32_t q, float scale, float zero)
{
    // q*scale is exact in binary32, so the fused form rounds once, like multiply-then-add would
    const float v = __fmaf_rn((float)q, scale, zero);
    return fminf(fmaxf(v, -65504.0f), 65504.0f);
}

template <int BITS, int LPG>
__device__ __forceinline__ uint32_t decompress_slab(const CodecArgs &a, const uint8_t *__restrict__ rec, __half *__restrict__ dst,
                                                    int s_idx, int lane)
{
    constexpr int kLaneBytes = kElemsPerLane * BITS / 8;
    constexpr int kPerWord = 32 / BITS;
    constexpr uint32_t kMask = (1u << BITS) - 1u;
    const uint32_t *params = reinterpret_cast<const uint32_t *>(rec) + (int64_t)s_idx * a.groups_per_slab;
    const uint8_t *codes = rec + a.codes_off + (int64_t)s_idx * a.slab_elems * BITS / 8;
    uint32_t sum = 0;
    for (int e0 = lane * kElemsPerLane; e0 < a.slab_elems; e0 += kElemsPerWarpIter) {
        uint32_t c[BITS / 2];
        load_codes<BITS>(codes + (int64_t)(e0 / kElemsPerLane) * kLaneBytes, c);
        const uint32_t p = __ldg(params + e0 / (kElemsPerLane * LPG));
        const float scale = __half2float(__ushort_as_half((unsigned short)(p & 0xffffu)));
        const float zero = __half2float(__ushort_as_half((unsigned short)(p >> 16)));
        uint32_t w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int e = 2 * k;
            const uint32_t q0 = (c[e / kPerWord] >> ((e % kPerWord) * BITS)) & kMask;
            const uint32_t q1 = (c[(e + 1) / kPerWord] >> (((e + 1) % kPerWord) * BITS)) & kMask;
            w[k] = as_u32(__floats2half2_rn(decode(q0, scale, zero), decode(q1, scale, zero)));
        }
        uint4 *out = reinterpret_cast<uint4 *>(dst + e0);
        out[0] = make_uint4(w[0], w[1], w[2], w[3]);
        out[1] = make_uint4(w[4], w[5], w[6], w[7]);
#pragma unroll
        for (int j = 0; j < BITS / 2; ++j) sum += c[j];
        if ((lane & (LPG - 1)) == 0) sum += p;
    }
    return sum;
}

template <int LPG>
__global__ void __launch_bounds__(kThreads) decompress_kernel(const CodecArgs a)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = (int64_t)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const int64_t n_warps = (int64_t)gridDim.x * kWarpsPerBlock;
    const int64_t total = (int64_t)a.n * a.n_slabs;
    for (int64_t item = warp; item < total; item += n_warps) {
        const int i = (int)(item / a.n_slabs);
        const int s_idx = (int)(item - (int64_t)i * a.n_slabs);
        const ChunkEntry e = a.entries[i];
        const uint8_t *rec = a.buf + e.offset;
        __half *dst = a.kv_out + slab_offset(a, s_idx, e.chunk_id);
        uint32_t sum;
        if (e.bits == 8) sum = decompress_slab<8, LPG>(a, rec, dst, s_idx, lane);
        else if (e.bits == 4) sum = decompress_slab<4, LPG>(a, rec, dst, s_idx, lane);
        else sum = decompress_slab<2, LPG>(a, rec, dst, s_idx, lane);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.sums[i], sum);
    }
}

// status word = number of records whose recomputed sum differs from the expected one
__global__ void verify_kernel(const ChunkEntry *entries, const uint32_t *sums, int n, uint32_t *status)
{
    uint32_t bad = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x) bad += (sums[i] != entries[i].checksum);
    bad = __reduce_add_sync(0xffffffffu, bad);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(status, bad);
}

// ---------------------------------------------------------------------------------------------- host side

static int fill_args(const llms_kv_desc &d, CodecArgs &a, int n, void *workspace)
{
    a.n = n;
    a.n_slabs = (int)slabs_per_chunk(d);
    a.slab_elems = (int)slab_elems(d);
    a.groups_per_slab = (int)groups_per_slab(d);
    a.n_kv_heads = d.n_kv_heads;
    a.params_bytes = (uint32_t)(groups_per_chunk(d) * 4);
    a.codes_off = (uint32_t)round_up(a.params_bytes, 16);
    a.stride_l = d.stride_l;
    a.stride_s = d.stride_s;
    a.stride_h = d.stride_h;
    a.chunk_stride = (int64_t)d.chunk_len * d.head_dim;
    a.entries = reinterpret_cast<ChunkEntry *>(static_cast<uint8_t *>(workspace) + kWsEntriesOffset);
    a.sums = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + ws_sums_offset(n));
    return LLMS_OK;
}

static int grid_for(int64_t items)
{
    const int64_t want = (items + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int64_t cap = (int64_t)sm_count() * 8;  // 8 CTAs of 256 threads fill an SM
    return (int)(want < cap ? want : cap);
}

template <typename F>
static int dispatch_lpg(int group_size, F &&f)
{
    switch (group_size / kElemsPerLane) {
    case 1: f(std::integral_constant<int, 1>()); break;
    case 2: f(std::integral_constant<int, 2>()); break;
    case 4: f(std::integral_constant<int, 4>()); break;
    case 8: f(std::integral_constant<int, 8>()); break;
    case 16: f(std::integral_constant<int, 16>()); break;
    case 32: f(std::integral_constant<int, 32>()); break;
    default: return LLMS_ERR_UNSUPPORTED;
    }
    return LLMS_OK;
}

static int check_common(const llms_kv_desc *desc, int n, const void *workspace, uint64_t workspace_bytes)
{
    int rc = check_desc_codec(desc);
    if (rc) return rc;
    if (desc->quant_mode != 0) return LLMS_ERR_UNSUPPORTED;
    if (n < 0) return LLMS_ERR_INVALID_ARG;
    if (n == 0) return LLMS_OK;
    if (!workspace) return LLMS_ERR_INVALID_ARG;
    if (!aligned(workspace, 16)) return LLMS_ERR_MISALIGNED;
    if (workspace_bytes < ws_total(n)) return LLMS_ERR_BUF_TOO_SMALL;
    if (groups_per_chunk(*desc) * 4 > 0xffffffffull) return LLMS_ERR_UNSUPPORTED;
    if (slab_elems(*desc) > 0x7fffffff / 8) return LLMS_ERR_UNSUPPORTED;
    return LLMS_OK;
}

}  // namespace llms

using namespace llms;

extern "C" int llms_compress_chunks(const llms_kv_desc *desc, const void *kv, const uint32_t *chunk_ids,
                                    const uint8_t *bits, int n, void *out_buf, uint64_t out_bytes,
                                    llms_chunk_meta *meta, void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_common(desc, n, workspace, workspace_bytes);
    if (rc) return rc;
    if (n == 0) return LLMS_OK;
    if (!kv || !chunk_ids || !bits || !out_buf || !meta) return LLMS_ERR_INVALID_ARG;
    if (!aligned(kv, 16) || !aligned(out_buf, 256)) return LLMS_ERR_MISALIGNED;
    const uint32_t nc = (uint32_t)n_chunks(*desc);
    std::vector<uint8_t> seen(nc, 0);
    uint64_t off = 0;
    for (int i = 0; i < n; ++i) {
        uint64_t nb;
        rc = llms_record_bytes(desc, bits[i], &nb);
        if (rc) return rc;
        if (chunk_ids[i] >= nc || seen[chunk_ids[i]]) return LLMS_ERR_INVALID_ARG;
        seen[chunk_ids[i]] = 1;
        off += nb;
    }
    if (off > out_bytes) return LLMS_ERR_BUF_TOO_SMALL;
    off = 0;
    for (int i = 0; i < n; ++i) {
        uint64_t nb;
        llms_record_bytes(desc, bits[i], &nb);
        meta[i].chunk_id = chunk_ids[i];
        meta[i].bits = bits[i];
        meta[i].offset = off;
        meta[i].nbytes = nb;
        meta[i].n_groups = (uint32_t)groups_per_chunk(*desc);
        meta[i].checksum = 0;  // the kernel accumulates into the device copy
        off += nb;
    }
    CodecArgs a{};
    fill_args(*desc, a, n, workspace);
    a.kv_in = static_cast<const __half *>(kv);
    a.buf = static_cast<uint8_t *>(out_buf);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    LLMS_CUDA_TRY(cudaMemcpyAsync(a.entries, meta, (size_t)n * sizeof(ChunkEntry), cudaMemcpyHostToDevice, st));
    const int grid = grid_for((int64_t)n * a.n_slabs);
    rc = dispatch_lpg(desc->group_size, [&](auto lpg) {
        compress_kernel<decltype(lpg)::value><<<grid, kThreads, 0, st>>>(a);
    });
    if (rc) return rc;
    LLMS_CUDA_TRY(cudaGetLastError());
    LLMS_CUDA_TRY(cudaMemcpyAsync(meta, a.entries, (size_t)n * sizeof(ChunkEntry), cudaMemcpyDeviceToHost, st));
    return LLMS_OK;
}

extern "C" int llms_decompress_chunks(const llms_kv_desc *desc, const void *buf, const llms_chunk_meta *meta,
                                      const uint32_t *dst_chunk_ids, int n, void *kv_out,
                                      void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_common(desc, n, workspace, workspace_bytes);
    if (rc) return rc;
    if (n == 0) return LLMS_OK;
    if (!buf || !meta || !kv_out) return LLMS_ERR_INVALID_ARG;
    if (!aligned(kv_out, 16) || !aligned(buf, 256)) return LLMS_ERR_MISALIGNED;
    const uint32_t nc = (uint32_t)n_chunks(*desc);
    std::vector<uint8_t> seen(nc, 0);
    std::vector<llms_chunk_meta> staged(meta, meta + n);
    for (int i = 0; i < n; ++i) {
        uint64_t nb;
        rc = llms_record_bytes(desc, (int)meta[i].bits, &nb);
        if (rc) return rc;
        if (meta[i].nbytes != nb || meta[i].n_groups != (uint32_t)groups_per_chunk(*desc)) return LLMS_ERR_INVALID_ARG;
        if (meta[i].offset % 256) return LLMS_ERR_MISALIGNED;
        const uint32_t dst = dst_chunk_ids ? dst_chunk_ids[i] : meta[i].chunk_id;
        if (dst >= nc || seen[dst]) return LLMS_ERR_INVALID_ARG;
        seen[dst] = 1;
        staged[i].chunk_id = dst;
    }
    CodecArgs a{};
    fill_args(*desc, a, n, workspace);
    a.kv_out = static_cast<__half *>(kv_out);
    a.buf = const_cast<uint8_t *>(static_cast<const uint8_t *>(buf));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t *status = static_cast<uint32_t *>(workspace);
    // `staged` is pageable: the copy has left it by the time cudaMemcpyAsync returns
    LLMS_CUDA_TRY(cudaMemcpyAsync(a.entries, staged.data(), (size_t)n * sizeof(ChunkEntry), cudaMemcpyHostToDevice, st));
    LLMS_CUDA_TRY(cudaMemsetAsync(a.sums, 0, (size_t)n * 4, st));
    LLMS_CUDA_TRY(cudaMemsetAsync(status, 0, 4, st));
    const int grid = grid_for((int64_t)n * a.n_slabs);
    rc = dispatch_lpg(desc->group_size, [&](auto lpg) {
        decompress_kernel<decltype(lpg)::value><<<grid, kThreads, 0, st>>>(a);
    });
    if (rc) return rc;
    LLMS_CUDA_TRY(cudaGetLastError());
    verify_kernel<<<1, 256, 0, st>>>(a.entries, a.sums, n, status);
    LLMS_CUDA_TRY(cudaGetLastError());
    return LLMS_OK;
}

extern "C" int llms_codec_corrupt_count(const void *workspace, uint32_t *n_corrupt, void *stream)
{
    if (!workspace) return LLMS_ERR_INVALID_ARG;
    uint32_t bad = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    LLMS_CUDA_TRY(cudaMemcpyAsync(&bad, workspace, 4, cudaMemcpyDeviceToHost, st));
    LLMS_CUDA_TRY(cudaStreamSynchronize(st));
    if (n_corrupt) *n_corrupt = bad;
    return bad ? LLMS_ERR_CORRUPT : LLMS_OK;
}

// ---------------------------------------------------------------------------------------------- no-allocation variant

namespace llms {

constexpr uint64_t kStaticWorkspaceBytes =
    (kWsEntriesOffset + (uint64_t)LLMS_STATIC_MAX_CHUNKS * (sizeof(ChunkEntry) + 4) + 255) / 256 * 256;

// Scratch of llms_compress_chunks_static: lives in the library image, one copy on every GPU that loads it.
static __device__ __align__(256) unsigned char g_static_workspace[kStaticWorkspaceBytes];

// Device address of the array above, looked up once per device.  (In host code the array's name is only a handle
// for the runtime; the address a kernel can use has to be asked for.)
static int static_workspace_address(void **out)
{
    static void *cached[64] = {nullptr};
    int dev = -1;
    LLMS_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return LLMS_ERR_UNSUPPORTED;
    if (cached[dev] == nullptr) {
        void *p = nullptr;
        LLMS_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_workspace));
        if (p == nullptr) return LLMS_ERR_CUDA;
        cached[dev] = p;  // two threads racing here store the same value
    }
    *out = cached[dev];
    return LLMS_OK;
}

}  // namespace llms

extern "C" int llms_compress_chunks_static(const llms_kv_desc *desc, const void *kv, const uint32_t *chunk_ids,
                                           const uint8_t *bits, int n, void *out_buf, uint64_t out_bytes,
                                           llms_chunk_meta *meta, void *stream)
{
    if (n > LLMS_STATIC_MAX_CHUNKS) return LLMS_ERR_BUF_TOO_SMALL;  // the built-in scratch holds no more entries
    void *ws = nullptr;
    const int rc = static_workspace_address(&ws);
    if (rc) return rc;
    // The chunk table copied in by the call below carries zeroed checksum fields, which is all of the
    // scratch that has to start from zero; whatever the previous call left behind is overwritten.
    return llms_compress_chunks(desc, kv, chunk_ids, bits, n, out_buf, out_bytes, meta, ws, kStaticWorkspaceBytes, stream);
}
