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
constexpr int kUnroll = 4;                             // warp passes whose loads are issued together

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
    int slab_major;        // 1: consecutive work items walk the listed chunks of one slab index (linear KV addresses
                           //    when the ids are consecutive); 0: they walk the slabs of one chunk (linear record addresses)
    uint32_t codes_off;    // byte offset of the code stream in a record
    uint32_t params_bytes; // 4 * n_groups
    int64_t stride_l, stride_s, stride_h, chunk_stride;
};

__device__ __forceinline__ int64_t slab_offset(const CodecArgs &a, uint32_t s_idx, uint32_t chunk)
{
    const uint32_t ls = s_idx / (uint32_t)a.n_kv_heads;
    const uint32_t h = s_idx - ls * (uint32_t)a.n_kv_heads;
    return (int64_t)(ls >> 1) * a.stride_l + (int64_t)(ls & 1) * a.stride_s + (int64_t)h * a.stride_h +
           (int64_t)chunk * a.chunk_stride;
}

__device__ __forceinline__ void item_to_chunk_slab(const CodecArgs &a, uint32_t item, uint32_t &i, uint32_t &s_idx)
{
    if (a.slab_major) {
        s_idx = item / (uint32_t)a.n;
        i = item - s_idx * (uint32_t)a.n;
    } else {
        i = item / (uint32_t)a.n_slabs;
        s_idx = item - i * (uint32_t)a.n_slabs;
    }
}

__device__ __forceinline__ __half2 as_h2(uint32_t u) { return *reinterpret_cast<__half2 *>(&u); }
__device__ __forceinline__ uint32_t as_u32(__half2 h) { return *reinterpret_cast<uint32_t *>(&h); }

// 32 bytes per lane.  WIDE: one 256-bit access (needs 32-byte alignment); otherwise two 128-bit accesses.
// Data touched once: no L1 allocation.
template <bool WIDE>
__device__ __forceinline__ void load32(const void *p, uint32_t (&w)[8])
{
    if constexpr (WIDE) {
        asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7])
                     : "l"(p));
    } else {
        asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(p));
        asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "l"(static_cast<const char *>(p) + 16));
    }
}

template <bool WIDE>
__device__ __forceinline__ void store32(void *p, const uint32_t (&w)[8])
{
    if constexpr (WIDE) {
        asm volatile("st.global.L1::no_allocate.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                     :: "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "l"(p)
                     : "memory");
    } else {
        asm volatile("st.global.L1::no_allocate.v4.b32 [%4], {%0,%1,%2,%3};"
                     :: "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "l"(p) : "memory");
        asm volatile("st.global.L1::no_allocate.v4.b32 [%4], {%0,%1,%2,%3};"
                     :: "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "l"(static_cast<char *>(p) + 16) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------- quantize

// Adding 1.5 * 2^23 rounds a value in [0, 2^22) to an integer, ties to even, and leaves that integer in the
// low mantissa bits: bits = 0x4B400000 + q.
constexpr float kRoundMagic = 12582912.0f;
constexpr uint32_t kRoundMagicBits = 0x4B400000u;

// Quantize the lane's 16 values and pack them into BITS/2 words.  CLAMP is only needed when the scale is a
// subnormal fp16 number: otherwise (x - zero) / scale cannot reach 2^BITS - 1/2.
template <int BITS, bool CLAMP>
__device__ __forceinline__ void quantize_pack16(const uint32_t (&w)[8], float zero, float inv, uint32_t (&out)[BITS / 2])
{
    constexpr float kQmax = (float)((1 << BITS) - 1);
    uint32_t t[16];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const float2 f = __half22float2(as_h2(w[k]));
        float v0 = __fmul_rn(__fsub_rn(f.x, zero), inv);  // >= 0: zero is the minimum
        float v1 = __fmul_rn(__fsub_rn(f.y, zero), inv);
        if constexpr (CLAMP) {
            v0 = fminf(v0, kQmax);
            v1 = fminf(v1, kQmax);
        }
        t[2 * k] = __float_as_uint(__fadd_rn(v0, kRoundMagic));
        t[2 * k + 1] = __float_as_uint(__fadd_rn(v1, kRoundMagic));
    }
    if constexpr (BITS == 8) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t lo = __byte_perm(t[4 * j], t[4 * j + 1], 0x0040);      // bytes: q0 q1 . .
            const uint32_t hi = __byte_perm(t[4 * j + 2], t[4 * j + 3], 0x0040);  // bytes: q2 q3 . .
            out[j] = __byte_perm(lo, hi, 0x5410);
        }
    } else {
        // sum of (magic + q_k) << (k*BITS), minus the magic's share: arithmetic mod 2^32, one shift-add per code
        constexpr int kPerWord = 32 / BITS;
        uint32_t ones = 0;
#pragma unroll
        for (int k = 0; k < kPerWord; ++k) ones += 1u << (k * BITS);
        const uint32_t bias = kRoundMagicBits * ones;
#pragma unroll
        for (int j = 0; j < BITS / 2; ++j) {
            uint32_t acc = 0u - bias;
#pragma unroll
            for (int k = 0; k < kPerWord; ++k) acc += t[j * kPerWord + k] << (k * BITS);
            out[j] = acc;
        }
    }
}

template <int BITS>
__device__ __forceinline__ void store_codes(uint8_t *p, const uint32_t (&c)[BITS / 2])
{
    if constexpr (BITS == 8)
        asm volatile("st.global.L1::no_allocate.v4.b32 [%4], {%0,%1,%2,%3};" :: "r"(c[0]), "r"(c[1]), "r"(c[2]), "r"(c[3]), "l"(p) : "memory");
    else if constexpr (BITS == 4)
        asm volatile("st.global.L1::no_allocate.v2.b32 [%2], {%0,%1};" :: "r"(c[0]), "r"(c[1]), "l"(p) : "memory");
    else
        asm volatile("st.global.L1::no_allocate.b32 [%1], %0;" :: "r"(c[0]), "l"(p) : "memory");
}

// One slab by one warp.  Returns this lane's share of the checksum.
template <int BITS, int LPG, bool WIDE>
__device__ __forceinline__ uint32_t compress_slab(const CodecArgs &a, const __half *__restrict__ src, uint8_t *__restrict__ rec,
                                                  uint32_t s_idx, int lane)
{
    constexpr float kQmax = (float)((1 << BITS) - 1);
    constexpr int kLaneBytes = kElemsPerLane * BITS / 8;
    uint32_t *params = reinterpret_cast<uint32_t *>(rec) + (uint64_t)s_idx * a.groups_per_slab;
    uint8_t *codes = rec + a.codes_off + (uint64_t)s_idx * a.slab_elems * BITS / 8;
    uint32_t sum = 0;
    for (int base = 0; base < a.slab_elems; base += kUnroll * kElemsPerWarpIter) {
        uint32_t w[kUnroll][8];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {  // all loads of the block first: 128 bytes in flight per lane
            const int e0 = base + u * kElemsPerWarpIter + lane * kElemsPerLane;
            if (e0 < a.slab_elems) {
                load32<WIDE>(src + e0, w[u]);
            } else {
#pragma unroll
                for (int k = 0; k < 8; ++k) w[u][k] = 0;  // inactive lanes form whole inactive groups
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int e0 = base + u * kElemsPerWarpIter + lane * kElemsPerLane;
            if (base + u * kElemsPerWarpIter >= a.slab_elems) break;  // warp-uniform
            const bool active = e0 < a.slab_elems;
            // min and max of the lane's 16 values, two at a time
            __half2 mn2 = as_h2(w[u][0]), mx2 = as_h2(w[u][0]);
#pragma unroll
            for (int k = 1; k < 8; ++k) {
                mn2 = __hmin2(mn2, as_h2(w[u][k]));
                mx2 = __hmax2(mx2, as_h2(w[u][k]));
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
            if (__any_sync(0xffffffffu, scale < 6.103515625e-05f)) quantize_pack16<BITS, true>(w[u], zero, inv, c);
            else quantize_pack16<BITS, false>(w[u], zero, inv, c);
            if (active) {
                store_codes<BITS>(codes + (uint32_t)(e0 / kElemsPerLane) * kLaneBytes, c);
#pragma unroll
                for (int j = 0; j < BITS / 2; ++j) sum += c[j];
                if ((lane & (LPG - 1)) == 0) {
                    const uint32_t p = (uint32_t)__half_as_ushort(scale_h) | ((uint32_t)__half_as_ushort(__float2half_rn(zero)) << 16);
                    params[e0 / (kElemsPerLane * LPG)] = p;
                    sum += p;
                }
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

__device__ __forceinline__ ChunkEntry load_entry(const ChunkEntry *p)
{
    const uint4 lo = *reinterpret_cast<const uint4 *>(p);
    const uint4 hi = *(reinterpret_cast<const uint4 *>(p) + 1);
    ChunkEntry e;
    e.chunk_id = lo.x; e.bits = lo.y;
    e.offset = (uint64_t)lo.z | ((uint64_t)lo.w << 32);
    e.nbytes = (uint64_t)hi.x | ((uint64_t)hi.y << 32);
    e.n_groups = hi.z; e.checksum = hi.w;
    return e;
}

template <int LPG, bool WIDE>
__global__ void __launch_bounds__(kThreads) compress_kernel(const CodecArgs a)
{
    const int lane = threadIdx.x & 31;
    const uint32_t warp = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * kWarpsPerBlock;
    const uint32_t total = (uint32_t)a.n * (uint32_t)a.n_slabs;
    for (uint32_t item = warp; item < total; item += n_warps) {
        uint32_t i, s_idx;
        item_to_chunk_slab(a, item, i, s_idx);
        const ChunkEntry e = load_entry(a.entries + i);
        const __half *src = a.kv_in + slab_offset(a, s_idx, e.chunk_id);
        uint8_t *rec = a.buf + e.offset;
        uint32_t sum;
        if (e.bits == 8) sum = compress_slab<8, LPG, WIDE>(a, src, rec, s_idx, lane);
        else if (e.bits == 4) sum = compress_slab<4, LPG, WIDE>(a, src, rec, s_idx, lane);
        else sum = compress_slab<2, LPG, WIDE>(a, src, rec, s_idx, lane);
        if (s_idx == 0) zero_padding(a, rec, e, lane);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.entries[i].checksum, sum);
    }
}

// ---------------------------------------------------------------------------------------------- dequantize

template <int BITS>
__device__ __forceinline__ void load_codes(const uint8_t *p, uint32_t (&c)[BITS / 2])
{
    if constexpr (BITS == 8)
        asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3]) : "l"(p));
    else if constexpr (BITS == 4)
        asm volatile("ld.global.nc.L1::no_allocate.v2.b32 {%0,%1}, [%2];" : "=r"(c[0]), "=r"(c[1]) : "l"(p));
    else
        asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(c[0]) : "l"(p));
}

// Spread the lane's 16 codes over bytes: code e ends up in byte (e % 4) of b[e / 4] (BITS 8),
// byte (e / 2 % 4) of b[(e % 2) + 2 * (e / 8)] (BITS 4) or byte (e / 4) of b[e % 4] (BITS 2).
template <int BITS>
__device__ __forceinline__ uint32_t code_as_float_bits(const uint32_t (&c)[BITS / 2], const uint32_t (&b)[4], int e)
{
    // 0x4B000000 | q is the binary32 number 2^23 + q
    if constexpr (BITS == 8) return __byte_perm(c[e / 4], 0x4B000000u, 0x7650 | (e % 4));
    else if constexpr (BITS == 4) return __byte_perm(b[(e % 2) + 2 * (e / 8)], 0x4B000000u, 0x7650 | ((e / 2) % 4));
    else return __byte_perm(b[e % 4], 0x4B000000u, 0x7650 | (e / 4));
}

template <int BITS, bool CLAMP>
__device__ __forceinline__ void dequantize16(const uint32_t (&c)[BITS / 2], float scale, float zero, uint32_t (&w)[8])
{
    uint32_t b[4] = {0, 0, 0, 0};
    if constexpr (BITS == 4) {
        b[0] = c[0] & 0x0F0F0F0Fu; b[1] = (c[0] >> 4) & 0x0F0F0F0Fu;
        b[2] = c[1] & 0x0F0F0F0Fu; b[3] = (c[1] >> 4) & 0x0F0F0F0Fu;
    } else if constexpr (BITS == 2) {
        b[0] = c[0] & 0x03030303u; b[1] = (c[0] >> 2) & 0x03030303u;
        b[2] = (c[0] >> 4) & 0x03030303u; b[3] = (c[0] >> 6) & 0x03030303u;
    }
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const float q0 = __fsub_rn(__uint_as_float(code_as_float_bits<BITS>(c, b, 2 * k)), 8388608.0f);      // exact
        const float q1 = __fsub_rn(__uint_as_float(code_as_float_bits<BITS>(c, b, 2 * k + 1)), 8388608.0f);
        // q*scale is exact in binary32, so the fused form rounds once, like multiply-then-add would
        float y0 = __fmaf_rn(q0, scale, zero);
        float y1 = __fmaf_rn(q1, scale, zero);
        if constexpr (CLAMP) {  // zero >= -65504 and scale >= 0: only the upper end can leave the fp16 range
            y0 = fminf(y0, 65504.0f);
            y1 = fminf(y1, 65504.0f);
        }
        w[k] = as_u32(__floats2half2_rn(y0, y1));
    }
}

template <int BITS, int LPG, bool WIDE>
__device__ __forceinline__ uint32_t decompress_slab(const CodecArgs &a, const uint8_t *__restrict__ rec, __half *__restrict__ dst,
                                                    uint32_t s_idx, int lane)
{
    constexpr float kQmax = (float)((1 << BITS) - 1);
    constexpr int kLaneBytes = kElemsPerLane * BITS / 8;
    const uint32_t *params = reinterpret_cast<const uint32_t *>(rec) + (uint64_t)s_idx * a.groups_per_slab;
    const uint8_t *codes = rec + a.codes_off + (uint64_t)s_idx * a.slab_elems * BITS / 8;
    uint32_t sum = 0;
    for (int base = 0; base < a.slab_elems; base += kUnroll * kElemsPerWarpIter) {
        uint32_t c[kUnroll][BITS / 2];
        uint32_t p[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int e0 = base + u * kElemsPerWarpIter + lane * kElemsPerLane;
            if (e0 < a.slab_elems) {
                load_codes<BITS>(codes + (uint32_t)(e0 / kElemsPerLane) * kLaneBytes, c[u]);
                p[u] = __ldg(params + e0 / (kElemsPerLane * LPG));
            } else {
#pragma unroll
                for (int j = 0; j < BITS / 2; ++j) c[u][j] = 0;
                p[u] = 0;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int e0 = base + u * kElemsPerWarpIter + lane * kElemsPerLane;
            if (base + u * kElemsPerWarpIter >= a.slab_elems) break;  // warp-uniform
            const float scale = __half2float(__ushort_as_half((unsigned short)(p[u] & 0xffffu)));
            const float zero = __half2float(__ushort_as_half((unsigned short)(p[u] >> 16)));
            uint32_t w[8];
            if (__any_sync(0xffffffffu, __fmaf_rn(kQmax, scale, zero) > 65504.0f)) dequantize16<BITS, true>(c[u], scale, zero, w);
            else dequantize16<BITS, false>(c[u], scale, zero, w);
            if (e0 < a.slab_elems) {
                store32<WIDE>(dst + e0, w);
#pragma unroll
                for (int j = 0; j < BITS / 2; ++j) sum += c[u][j];
                if ((lane & (LPG - 1)) == 0) sum += p[u];
            }
        }
    }
    return sum;
}

template <int LPG, bool WIDE>
__global__ void __launch_bounds__(kThreads) decompress_kernel(const CodecArgs a)
{
    const int lane = threadIdx.x & 31;
    const uint32_t warp = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    const uint32_t n_warps = gridDim.x * kWarpsPerBlock;
    const uint32_t total = (uint32_t)a.n * (uint32_t)a.n_slabs;
    for (uint32_t item = warp; item < total; item += n_warps) {
        uint32_t i, s_idx;
        item_to_chunk_slab(a, item, i, s_idx);
        const ChunkEntry e = load_entry(a.entries + i);
        const uint8_t *rec = a.buf + e.offset;
        __half *dst = a.kv_out + slab_offset(a, s_idx, e.chunk_id);
        uint32_t sum;
        if (e.bits == 8) sum = decompress_slab<8, LPG, WIDE>(a, rec, dst, s_idx, lane);
        else if (e.bits == 4) sum = decompress_slab<4, LPG, WIDE>(a, rec, dst, s_idx, lane);
        else sum = decompress_slab<2, LPG, WIDE>(a, rec, dst, s_idx, lane);
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
    a.slab_major = 1;  // measured: linear KV addresses beat linear record addresses (decompress 0.54 vs 0.72 ms on the 7B shape)
    a.entries = reinterpret_cast<ChunkEntry *>(static_cast<uint8_t *>(workspace) + kWsEntriesOffset);
    a.sums = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + ws_sums_offset(n));
    return LLMS_OK;
}

// Persistent grid: as many CTAs as are resident at once, or fewer when there is less work.
template <typename K>
static int grid_for(K kernel, int64_t items)
{
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm <= 0) {
        cudaGetLastError();
        per_sm = 2;
    }
    const int64_t want = (items + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int64_t cap = (int64_t)sm_count() * per_sm;
    return (int)(want < cap ? want : cap);
}

// 256-bit accesses need every slab to start on a 32-byte boundary
static bool wide_ok(const llms_kv_desc &d, const void *kv)
{
    return aligned(kv, 32) && ((d.stride_l | d.stride_s | d.stride_h) % 16) == 0;
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
    if ((uint64_t)n * (uint64_t)slabs_per_chunk(*desc) > 0x7fffffffull) return LLMS_ERR_UNSUPPORTED;
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
    const int64_t items = (int64_t)n * a.n_slabs;
    const bool wide = wide_ok(*desc, kv);
    rc = dispatch_lpg(desc->group_size, [&](auto lpg) {
        constexpr int kLpg = decltype(lpg)::value;
        if (wide) compress_kernel<kLpg, true><<<grid_for(compress_kernel<kLpg, true>, items), kThreads, 0, st>>>(a);
        else compress_kernel<kLpg, false><<<grid_for(compress_kernel<kLpg, false>, items), kThreads, 0, st>>>(a);
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
    const int64_t items = (int64_t)n * a.n_slabs;
    const bool wide = wide_ok(*desc, kv_out);
    rc = dispatch_lpg(desc->group_size, [&](auto lpg) {
        constexpr int kLpg = decltype(lpg)::value;
        if (wide) decompress_kernel<kLpg, true><<<grid_for(decompress_kernel<kLpg, true>, items), kThreads, 0, st>>>(a);
        else decompress_kernel<kLpg, false><<<grid_for(decompress_kernel<kLpg, false>, items), kThreads, 0, st>>>(a);
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
