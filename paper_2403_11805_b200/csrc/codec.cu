// Chunk codec kernels for sm_100a: group quantize + bit-pack (swap-out) and unpack + dequantize (swap-in).
//
// Work unit = one warp pass over a slab (chunk_len*head_dim contiguous fp16 of one chunk, layer, K/V, head):
// 2048 elements.  Warps of a persistent grid walk the units with a stride; the loads of the next unit are
// issued before the current one is computed (register buffers), and the bit-width is uniform per launch.
//
// Encoder: every load instruction of a warp reads 1 KiB of consecutive bytes (piece j of lane L = elements
// j*512 + L*16; with 128 consecutive bytes per lane instead, a streaming probe reached 5.6 instead of 6.9 TB/s);
// the unit is then transposed through padded shared memory so that a lane owns 64 consecutive elements.  A
// group of G >= 64 channels is G/64 neighbouring lanes (min/max by xor-shuffles on a packed (min, -max) half2);
// smaller groups sit inside a lane.  A lane's packed codes are 16/32/64 contiguous bytes at 2/4/8 bits.  The
// unit two strides ahead is pulled into L2 by a bulk prefetch.
//
// Decoder: keeps the interleaved split for its stores (1 KiB of consecutive bytes per store instruction) and
// needs no lane cooperation: each piece looks its group's parameters up.
//
// The arithmetic is fixed by the record format (see llms.h): every binary32 operation is a single IEEE
// round-to-nearest operation (intrinsics, or sm_100 mixed-precision PTX whose fp16 inputs convert exactly),
// nothing is contracted or approximated.
#include <string.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <utility>
#include <vector>

#include "llms_internal.cuh"

namespace llms {

constexpr int kWarpsPerBlock = 8;
constexpr int kThreads = kWarpsPerBlock * 32;
constexpr int kPieceElems = 16;                 // one 32-byte access
constexpr int kPieces = 4;                      // pieces per lane per pass
constexpr int kLaneElems = kPieces * kPieceElems;
constexpr int kPassElems = 32 * kLaneElems;     // 2048 elements = 4 KiB of fp16
// 32-bit words that hold the packed codes of one piece; at 1 bit a piece is the low half of one word
__host__ __device__ constexpr int piece_words(int bits) { return bits >= 2 ? bits / 2 : 1; }
constexpr uint32_t kPrefetchAhead = 2;          // compress: units ahead that are pulled into L2 (measured: 2 -> 0.521 ms,
                                                // 3 -> 0.535, 5 -> 0.59, 8 -> 0.79 for compress on the 7B shape)

// Division by a launch-time constant as multiply-high and shift: exact for numerators below 2^31.
struct FastDiv {
    uint32_t d, mul, shr;
    __host__ void set(uint32_t divisor)
    {
        d = divisor;
        mul = 0;
        shr = 0;
        if (divisor > 1) {
            uint32_t lg = 0;
            while ((1ull << lg) < divisor) ++lg;         // ceil(log2 d)
            const uint32_t p = 31 + lg;
            mul = (uint32_t)(((1ull << p) + divisor - 1) / divisor);
            shr = p - 32;
        }
    }
    __device__ __forceinline__ void divmod(uint32_t x, uint32_t &q, uint32_t &r) const
    {
        q = d == 1 ? x : (__umulhi(x, mul) >> shr);
        r = x - q * d;
    }
};

struct CodecArgs {
    const __half *kv_in;   // compress: source
    __half *kv_out;        // decompress: destination
    uint8_t *buf;          // swap buffer (written by compress, read by decompress)
    ChunkEntry *entries;   // n entries in the workspace (caller's order)
    uint32_t *sums;        // decompress: recomputed checksums
    const uint32_t *order; // entry indices grouped by bit-width; this launch covers order[0 .. n)
    const UnitEntry *table; // the same chunks with what a unit needs to know, one 16-byte load
    uint32_t *feed;        // channel-wise launches: this launch's work-split counters (zero at the start)
    int n;                 // chunks of this launch (all of one bit-width)
    int n_slabs;           // slabs per chunk
    int slab_elems;        // chunk_len * head_dim
    int groups_per_slab;
    int n_kv_heads;
    int passes;            // warp passes per slab (1 when packed)
    int unit_rows;         // slabs per chunk, or, packed, units per chunk
    int packed;            // 1: slabs shorter than a pass, a unit covers slabs_per_unit whole slabs (see UnitPos)
    int slab_shift;        // packed: log2(slab_elems)
    int slabs_per_unit;    // packed: kPassElems / slab_elems
    uint32_t chunk_elems;  // n_slabs * slab_elems
    FastDiv div_passes, div_n, div_heads;
    uint32_t total_units;  // n * n_slabs * passes
    uint32_t codes_off;    // byte offset of the code stream in a record
    uint32_t params_bytes; // 4 * n_groups
    int64_t stride_l, stride_s, stride_h, chunk_stride;
};

// Where a unit's data is.  Units are numbered slab-major: consecutive units walk the passes of a slab, then
// the listed chunks of one slab index, so KV addresses run linearly when the chunk ids are consecutive
// (measured: faster than walking the slabs of one chunk, which makes the record addresses linear instead).
//
// Packed units: when a slab is shorter than a pass (small chunk_len * head_dim) and divides it, a unit covers
// kPassElems / slab_elems consecutive slabs of one chunk instead of a mostly empty pass of one.  In the record
// those slabs are adjacent (codes and parameters are stored in slab order), so s_idx and e0 below keep their
// meaning for every record offset, with e0 running past the end of slab s_idx; only the KV addresses have to be
// looked up slab by slab.
struct UnitPos {
    uint32_t i, k, s_idx, chunk_id;  // i: entry index (caller's order), k: position in this launch's list
    uint64_t rec_off;
    int e0;                // first element of this lane, counted from the start of slab s_idx
    int limit;             // elements of this unit that exist, counted from the unit's first element
    int64_t kv_off;        // element offset of the unit's first element in the KV tensor (not packed)
};

__device__ __forceinline__ int64_t slab_offset(const CodecArgs &a, uint32_t s_idx, uint32_t chunk)
{
    uint32_t ls, h;
    a.div_heads.divmod(s_idx, ls, h);
    return (int64_t)(ls >> 1) * a.stride_l + (int64_t)(ls & 1) * a.stride_s + (int64_t)h * a.stride_h +
           (int64_t)chunk * a.chunk_stride;
}

template <bool PACKED>
__device__ __forceinline__ void decode_unit(const CodecArgs &a, uint32_t unit, int lane, UnitPos &u)
{
    uint32_t item, pass, k;
    a.div_passes.divmod(unit, item, pass);
    uint32_t row;
    a.div_n.divmod(item, row, k);
    u.k = k;
    const uint4 ent = *reinterpret_cast<const uint4 *>(a.table + k);       // chunk, entry, record offset: one load
    u.chunk_id = ent.x;
    u.i = ent.y;
    u.rec_off = (uint64_t)ent.z | ((uint64_t)ent.w << 32);
    if constexpr (PACKED) {
        u.s_idx = row * (uint32_t)a.slabs_per_unit;
        u.e0 = lane * kLaneElems;
        u.limit = (int)min((uint32_t)kPassElems, a.chunk_elems - row * kPassElems);
    } else {
        u.s_idx = row;
        u.e0 = (int)pass * kPassElems + lane * kLaneElems;
        u.limit = min(kPassElems, a.slab_elems - (int)pass * kPassElems);
        u.kv_off = slab_offset(a, row, ent.x) + (int)pass * kPassElems;
    }
}

// KV offset of element v of a unit (v counted from the unit's first element)
template <bool PACKED>
__device__ __forceinline__ int64_t unit_elem_offset(const CodecArgs &a, uint32_t s_idx, uint32_t chunk, int pass_e0, int v)
{
    if constexpr (PACKED) return slab_offset(a, s_idx + (uint32_t)(v >> a.slab_shift), chunk) + (v & (a.slab_elems - 1));
    return slab_offset(a, s_idx, chunk) + pass_e0 + v;
}

__device__ __forceinline__ __half2 as_h2(uint32_t u) { return *reinterpret_cast<__half2 *>(&u); }
__device__ __forceinline__ uint32_t as_u32(__half2 h) { return *reinterpret_cast<uint32_t *>(&h); }

__device__ __forceinline__ void split_halves(uint32_t w, unsigned short &lo, unsigned short &hi)
{
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w));
}

// fp32(x) + c with one rounding; x is an fp16 bit pattern (converts exactly)
__device__ __forceinline__ float add_f32_f16(unsigned short x, float c)
{
    float d;
    asm("add.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    return d;
}

// fp32(a) * fp32(b) + c with one rounding; a, b are fp16 bit patterns
__device__ __forceinline__ float fma_f32_f16(unsigned short x, unsigned short y, float c)
{
    float d;
    asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(d) : "h"(x), "h"(y), "f"(c));
    return d;
}

// ---------------------------------------------------------------------------------------------- checked build
// Compiled with LLMS_DEBUG_BOUNDS (python -m paper_2403_11805_b200.build --debug-bounds: a library of its own, never the
// one the binding loads by default) every access the group-wise kernels make to the KV tensor and to the swap buffer
// is first compared with the two address ranges the host set for the call; an access outside them is counted, its
// address kept if it is the first, and skipped (loads give zeros).  Nothing of this exists in the ordinary build.
#ifdef LLMS_DEBUG_BOUNDS
struct DebugRanges {
    unsigned long long lo[2], hi[2];
};
__device__ DebugRanges g_debug_ranges;
__device__ unsigned int g_debug_violations;
__device__ unsigned long long g_debug_first_address;

__device__ __forceinline__ bool access_ok(const void *p, unsigned int bytes)
{
    const unsigned long long a = reinterpret_cast<unsigned long long>(p);
#pragma unroll
    for (int r = 0; r < 2; ++r)
        if (a >= g_debug_ranges.lo[r] && a + bytes <= g_debug_ranges.hi[r]) return true;
    if (atomicAdd(&g_debug_violations, 1u) == 0) g_debug_first_address = a;
    return false;
}
#else
__device__ __forceinline__ bool access_ok(const void *, unsigned int) { return true; }
#endif

// Global accesses of data that is touched once: no L1 allocation.  WIDE: one 256-bit access (32-byte aligned).
template <bool WIDE>
__device__ __forceinline__ void load32(const void *p, uint32_t (&w)[8])
{
    if (!access_ok(p, 32)) {
#pragma unroll
        for (int k = 0; k < 8; ++k) w[k] = 0;
        return;
    }
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

__device__ __forceinline__ void st256(void *p, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t a4,
                                      uint32_t a5, uint32_t a6, uint32_t a7)
{
    if (!access_ok(p, 32)) return;
    asm volatile("st.global.L1::no_allocate.v8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"
                 :: "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(a4), "r"(a5), "r"(a6), "r"(a7), "l"(p) : "memory");
}
__device__ __forceinline__ void st128(void *p, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3)
{
    if (!access_ok(p, 16)) return;
    asm volatile("st.global.L1::no_allocate.v4.b32 [%4], {%0,%1,%2,%3};" :: "r"(a0), "r"(a1), "r"(a2), "r"(a3), "l"(p) : "memory");
}
__device__ __forceinline__ void st64(void *p, uint32_t a0, uint32_t a1)
{
    if (!access_ok(p, 8)) return;
    asm volatile("st.global.L1::no_allocate.v2.b32 [%2], {%0,%1};" :: "r"(a0), "r"(a1), "l"(p) : "memory");
}
__device__ __forceinline__ void st32(void *p, uint32_t a0)
{
    if (!access_ok(p, 4)) return;
    asm volatile("st.global.L1::no_allocate.b32 [%1], %0;" :: "r"(a0), "l"(p) : "memory");
}
__device__ __forceinline__ void st16(void *p, uint32_t a0)
{
    if (!access_ok(p, 2)) return;
    asm volatile("st.global.L1::no_allocate.b16 [%1], %0;" :: "h"((unsigned short)a0), "l"(p) : "memory");
}
__device__ __forceinline__ void ld16(const void *p, uint32_t *w)
{
    if (!access_ok(p, 2)) {
        w[0] = 0;
        return;
    }
    unsigned short v;
    asm volatile("ld.global.nc.L1::no_allocate.b16 %0, [%1];" : "=h"(v) : "l"(p));
    w[0] = v;
}
__device__ __forceinline__ void ld256(const void *p, uint32_t *w)
{
    if (!access_ok(p, 32)) {
        w[0] = 0;
        w[1] = 0;
        w[2] = 0;
        w[3] = 0;
        w[4] = 0;
        w[5] = 0;
        w[6] = 0;
        w[7] = 0;
        return;
    }
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]), "=r"(w[4]), "=r"(w[5]), "=r"(w[6]), "=r"(w[7]) : "l"(p));
}
__device__ __forceinline__ void ld128(const void *p, uint32_t *w)
{
    if (!access_ok(p, 16)) {
        w[0] = 0;
        w[1] = 0;
        w[2] = 0;
        w[3] = 0;
        return;
    }
    asm volatile("ld.global.nc.L1::no_allocate.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(w[0]), "=r"(w[1]), "=r"(w[2]), "=r"(w[3]) : "l"(p));
}
__device__ __forceinline__ void ld64(const void *p, uint32_t *w)
{
    if (!access_ok(p, 8)) {
        w[0] = 0;
        w[1] = 0;
        return;
    }
    asm volatile("ld.global.nc.L1::no_allocate.v2.b32 {%0,%1}, [%2];" : "=r"(w[0]), "=r"(w[1]) : "l"(p));
}
__device__ __forceinline__ void ld32(const void *p, uint32_t *w)
{
    if (!access_ok(p, 4)) {
        w[0] = 0;
        return;
    }
    asm volatile("ld.global.nc.L1::no_allocate.b32 %0, [%1];" : "=r"(w[0]) : "l"(p));
}

template <bool WIDE>
__device__ __forceinline__ void store32(void *p, const uint32_t (&w)[8])
{
    if constexpr (WIDE) {
        st256(p, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
    } else {
        st128(p, w[0], w[1], w[2], w[3]);
        st128(static_cast<char *>(p) + 16, w[4], w[5], w[6], w[7]);
    }
}

// Group geometry for a lane that owns 64 consecutive elements.
template <int G>
struct Geo {
    static constexpr int kLanesPerGroup = G >= kLaneElems ? G / kLaneElems : 1;
    static constexpr int kGroupsPerLane = G >= kLaneElems ? 1 : kLaneElems / G;
    static constexpr int kPiecesPerGroup = kPieces / kGroupsPerLane;
};

// Record checksums are sums of 32-bit words, so partial sums may be added in any order.  A launch with few
// chunks would send every unit's partial sum to the same few addresses (measured: with 5 chunks per launch the
// same-address atomics made the kernels up to twice as slow), so a CTA first adds them up in shared memory,
// one slot per chunk of the launch, and sends one atomic per chunk when it ends.  Launches with more chunks than
// slots add straight to global memory, where that many addresses do not collide.
constexpr int kSumSlots = 1024;

__device__ __forceinline__ void cta_sums_clear(uint32_t *slots, int n)
{
    if (n <= kSumSlots)
        for (int k = threadIdx.x; k < n; k += kThreads) slots[k] = 0;
    __syncthreads();
}

__device__ __forceinline__ void unit_sum_add(uint32_t *slots, int n, uint32_t k, uint32_t *global_slot, uint32_t sum, int lane)
{
    sum = __reduce_add_sync(0xffffffffu, sum);
    if (lane == 0) {
        if (n <= kSumSlots) atomicAdd(&slots[k], sum);
        else atomicAdd(global_slot, sum);
    }
}

// ---------------------------------------------------------------------------------------------- quantize

// Adding 1.5 * 2^23 rounds a value in [0, 2^22) to an integer, ties to even, and leaves that integer in the
// low mantissa bits: bits = 0x4B400000 + q.
constexpr float kRoundMagic = 12582912.0f;
constexpr uint32_t kRoundMagicBits = 0x4B400000u;
constexpr float kMinNormalHalf = 6.103515625e-05f;

struct GroupParams {
    float neg_zero_point;  // -(minimum)
    float inv;             // 1 / scale, or 0 when scale == 0 (every code becomes 0)
    uint32_t word;         // scale bits | zero-point bits << 16
    bool needs_clamp;      // scale is a subnormal fp16 number (or 0): (x - zero)/scale may pass 2^b - 1
};

// mm = (min, -max) of a group
template <int BITS>
__device__ __forceinline__ GroupParams group_params(__half2 mm)
{
    constexpr float kQmax = (float)((1 << BITS) - 1);
    // adding +0 turns a -0 minimum or maximum into +0 and changes nothing else
    const float zero = __fadd_rn(__low2float(mm), 0.0f);
    const float top = __fadd_rn(-__high2float(mm), 0.0f);
    // a range above 65504 (possible at 1 bit only) keeps the largest finite scale
    unsigned short scale_bits;
    asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(scale_bits) : "f"(__fdiv_rn(__fsub_rn(top, zero), kQmax)));
    const __half scale_h = __ushort_as_half(scale_bits);
    const float scale = __half2float(scale_h);
    GroupParams g;
    g.neg_zero_point = -zero;
    g.inv = scale == 0.0f ? 0.0f : __frcp_rn(scale);
    g.word = (uint32_t)__half_as_ushort(scale_h) | ((uint32_t)__half_as_ushort(__float2half_rn(zero)) << 16);
    g.needs_clamp = scale < kMinNormalHalf;
    return g;
}

// min and max of 16 values as two half2 (element-wise over the pairs)
__device__ __forceinline__ void piece_minmax(const uint32_t (&w)[8], __half2 &mn2, __half2 &mx2)
{
    mn2 = as_h2(w[0]);
    mx2 = as_h2(w[0]);
#pragma unroll
    for (int k = 1; k < 8; ++k) {
        mn2 = __hmin2(mn2, as_h2(w[k]));
        mx2 = __hmax2(mx2, as_h2(w[k]));
    }
}

// Quantize 16 values and pack them into BITS/2 words.  No clamp: only valid when the scale is a normal fp16
// number, where (x - zero) / scale stays below 2^BITS - 1/2.
template <int BITS>
__device__ __forceinline__ void quantize_piece(const uint32_t (&w)[8], float neg_zero, float inv, uint32_t (&out)[piece_words(BITS)])
{
    uint32_t t[16];
    const float2 inv2 = make_float2(inv, inv);
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        unsigned short lo, hi;
        split_halves(w[k], lo, hi);
        // (x - zero) * inv, two roundings; >= 0 because zero is the minimum.  The pair's two multiplications are one
        // packed binary32 instruction (same rounding per value).  The rounding additions stay scalar: a packed
        // multiplication followed by a packed addition comes out of the assembler as one fused operation, which
        // rounds once and gives another code a few times per million values.
        const float2 d = make_float2(add_f32_f16(lo, neg_zero), add_f32_f16(hi, neg_zero));
        const float2 r = __fmul2_rn(d, inv2);
        t[2 * k] = __float_as_uint(__fadd_rn(r.x, kRoundMagic));
        t[2 * k + 1] = __float_as_uint(__fadd_rn(r.y, kRoundMagic));
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
        constexpr int kPerWord = BITS >= 2 ? 32 / BITS : 16;
        uint32_t ones = 0;
#pragma unroll
        for (int k = 0; k < kPerWord; ++k) ones += 1u << (k * BITS);
        const uint32_t bias = kRoundMagicBits * ones;
#pragma unroll
        for (int j = 0; j < piece_words(BITS); ++j) {
            uint32_t acc = 0u - bias;
#pragma unroll
            for (int k = 0; k < kPerWord; ++k) acc += t[j * kPerWord + k] << (k * BITS);
            out[j] = acc;
        }
    }
}

// The rare case (subnormal scale): same arithmetic plus the clamp, written for size, not speed.
__device__ __noinline__ void quantize_piece_clamped(const uint32_t *w, float neg_zero, float inv, int bits, uint32_t *out)
{
    const float qmax = (float)((1 << bits) - 1);
    for (int j = 0; j < piece_words(bits); ++j) out[j] = 0;
    for (int k = 0; k < 16; ++k) {
        const unsigned short x = (unsigned short)(w[k >> 1] >> ((k & 1) * 16));
        const float v = fminf(__fmul_rn(add_f32_f16(x, neg_zero), inv), qmax);
        const uint32_t q = (uint32_t)__float2int_rn(v);
        out[(k * bits) >> 5] |= q << ((k * bits) & 31);
    }
}

template <int BITS, int G, bool WIDE>
__device__ __forceinline__ uint32_t compress_unit_bits(const CodecArgs &a, const UnitPos &u, const uint32_t (&w)[kPieces][8],
                                                       uint8_t *__restrict__ rec, int lane)
{
    using geo = Geo<G>;
    constexpr int kPieceBytes = kPieceElems * BITS / 8;
    const int le0 = lane * kLaneElems;  // this lane's first element inside the unit
    // ---- group minima and maxima
    GroupParams gp[geo::kGroupsPerLane];
    {
        __half2 mn2[kPieces], mx2[kPieces];
#pragma unroll
        for (int j = 0; j < kPieces; ++j) piece_minmax(w[j], mn2[j], mx2[j]);
#pragma unroll
        for (int g = 0; g < geo::kGroupsPerLane; ++g) {
            __half2 mn = mn2[g * geo::kPiecesPerGroup], mx = mx2[g * geo::kPiecesPerGroup];
#pragma unroll
            for (int j = 1; j < geo::kPiecesPerGroup; ++j) {
                mn = __hmin2(mn, mn2[g * geo::kPiecesPerGroup + j]);
                mx = __hmax2(mx, mx2[g * geo::kPiecesPerGroup + j]);
            }
            // (min, -max) in one register: a single min per shuffle step reduces both
            __half2 mm = __halves2half2(__hmin(__low2half(mn), __high2half(mn)), __hneg(__hmax(__low2half(mx), __high2half(mx))));
#pragma unroll
            for (int m = geo::kLanesPerGroup / 2; m > 0; m >>= 1)
                mm = __hmin2(mm, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mm), m)));
            gp[g] = group_params<BITS>(mm);
        }
    }
    // ---- codes
    uint32_t c[kPieces][piece_words(BITS)];
    bool any_clamp = false;
#pragma unroll
    for (int g = 0; g < geo::kGroupsPerLane; ++g)  // groups past the end of the slab (loaded as zeros) do not count
        any_clamp |= gp[g].needs_clamp && le0 + (geo::kGroupsPerLane > 1 ? g * G : 0) < u.limit;
    if (__any_sync(0xffffffffu, any_clamp)) {
#pragma unroll
        for (int j = 0; j < kPieces; ++j) {
            const GroupParams &g = gp[j / geo::kPiecesPerGroup];
            uint32_t tmp_in[8], tmp_out[4];
#pragma unroll
            for (int k = 0; k < 8; ++k) tmp_in[k] = w[j][k];
            quantize_piece_clamped(tmp_in, g.neg_zero_point, g.inv, BITS, tmp_out);
#pragma unroll
            for (int k = 0; k < piece_words(BITS); ++k) c[j][k] = tmp_out[k];
        }
    } else {
#pragma unroll
        for (int j = 0; j < kPieces; ++j) {
            const GroupParams &g = gp[j / geo::kPiecesPerGroup];
            quantize_piece<BITS>(w[j], g.neg_zero_point, g.inv, c[j]);
        }
    }
    // ---- stores
    uint8_t *codes = rec + a.codes_off + (uint64_t)u.s_idx * a.slab_elems * BITS / 8 + (uint32_t)u.e0 * BITS / 8;
    uint32_t *params = reinterpret_cast<uint32_t *>(rec) + (uint64_t)u.s_idx * a.groups_per_slab + (uint32_t)u.e0 / G;
    uint32_t sum = 0;
    const bool lane_full = le0 + kLaneElems <= u.limit;
    constexpr uintptr_t kLaneAlign = BITS == 1 ? 7 : BITS == 2 ? 15 : 31;
    if (lane_full && (reinterpret_cast<uintptr_t>(codes) & kLaneAlign) == 0) {
        if constexpr (BITS == 8) {
            st256(codes, c[0][0], c[0][1], c[0][2], c[0][3], c[1][0], c[1][1], c[1][2], c[1][3]);
            st256(codes + 32, c[2][0], c[2][1], c[2][2], c[2][3], c[3][0], c[3][1], c[3][2], c[3][3]);
        } else if constexpr (BITS == 4) {
            st256(codes, c[0][0], c[0][1], c[1][0], c[1][1], c[2][0], c[2][1], c[3][0], c[3][1]);
        } else if constexpr (BITS == 2) {
            st128(codes, c[0][0], c[1][0], c[2][0], c[3][0]);
        } else {
            st64(codes, c[0][0] | (c[1][0] << 16), c[2][0] | (c[3][0] << 16));
        }
        if constexpr (BITS == 1) {
            sum = c[0][0] + (c[1][0] << 16) + c[2][0] + (c[3][0] << 16);
        } else {
#pragma unroll
            for (int j = 0; j < kPieces; ++j)
#pragma unroll
                for (int k = 0; k < piece_words(BITS); ++k) sum += c[j][k];
        }
    } else {
#pragma unroll
        for (int j = 0; j < kPieces; ++j) {
            if (le0 + j * kPieceElems < u.limit) {
                if constexpr (BITS == 8) st128(codes + j * kPieceBytes, c[j][0], c[j][1], c[j][2], c[j][3]);
                else if constexpr (BITS == 4) st64(codes + j * kPieceBytes, c[j][0], c[j][1]);
                else if constexpr (BITS == 2) st32(codes + j * kPieceBytes, c[j][0]);
                else st16(codes + j * kPieceBytes, c[j][0]);
                if constexpr (BITS == 1) {  // half a word: which half follows from the address (records are 256-byte aligned)
                    sum += c[j][0] << ((reinterpret_cast<uintptr_t>(codes + j * kPieceBytes) & 2) * 8);
                } else {
#pragma unroll
                    for (int k = 0; k < piece_words(BITS); ++k) sum += c[j][k];
                }
            }
        }
    }
    if constexpr (geo::kGroupsPerLane == 1) {
        if (le0 < u.limit && (lane & (geo::kLanesPerGroup - 1)) == 0) {
            st32(params, gp[0].word);
            sum += gp[0].word;
        }
    } else {
#pragma unroll
        for (int g = 0; g < geo::kGroupsPerLane; ++g) {
            if (le0 + g * G < u.limit) {
                st32(params + g, gp[g].word);
                sum += gp[g].word;
            }
        }
    }
    return sum;
}

// Zero the two padding runs of a record (after the parameter block, after the code stream).
__device__ __forceinline__ void zero_padding(const CodecArgs &a, uint8_t *rec, uint32_t bits, int lane)
{
    for (uint32_t k = a.params_bytes + lane; k < a.codes_off; k += 32)
        if (access_ok(rec + k, 1)) rec[k] = 0;
    const uint64_t codes_end = a.codes_off + (uint64_t)a.n_slabs * a.slab_elems * bits / 8;
    const uint64_t nbytes = (codes_end + 255) / 256 * 256;
    for (uint64_t k = codes_end + lane; k < nbytes; k += 32)
        if (access_ok(rec + k, 1)) rec[k] = 0;
}

// The unit is fetched so that every load instruction of the warp reads 1 KiB of consecutive bytes (piece j of
// lane L = elements [j*512 + L*16, +16) of the pass): measured on this part, a stream read with 128 consecutive
// bytes per lane tops out near 5.6 TB/s, one with consecutive lanes on consecutive 32 bytes near 6.9 TB/s.
template <bool WIDE, bool PACKED>
__device__ __forceinline__ void load_unit(const CodecArgs &a, const UnitPos &u, int lane, uint32_t (&w)[kPieces][8])
{
    const __half *src0 = nullptr;  // piece 0 when the unit lies inside one slab
    if constexpr (!PACKED) src0 = a.kv_in + u.kv_off + lane * kPieceElems;
#pragma unroll
    for (int j = 0; j < kPieces; ++j) {
        const int v = j * (32 * kPieceElems) + lane * kPieceElems;
        if (v < u.limit) {
            if constexpr (PACKED) load32<WIDE>(a.kv_in + unit_elem_offset<true>(a, u.s_idx, u.chunk_id, 0, v), w[j]);
            else load32<WIDE>(src0 + j * (32 * kPieceElems), w[j]);
        } else {
#pragma unroll
            for (int k = 0; k < 8; ++k) w[j][k] = 0;  // past the end: whole inactive groups
        }
    }
}

// ... and brought to the layout the arithmetic wants (lane L holds elements [L*64, +64) of the pass) through the
// warp's patch of shared memory: stored from the registers the loads landed in, read back into others.  Rows of 128 bytes are padded to 144: both the 32-byte-per-lane writes and the
// 128-byte-per-lane reads are then free of bank conflicts.
constexpr int kTransposeRowBytes = 128 + 16;
constexpr int kTransposeBytes = 32 * kTransposeRowBytes;

__device__ __forceinline__ void patch_store(const uint32_t (&raw)[kPieces][8], unsigned char *patch, int lane)
{
#pragma unroll
    for (int j = 0; j < kPieces; ++j) {
        // piece j of this lane = 16-byte chunks 64j + 2L and 64j + 2L + 1 of the unit; chunk n -> row n/8, column n%8
        unsigned char *dst = patch + (8 * j + (lane >> 2)) * kTransposeRowBytes + (lane & 3) * 32;
        *reinterpret_cast<uint4 *>(dst) = make_uint4(raw[j][0], raw[j][1], raw[j][2], raw[j][3]);
        *reinterpret_cast<uint4 *>(dst + 16) = make_uint4(raw[j][4], raw[j][5], raw[j][6], raw[j][7]);
    }
}

__device__ __forceinline__ void patch_load(unsigned char *patch, int lane, uint32_t (&w)[kPieces][8])
{
    __syncwarp();
    const unsigned char *row = patch + lane * kTransposeRowBytes;
#pragma unroll
    for (int j = 0; j < kPieces; ++j) {
        const uint4 lo = *reinterpret_cast<const uint4 *>(row + j * 32);
        const uint4 hi = *reinterpret_cast<const uint4 *>(row + j * 32 + 16);
        w[j][0] = lo.x; w[j][1] = lo.y; w[j][2] = lo.z; w[j][3] = lo.w;
        w[j][4] = hi.x; w[j][5] = hi.y; w[j][6] = hi.z; w[j][7] = hi.w;
    }
    __syncwarp();  // the patch is free for the next unit
}

// Ask for a unit's KV bytes to be brought into L2 (one bulk prefetch by one lane): the register loads of that
// unit, issued one unit later, then find them there instead of waiting for DRAM.
template <bool PACKED>
__device__ __forceinline__ void prefetch_unit_l2(const CodecArgs &a, const UnitPos &u, int lane)
{
    if constexpr (PACKED) {  // one prefetch per slab of the unit
        if (lane < a.slabs_per_unit && lane * a.slab_elems < u.limit) {
            const __half *src = a.kv_in + slab_offset(a, u.s_idx + lane, u.chunk_id);
            asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(src), "r"((uint32_t)a.slab_elems * 2) : "memory");
        }
    } else if (lane == 0) {
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(a.kv_in + u.kv_off), "r"((uint32_t)u.limit * 2) : "memory");
    }
}

template <int BITS, int G, bool WIDE>
__device__ __forceinline__ void compress_unit(const CodecArgs &a, const UnitPos &u, const uint32_t (&w)[kPieces][8], int lane,
                                              uint32_t *sum_slots)
{
    uint8_t *rec = a.buf + u.rec_off;
    const uint32_t sum = compress_unit_bits<BITS, G, WIDE>(a, u, w, rec, lane);
    if (u.s_idx == 0 && u.e0 < kPassElems) zero_padding(a, rec, BITS, lane);  // first pass of the chunk's first slab
    unit_sum_add(sum_slots, a.n, u.k, &a.entries[u.i].checksum, sum, lane);
}

// ---------------------------------------------------------------------------------------------- work split
// Which unit a warp takes next.  With a fixed split (warp w takes units w, w + W, w + 2W, ...) the kernel lasts as
// long as its slowest warp, and the memory system does not serve all SMs at the same rate: in a plain stream with
// the decoder's 1:4 read:write mix and a fixed split the CTAs ended between 305 and 454 us around a median of 378
// (measured), a sixth of the time lost to waiting for the last ones.  Here only a warp's first batch of units is
// fixed (batch number = warp number); every further batch number is drawn from a counter in the workspace header,
// one draw ahead of need, so the round trip of the atomic hides behind a batch of work.  One counter would take a
// draw every few nanoseconds, so the warps are spread over kFeedCounters of them, 128 bytes apart: counter j hands
// out the batches W + j, W + j + C, W + j + 2C, ...  Consecutive draws get neighbouring units, so at any moment the
// grid still works on one narrow band of addresses, as with the fixed split.
constexpr int kFeedCounters = 16;
constexpr int kFeedStrideWords = 32;

struct UnitFeed {
    uint32_t *ctr;
    uint32_t slot, n_slots, n_warps, batch, cur, left, pending, total;

    __device__ __forceinline__ void start(uint32_t *counters, uint32_t total_units, int lane)
    {
        const uint32_t gw = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
        n_warps = gridDim.x * kWarpsPerBlock;
        n_slots = min((uint32_t)kFeedCounters, n_warps);  // every counter has warps that draw from it
        slot = gw % n_slots;
        ctr = counters + slot * kFeedStrideWords;
        total = total_units;
        batch = total_units >= 4 * n_warps ? 2u : 1u;     // little work: single units, so that every warp gets some
        cur = gw * batch;
        left = batch;
        pending = 0;
        if (cur < total && lane == 0) pending = atomicAdd(ctr, 1u);
    }
    // The next unit of this warp; total or more when there is none (and then on every later call too).  Called by
    // all lanes of the warp together.
    __device__ __forceinline__ uint32_t pop(int lane)
    {
        if (left == 0) {
            const uint32_t drawn = __shfl_sync(0xffffffffu, pending, 0);
            cur = (n_warps + drawn * n_slots + slot) * batch;
            left = batch;
            if (cur < total && lane == 0) pending = atomicAdd(ctr, 1u);
        }
        --left;
        return cur++;
    }
};

// The chunks of one bit-width, start to finish: one phase of the kernel below.
template <int BITS, int G, bool WIDE, bool PACKED>
__device__ __forceinline__ void compress_phase(const CodecArgs &a, uint32_t *counters, unsigned char (*patches)[kTransposeBytes],
                                               uint32_t *sum_slots)
{
    const int lane = threadIdx.x & 31;
    UnitFeed feed;
    feed.start(counters, a.total_units, lane);
    const uint32_t unit = feed.pop(lane);
    cta_sums_clear(sum_slots, a.n);
    if (unit < a.total_units) {
        unsigned char *patch = patches[threadIdx.x >> 5];
        // A unit is decoded once, two turns ahead of its own: then its bytes are asked into L2, one trip later its
        // loads are issued (pn -> pb), another trip later it is computed (pb -> pa).  The loads land in `raw`; a trip
        // first puts the current unit's raw registers into the warp's patch of shared memory, then issues the next
        // unit's loads into the same registers, then reads the current unit back in the layout the arithmetic wants
        // (`cur`).  One unit per trip: unrolled by two the loop no longer fits the instruction cache well and the
        // kernel is 1.5% slower (measured).
        static_assert(kPrefetchAhead == 2, "the loop below looks exactly two units ahead");
        UnitPos pa, pb, pn;
        uint32_t raw[kPieces][8], cur[kPieces][8];
        decode_unit<PACKED>(a, unit, lane, pa);
        load_unit<WIDE, PACKED>(a, pa, lane, raw);
        uint32_t ahead = feed.pop(lane);
        bool has_next = ahead < a.total_units;
        if (has_next) decode_unit<PACKED>(a, ahead, lane, pn);
#pragma unroll 1
        for (;;) {
            patch_store(raw, patch, lane);
            const bool more = has_next;
            if (more) {
                pb = pn;
                load_unit<WIDE, PACKED>(a, pb, lane, raw);
            }
            ahead = feed.pop(lane);
            has_next = ahead < a.total_units;
            if (has_next) {
                decode_unit<PACKED>(a, ahead, lane, pn);
                prefetch_unit_l2<PACKED>(a, pn, lane);
            }
            patch_load(patch, lane, cur);
            compress_unit<BITS, G, WIDE>(a, pa, cur, lane, sum_slots);
            if (!more) break;
            pa = pb;
        }
    }
    __syncthreads();
    if (a.n <= kSumSlots)
        for (int k = threadIdx.x; k < a.n; k += kThreads)
            if (sum_slots[k]) atomicAdd(&a.entries[a.order[k]].checksum, sum_slots[k]);
}

// The launch arguments of a call, one set per bit-width (8, 4, 2, 1; n == 0: that width is absent).
struct CodecArgsByWidth {
    CodecArgs w[4];
    // what the CTA that finishes last does with the sums of the whole call
    uint32_t *done;                   // third word of the workspace header: CTAs that have finished (starts at 0)
    uint32_t *feed;                   // the work-split counters of the header (all zero at the start), one set per width
    const ChunkEntry *entries;        // all n_total entries of the call
    const uint32_t *sums;             // decoder: recomputed sums
    uint32_t *status;                 // decoder: first word of the header, records whose sum is wrong
    llms_chunk_meta *live_meta;       // the caller's meta array if the device can reach it (page-locked), else NULL
    int n_total;
    int expect_live;                  // decoder: 1 = the expected sums are read from live_meta now, 0 = from entries
};

__device__ __forceinline__ uint32_t *feed_counters(uint32_t *feed, int width_index)
{
    return feed + width_index * (kFeedCounters * kFeedStrideWords);
}

// True in every thread of exactly one CTA of the grid: the one that comes here last.  Each thread's earlier atomics
// on global memory are visible to that CTA's loads that bypass L1 (__ldcg).  Nobody waits for anybody.
__device__ __forceinline__ bool cta_is_last(uint32_t *done)
{
    __shared__ uint32_t ticket;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) ticket = atomicAdd(done, 1u);
    __syncthreads();
    const bool last = ticket == gridDim.x - 1;
    if (last) __threadfence();
    return last;
}

// One launch per call.  The bit-widths are phases in time, not branches per unit: every warp first works through
// its share of the 8-bit chunks, then of the 4-bit ones, and so on, so the SM runs one code path at a time (with
// the widths mixed unit by unit the warps stalled on instruction fetch), no launch boundary separates the widths
// (one launch per width cost a drained GPU and a few microseconds between each pair), and a warp that is done
// with one width starts on the next while others finish.
template <int G, bool WIDE, bool PACKED>
__global__ void __launch_bounds__(kThreads, 2) compress_kernel(const __grid_constant__ CodecArgsByWidth all)
{
    __shared__ __align__(16) unsigned char patches[kWarpsPerBlock][kTransposeBytes];
    __shared__ uint32_t sum_slots[kSumSlots];
    grid_dependency_wait();   // the chunk tables may come from a kernel that is still finishing (a no-op otherwise)
    if (all.w[0].n) compress_phase<8, G, WIDE, PACKED>(all.w[0], feed_counters(all.feed, 0), patches, sum_slots);
    if (all.w[1].n) compress_phase<4, G, WIDE, PACKED>(all.w[1], feed_counters(all.feed, 1), patches, sum_slots);
    if (all.w[2].n) compress_phase<2, G, WIDE, PACKED>(all.w[2], feed_counters(all.feed, 2), patches, sum_slots);
    if (all.w[3].n) compress_phase<1, G, WIDE, PACKED>(all.w[3], feed_counters(all.feed, 3), patches, sum_slots);
    // The finished checksums go to the caller's page-locked meta array from the CTA that ends last (a kernel of its
    // own for these few stores cost a launch boundary; a device-to-host copy would also queue on the copy engine
    // behind whatever bulk copies other streams have in flight).
    if (all.live_meta && cta_is_last(all.done))
        for (int i = threadIdx.x; i < all.n_total; i += kThreads) all.live_meta[i].checksum = __ldcg(&all.entries[i].checksum);
}

// ---------------------------------------------------------------------------------------------- dequantize

// The decoder splits a pass differently from the encoder: piece j of lane L is elements
// [j*512 + L*16, +16) of the pass, so that every store instruction of the warp writes 1 KiB of consecutive
// addresses (a lane-contiguous split made each store touch 32 separate lines and ran slower).  Groups need no
// lane cooperation here; each piece just looks its group's parameters up.  Everything a piece needs sits at a
// compile-time distance from piece 0 (512 elements, 512/G groups), so a unit's addresses are computed once.
constexpr int kPieceStride = 32 * kPieceElems;  // elements between a lane's pieces

struct DecodePos {
    uint32_t i, k;           // entry index (checksum slot); position in this launch's list
    int room;                // elements from this lane's piece 0 to the end of the unit's data (<= 0: none)
    const uint8_t *codes;    // piece 0: packed codes
    const uint32_t *params;  // piece 0: parameter word of its group
    uint32_t s_idx, chunk_id;  // destination: first slab of the unit, chunk slot
    int pass_e0;             // first element of the unit inside slab s_idx (0 when packed)
};

template <int BITS, int G, bool PACKED>
__device__ __forceinline__ void decode_unit_for_decoder(const CodecArgs &a, uint32_t unit, int lane, DecodePos &u)
{
    static_assert(kPieceStride % G == 0 || G % kPieceStride == 0, "groups and pieces nest");
    uint32_t item, pass, row, k;
    a.div_passes.divmod(unit, item, pass);
    a.div_n.divmod(item, row, k);
    const uint4 t = *reinterpret_cast<const uint4 *>(a.table + k);  // chunk_id, entry, record offset
    u.i = t.y;
    u.k = k;
    u.chunk_id = t.x;
    int limit;
    if constexpr (PACKED) {
        u.s_idx = row * (uint32_t)a.slabs_per_unit;
        u.pass_e0 = 0;
        limit = (int)min((uint32_t)kPassElems, a.chunk_elems - row * kPassElems);
    } else {
        u.s_idx = row;
        u.pass_e0 = (int)pass * kPassElems;
        limit = a.slab_elems - u.pass_e0;
    }
    u.room = limit - lane * kPieceElems;
    const uint32_t e = (uint32_t)u.pass_e0 + lane * kPieceElems;    // piece 0, counted from the start of slab s_idx
    const uint8_t *rec = a.buf + ((uint64_t)t.z | ((uint64_t)t.w << 32));
    u.params = reinterpret_cast<const uint32_t *>(rec) + (u.s_idx * (uint32_t)a.groups_per_slab + e / G);
    u.codes = rec + a.codes_off + ((uint64_t)u.s_idx * a.slab_elems + e) * BITS / 8;
}

template <int BITS, int G>
__device__ __forceinline__ void load_unit_codes(const DecodePos &u, uint32_t (&c)[kPieces][piece_words(BITS)], uint32_t (&p)[kPieces])
{
    constexpr int kStrideBytes = kPieceStride * BITS / 8;
#pragma unroll
    for (int j = 0; j < kPieces; ++j) {
        if (u.room > j * kPieceStride) {
            const uint8_t *src = u.codes + j * kStrideBytes;
            if constexpr (BITS == 8) ld128(src, c[j]);
            else if constexpr (BITS == 4) ld64(src, c[j]);
            else if constexpr (BITS == 2) ld32(src, c[j]);
            else ld16(src, c[j]);
            p[j] = access_ok(u.params + j * (kPieceStride / G), 4) ? __ldg(u.params + j * (kPieceStride / G)) : 0u;
        } else {
#pragma unroll
            for (int k = 0; k < piece_words(BITS); ++k) c[j][k] = 0;
            p[j] = 0;
        }
    }
}

// 16 codes -> 8 half2 holding the codes as exact fp16 integers.  0x6400 | q is the fp16 number 1024 + q, so a
// code only has to be moved to the low bits of a 16-bit half.  At 8 bits one byte permute places two codes; at 4
// and 2 bits one shift and one and-or place the two codes that sit 16 bits apart.  which[e] tells where code e
// ended up: half2 index * 2 + (0 low half, 1 high half).
template <int BITS>
__device__ __forceinline__ void codes_to_half2(const uint32_t *c, __half2 (&q)[8])
{
    const __half2 k1024 = as_h2(0x64006400u);
    if constexpr (BITS == 8) {
#pragma unroll
        for (int m = 0; m < 4; ++m) {
            q[2 * m] = __hsub2(as_h2(__byte_perm(c[m], 0x64646464u, 0x4140)), k1024);      // codes 4m, 4m+1
            q[2 * m + 1] = __hsub2(as_h2(__byte_perm(c[m], 0x64646464u, 0x4342)), k1024);  // codes 4m+2, 4m+3
        }
    } else if constexpr (BITS == 4) {
#pragma unroll
        for (int m = 0; m < 2; ++m)
#pragma unroll
            for (int s = 0; s < 4; ++s)  // codes 8m + s (low half) and 8m + s + 4 (high half)
                q[4 * m + s] = __hsub2(as_h2(((c[m] >> (4 * s)) & 0x000F000Fu) | 0x64006400u), k1024);
    } else if constexpr (BITS == 2) {
#pragma unroll
        for (int s = 0; s < 8; ++s)      // codes s (low half) and s + 8 (high half)
            q[s] = __hsub2(as_h2(((c[0] >> (2 * s)) & 0x00030003u) | 0x64006400u), k1024);
    } else {
        const uint32_t z = (c[0] & 0xFFu) | ((c[0] & 0xFF00u) << 8);  // codes 0..7 in the low half, 8..15 in the high half
#pragma unroll
        for (int s = 0; s < 8; ++s)      // codes s (low half) and s + 8 (high half)
            q[s] = __hsub2(as_h2(((z >> s) & 0x00010001u) | 0x64006400u), k1024);
    }
}

// the fp16 bit pattern of code e (0..15) inside q[] as laid out above
template <int BITS>
__device__ __forceinline__ unsigned short code_half(const __half2 (&q)[8], int e)
{
    int idx, hi;
    if constexpr (BITS == 8) { idx = e / 2; hi = e % 2; }
    else if constexpr (BITS == 4) { idx = 4 * (e / 8) + e % 4; hi = (e % 8) / 4; }
    else { idx = e % 8; hi = e / 8; }
    unsigned short lo_h, hi_h;
    split_halves(as_u32(q[idx]), lo_h, hi_h);
    return hi ? hi_h : lo_h;
}

// Two binary32 values -> packed fp16, round to nearest even, magnitudes above 65504 become +-65504: the clamp
// and the conversion of the decode rule in one instruction.
__device__ __forceinline__ uint32_t pack_half2_clamped(float lo, float hi)
{
    uint32_t w;
    asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(hi), "f"(lo));
    return w;
}

// 16 decoded values.  q*scale is exact in binary32, so the mixed-precision fused form rounds once, as
// multiply-then-add would.
template <int BITS>
__device__ __forceinline__ void dequantize_piece(const uint32_t *c, unsigned short scale_h, float zero, uint32_t (&w)[8])
{
    __half2 q[8];
    codes_to_half2<BITS>(c, q);
#pragma unroll
    for (int k = 0; k < 8; ++k)
        w[k] = pack_half2_clamped(fma_f32_f16(code_half<BITS>(q, 2 * k), scale_h, zero),
                                  fma_f32_f16(code_half<BITS>(q, 2 * k + 1), scale_h, zero));
}

template <int BITS, int G, bool WIDE, bool PACKED>
__device__ __forceinline__ void decompress_unit(const CodecArgs &a, const DecodePos &u, const uint32_t (&c)[kPieces][piece_words(BITS)],
                                                const uint32_t (&p)[kPieces], int lane, uint32_t *sum_slots)
{
    // a lane's pieces all sit at the same place inside their groups: either every one opens a group or none does
    const bool opens_group = (lane * kPieceElems) % G == 0;
    __half *dst0 = nullptr;  // piece 0 when the unit lies inside one slab
    if constexpr (!PACKED) dst0 = a.kv_out + slab_offset(a, u.s_idx, u.chunk_id) + u.pass_e0 + lane * kPieceElems;
    uint32_t sum = 0;
#pragma unroll
    for (int j = 0; j < kPieces; ++j) {
        const unsigned short scale_h = (unsigned short)(p[j] & 0xffffu);
        const float zero = __half2float(__ushort_as_half((unsigned short)(p[j] >> 16)));
        uint32_t w[8];
        dequantize_piece<BITS>(c[j], scale_h, zero, w);
        if (u.room > j * kPieceStride) {
            if constexpr (PACKED)
                store32<WIDE>(a.kv_out + unit_elem_offset<true>(a, u.s_idx, u.chunk_id, 0, j * kPieceStride + lane * kPieceElems), w);
            else
                store32<WIDE>(dst0 + j * kPieceStride, w);
        }
        // pieces past the end of the slab were loaded as zeros and add nothing
        if constexpr (BITS == 1) {  // a piece is half of a record word; the pieces of a lane all sit in the same half
            sum += c[j][0] << ((reinterpret_cast<uintptr_t>(u.codes) & 2) * 8);
        } else {
#pragma unroll
            for (int k = 0; k < piece_words(BITS); ++k) sum += c[j][k];
        }
        if (opens_group) sum += p[j];  // the piece that opens a group accounts for its parameter word
    }
    unit_sum_add(sum_slots, a.n, u.k, &a.sums[u.i], sum, lane);
}

// Units whose loads are in flight per warp, the one being decoded included, and resident CTAs per SM.  Measured
// on the 7B shape (decompress call, ms; depth x CTAs): 2x2 0.448, 2x3 0.446, 3x2 0.448, 2x4 0.477, 4x1 0.495 (with
// the fixed work split that preceded the drawn one: 2x2 0.481): the store-heavy stream runs best with 16 to 24 warps
// per SM.
constexpr int kDecodeDepth = 2;
constexpr int kDecodeBlocksPerSm = 2;

// The units of one warp, start to finish.
template <int BITS, int G, bool WIDE, bool PACKED>
__device__ __forceinline__ void decompress_warp(const CodecArgs &a, UnitFeed &feed, int lane, uint32_t *sum_slots)
{
    constexpr int D = kDecodeDepth;
    static_assert(D >= 2, "the ring refills the slot freed one turn ago");
    DecodePos pos[D];
    uint32_t id[D];
    uint32_t c[D][kPieces][piece_words(BITS)], p[D][kPieces];
#pragma unroll
    for (int s = 0; s < D - 1; ++s) {
        id[s] = feed.pop(lane);
        if (id[s] < a.total_units) {
            decode_unit_for_decoder<BITS, G, PACKED>(a, id[s], lane, pos[s]);
            load_unit_codes<BITS, G>(pos[s], c[s], p[s]);
        }
    }
    if (id[0] >= a.total_units) return;
    for (;;) {
#pragma unroll
        for (int s = 0; s < D; ++s) {
            // ring slot s holds the current unit; the slot freed last takes the unit D-1 turns ahead
            const int fill = (s + D - 1) % D;
            id[fill] = feed.pop(lane);
            if (id[fill] < a.total_units) {
                decode_unit_for_decoder<BITS, G, PACKED>(a, id[fill], lane, pos[fill]);
                load_unit_codes<BITS, G>(pos[fill], c[fill], p[fill]);
            }
            decompress_unit<BITS, G, WIDE, PACKED>(a, pos[s], c[s], p[s], lane, sum_slots);
            if (id[(s + 1) % D] >= a.total_units) return;
        }
    }
}

template <int BITS, int G, bool WIDE, bool PACKED>
__device__ __forceinline__ void decompress_phase(const CodecArgs &a, uint32_t *counters, uint32_t *sum_slots)
{
    const int lane = threadIdx.x & 31;
    UnitFeed feed;
    feed.start(counters, a.total_units, lane);
    cta_sums_clear(sum_slots, a.n);
    decompress_warp<BITS, G, WIDE, PACKED>(a, feed, lane, sum_slots);
    __syncthreads();
    if (a.n <= kSumSlots)
        for (int k = threadIdx.x; k < a.n; k += kThreads)
            if (sum_slots[k]) atomicAdd(&a.sums[a.table[k].entry], sum_slots[k]);
}

// One launch per call, the bit-widths as phases in time (see compress_kernel).
template <int G, bool WIDE, bool PACKED>
__global__ void __launch_bounds__(kThreads, kDecodeBlocksPerSm) decompress_kernel(const __grid_constant__ CodecArgsByWidth all)
{
    __shared__ uint32_t sum_slots[kSumSlots];
    if (all.w[0].n) decompress_phase<8, G, WIDE, PACKED>(all.w[0], feed_counters(all.feed, 0), sum_slots);
    if (all.w[1].n) decompress_phase<4, G, WIDE, PACKED>(all.w[1], feed_counters(all.feed, 1), sum_slots);
    if (all.w[2].n) decompress_phase<2, G, WIDE, PACKED>(all.w[2], feed_counters(all.feed, 2), sum_slots);
    if (all.w[3].n) decompress_phase<1, G, WIDE, PACKED>(all.w[3], feed_counters(all.feed, 3), sum_slots);
    // the CTA that ends last compares every record's recomputed sum with the expected one
    if (cta_is_last(all.done)) {
        uint32_t bad = 0;
        for (int i = threadIdx.x; i < all.n_total; i += kThreads) {
            const uint32_t want = all.expect_live ? *reinterpret_cast<const volatile uint32_t *>(&all.live_meta[i].checksum)
                                                  : __ldcg(&all.entries[i].checksum);
            bad += __ldcg(&all.sums[i]) != want;
        }
        bad = __reduce_add_sync(0xffffffffu, bad);
        if ((threadIdx.x & 31) == 0 && bad) atomicAdd(all.status, bad);
    }
}

}  // namespace llms

#include "codec_cw.cuh"

namespace llms {

// status word = number of records whose recomputed sum differs from the expected one.  live_meta: the caller's
// meta array when it lies in page-locked host memory the device can read (the expected sums are then taken now, in
// stream order, not when the call was made); else NULL and the copies uploaded with the call are used.
__global__ void verify_kernel(const ChunkEntry *entries, const uint32_t *sums, int n, uint32_t *status,
                              const llms_chunk_meta *live_meta)
{
    uint32_t bad = 0;
    for (int i = threadIdx.x; i < n; i += blockDim.x)
        bad += (sums[i] != (live_meta ? *reinterpret_cast<const volatile uint32_t *>(&live_meta[i].checksum) : entries[i].checksum));
    bad = __reduce_add_sync(0xffffffffu, bad);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(status, bad);
}

// The finished checksums, stored by the device into the caller's page-locked meta array.  A device-to-host copy
// would do the same, but it queues on the copy engine behind whatever bulk copies other streams have in flight
// (measured in the multi-app driver: the encoder's stream then advances at the pace of the swap-out copies).
__global__ void publish_checksums_kernel(const ChunkEntry *entries, llms_chunk_meta *live_meta, int n)
{
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
        live_meta[i].checksum = entries[i].checksum;
}

// ---------------------------------------------------------------------------------------------- host side

static int fill_args(const llms_kv_desc &d, CodecArgs &a, int n, void *workspace, bool wide)
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
    a.chunk_elems = (uint32_t)a.n_slabs * (uint32_t)a.slab_elems;
    // slabs shorter than a pass: whole slabs are packed into a unit (only with 256-bit accesses; the channel-wise
    // kernels keep their own walk over slabs)
    a.packed = wide && d.quant_mode == 0 && a.slab_elems < kPassElems && kPassElems % a.slab_elems == 0 &&
               a.slab_elems % kLaneElems == 0;
    if (a.packed) {
        a.passes = 1;
        a.slabs_per_unit = kPassElems / a.slab_elems;
        a.slab_shift = 0;
        while ((1 << a.slab_shift) < a.slab_elems) ++a.slab_shift;
        a.unit_rows = (int)((a.chunk_elems + kPassElems - 1) / kPassElems);
    } else {
        a.passes = (a.slab_elems + kPassElems - 1) / kPassElems;
        a.unit_rows = a.n_slabs;
    }
    a.total_units = (uint32_t)n * (uint32_t)a.unit_rows * (uint32_t)a.passes;
    a.div_passes.set((uint32_t)a.passes);
    a.div_n.set((uint32_t)n);
    a.div_heads.set((uint32_t)a.n_kv_heads);
    a.entries = reinterpret_cast<ChunkEntry *>(static_cast<uint8_t *>(workspace) + kWsEntriesOffset);
    a.sums = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + ws_sums_offset(n));
    a.order = reinterpret_cast<const uint32_t *>(static_cast<uint8_t *>(workspace) + ws_order_offset(n));
    a.table = reinterpret_cast<const UnitEntry *>(static_cast<uint8_t *>(workspace) + ws_table_offset(n));
    a.feed = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + kWsFeedOffset);
    return LLMS_OK;
}

// Entry indices grouped by bit-width (8, then 4, then 2), list order kept inside a group.
constexpr int kNumWidths = 4;
struct BitGroups {
    std::vector<uint32_t> order;
    std::vector<UnitEntry> table;
    int first[kNumWidths], count[kNumWidths];
};

template <typename GetBits>
static BitGroups group_by_bits(int n, const llms_chunk_meta *meta, GetBits bits_of)
{
    static const uint32_t kWidths[kNumWidths] = {8, 4, 2, 1};
    BitGroups g;
    g.order.reserve(n);
    for (int k = 0; k < kNumWidths; ++k) {
        g.first[k] = (int)g.order.size();
        for (int i = 0; i < n; ++i)
            if (bits_of(i) == kWidths[k]) g.order.push_back((uint32_t)i);
        g.count[k] = (int)g.order.size() - g.first[k];
    }
    g.table.resize(n);
    for (int j = 0; j < n; ++j) {
        const llms_chunk_meta &m = meta[g.order[j]];
        g.table[j].chunk_id = m.chunk_id;
        g.table[j].entry = g.order[j];
        g.table[j].rec_off = m.offset;
    }
    return g;
}

// One host-to-device copy sets the workspace up: zeroed status words, the entries, the unit table, the order and,
// for the decoder, the zeroed checksum accumulators behind them.
static int upload_tables(void *workspace, const llms_chunk_meta *entries, const BitGroups &g, int n, bool zero_sums,
                         cudaStream_t st)
{
    std::vector<uint8_t> image(ws_sums_offset(n) + (zero_sums ? (size_t)n * 4 : 0), 0);
    memcpy(image.data() + kWsEntriesOffset, entries, (size_t)n * sizeof(ChunkEntry));
    memcpy(image.data() + ws_table_offset(n), g.table.data(), (size_t)n * sizeof(UnitEntry));
    memcpy(image.data() + ws_order_offset(n), g.order.data(), (size_t)n * 4);
    // `image` is pageable: the copy has left it by the time cudaMemcpyAsync returns
    LLMS_CUDA_TRY(cudaMemcpyAsync(workspace, image.data(), image.size(), cudaMemcpyHostToDevice, st));
    return LLMS_OK;
}

// The launch arguments of one bit-width's share of the call.
static CodecArgs args_for_group(const CodecArgs &a, const BitGroups &g, int k)
{
    CodecArgs b = a;
    b.order = a.order + g.first[k];
    b.table = a.table + g.first[k];
    b.n = g.count[k];
    b.feed = a.feed + k * (kFeedCounters * kFeedStrideWords);
    b.total_units = (uint32_t)b.n * (uint32_t)b.unit_rows * (uint32_t)b.passes;
    b.div_n.set((uint32_t)b.n);
    return b;
}

// Persistent grid: as many CTAs as are resident at once, or fewer when there is less work.
template <typename K>
static int grid_for(K kernel, int64_t items, size_t dyn_smem = 0)
{
    // the occupancy of a kernel does not change: asked once per kernel and device
    static std::mutex lock;
    static std::map<std::pair<const void *, int>, int> known;
    int dev = 0;
    cudaGetDevice(&dev);
    const std::pair<const void *, int> key(reinterpret_cast<const void *>(kernel), dev);
    int per_sm = 0;
    {
        std::lock_guard<std::mutex> guard(lock);
        auto it = known.find(key);
        if (it != known.end()) per_sm = it->second;
    }
    if (per_sm == 0) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, dyn_smem) != cudaSuccess || per_sm <= 0) {
            cudaGetLastError();
            per_sm = 2;
        }
        std::lock_guard<std::mutex> guard(lock);
        known[key] = per_sm;
    }
    const int64_t want = (items + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const int64_t cap = (int64_t)sm_count() * per_sm;
    return (int)(want < cap ? want : cap);
}

// Channel-wise launches: slabs of 4, 8 or 16 tokens per lane (the paper's 16-token chunks at head_dim 64, 128, 256)
// take the kernels that hold the slab in registers, anything else the two-pass ones.
template <int BITS>
static void launch_compress_cw(const CodecArgs &b, int head_dim, int chunk_len, cudaStream_t st)
{
    const int64_t items = (int64_t)b.n * b.n_slabs;
    const int lpc = 32 / (head_dim / 8);
    const int tok = chunk_len % lpc == 0 ? chunk_len / lpc : 0;
    if (tok == 4) compress_cw_reg_kernel<BITS, 4><<<grid_for(compress_cw_reg_kernel<BITS, 4>, items), kThreads, 0, st>>>(b, head_dim);
    else if (tok == 8) compress_cw_reg_kernel<BITS, 8><<<grid_for(compress_cw_reg_kernel<BITS, 8>, items), kThreads, 0, st>>>(b, head_dim);
    else if (tok == 16) compress_cw_reg_kernel<BITS, 16><<<grid_for(compress_cw_reg_kernel<BITS, 16>, items), kThreads, 0, st>>>(b, head_dim);
    else compress_cw_kernel<BITS><<<grid_for(compress_cw_kernel<BITS>, items), kThreads, 0, st>>>(b, head_dim, chunk_len);
}

template <int BITS>
static void launch_decompress_cw(const CodecArgs &b, int head_dim, int chunk_len, cudaStream_t st)
{
    const int64_t items = (int64_t)b.n * b.n_slabs;
    const int lpc = 32 / (head_dim / 8);
    const int tok = chunk_len % lpc == 0 ? chunk_len / lpc : 0;
    if (tok == 4) decompress_cw_reg_kernel<BITS, 4><<<grid_for(decompress_cw_reg_kernel<BITS, 4>, items), kThreads, 0, st>>>(b, head_dim);
    else if (tok == 8) decompress_cw_reg_kernel<BITS, 8><<<grid_for(decompress_cw_reg_kernel<BITS, 8>, items), kThreads, 0, st>>>(b, head_dim);
    else if (tok == 16) decompress_cw_reg_kernel<BITS, 16><<<grid_for(decompress_cw_reg_kernel<BITS, 16>, items), kThreads, 0, st>>>(b, head_dim);
    else decompress_cw_kernel<BITS><<<grid_for(decompress_cw_kernel<BITS>, items), kThreads, 0, st>>>(b, head_dim, chunk_len);
}

// The decoder's grid: never more CTAs per SM than it was tuned for, whatever the register count allows.
template <typename K>
static int decode_grid(K kernel, int64_t items)
{
    const int cap = sm_count() * kDecodeBlocksPerSm;
    const int grid = grid_for(kernel, items);
    return grid < cap ? grid : cap;
}


// 256-bit accesses need every slab to start on a 32-byte boundary
static bool wide_ok(const llms_kv_desc &d, const void *kv)
{
    return aligned(kv, 32) && ((d.stride_l | d.stride_s | d.stride_h) % 16) == 0;
}

template <typename F>
static int dispatch_group(int group_size, F &&f)
{
    switch (group_size) {
    case 16: f(std::integral_constant<int, 16>()); break;
    case 32: f(std::integral_constant<int, 32>()); break;
    case 64: f(std::integral_constant<int, 64>()); break;
    case 128: f(std::integral_constant<int, 128>()); break;
    case 256: f(std::integral_constant<int, 256>()); break;
    case 512: f(std::integral_constant<int, 512>()); break;
    default: return LLMS_ERR_UNSUPPORTED;
    }
    return LLMS_OK;
}

static int check_common(const llms_kv_desc *desc, int n, const void *workspace, uint64_t workspace_bytes)
{
    int rc = check_desc_codec(desc);
    if (rc) return rc;
    if (desc->quant_mode == 1 && desc->head_dim != 64 && desc->head_dim != 128 && desc->head_dim != 256) return LLMS_ERR_UNSUPPORTED;
    if (n < 0) return LLMS_ERR_INVALID_ARG;
    if (n == 0) return LLMS_OK;
    if (!workspace) return LLMS_ERR_INVALID_ARG;
    if (!aligned(workspace, 16)) return LLMS_ERR_MISALIGNED;
    if (workspace_bytes < ws_total(n)) return LLMS_ERR_BUF_TOO_SMALL;
    if (groups_per_chunk(*desc) * 4 > 0xffffffffull) return LLMS_ERR_UNSUPPORTED;
    if (slab_elems(*desc) > 0x7fffffff / 8) return LLMS_ERR_UNSUPPORTED;
    const uint64_t passes = ((uint64_t)slab_elems(*desc) + kPassElems - 1) / kPassElems;
    if ((uint64_t)n * (uint64_t)slabs_per_chunk(*desc) * passes > 0x7fffffffull) return LLMS_ERR_UNSUPPORTED;
    return LLMS_OK;
}

#ifdef LLMS_DEBUG_BOUNDS
// For the test of the check itself: the swap buffer's range is declared this much shorter than it is, so that accesses to
// its (perfectly valid) last bytes are counted and skipped.
static uint64_t g_debug_shrink_bytes = 0;
extern "C" void llms_debug_shrink_swap_range(uint64_t bytes) { g_debug_shrink_bytes = bytes; }
#endif

// The checked build's two address ranges for the kernels of a call: the KV tensor as the strides span it, and the swap
// buffer.  The ordinary build does nothing here.
static int set_debug_ranges(const llms_kv_desc &d, const void *kv, const void *buf, uint64_t buf_bytes, cudaStream_t st)
{
#ifdef LLMS_DEBUG_BOUNDS
    const uint64_t span = (uint64_t)(d.n_layers - 1) * d.stride_l + (uint64_t)d.stride_s + (uint64_t)(d.n_kv_heads - 1) * d.stride_h +
                          (uint64_t)d.n_tokens * d.head_dim;   // elements up to the end of the last slab
    DebugRanges r;
    r.lo[0] = reinterpret_cast<unsigned long long>(kv);
    r.hi[0] = r.lo[0] + span * 2;
    r.lo[1] = reinterpret_cast<unsigned long long>(buf);
    r.hi[1] = r.lo[1] + buf_bytes - std::min<uint64_t>(buf_bytes, g_debug_shrink_bytes);
    LLMS_CUDA_TRY(cudaMemcpyToSymbolAsync(g_debug_ranges, &r, sizeof(r), 0, cudaMemcpyHostToDevice, st));
#else
    (void)d; (void)kv; (void)buf; (void)buf_bytes; (void)st;
#endif
    return LLMS_OK;
}

// Launch the encoder over the chunk tables that sit in the workspace (entries, unit table, order grouped by bit-width;
// first[k] / count[k]: where the chunks of width 8, 4, 2, 1 start in the grouped order and how many there are), and see
// to it that the checksums reach `meta` (host) in stream order.
static int launch_compress(const llms_kv_desc &desc, const void *kv, void *out_buf, uint64_t out_bytes, void *workspace, int n,
                           const int (&first)[kNumWidths], const int (&count)[kNumWidths], llms_chunk_meta *meta, cudaStream_t st,
                           bool after_kernel = false)
{
    if (int rc = set_debug_ranges(desc, kv, out_buf, out_bytes, st)) return rc;
    CodecArgs a{};
    const bool wide = wide_ok(desc, kv);
    fill_args(desc, a, n, workspace, wide);
    a.kv_in = static_cast<const __half *>(kv);
    a.buf = static_cast<uint8_t *>(out_buf);
    BitGroups groups;
    for (int k = 0; k < kNumWidths; ++k) {
        groups.first[k] = first[k];
        groups.count[k] = count[k];
    }
    int rc = LLMS_OK;
    cudaError_t launch_err = cudaSuccess;
    bool published = false;  // the codec kernel itself stores the checksums into a page-locked meta array
    if (desc.quant_mode == 1) {
        for (int k = 0; k < kNumWidths; ++k) {
            if (groups.count[k] == 0) continue;
            const CodecArgs b = args_for_group(a, groups, k);
            if (k == 0) launch_compress_cw<8>(b, desc.head_dim, desc.chunk_len, st);
            else if (k == 1) launch_compress_cw<4>(b, desc.head_dim, desc.chunk_len, st);
            else if (k == 2) launch_compress_cw<2>(b, desc.head_dim, desc.chunk_len, st);
            else launch_compress_cw<1>(b, desc.head_dim, desc.chunk_len, st);
            LLMS_CUDA_TRY(cudaGetLastError());
        }
    } else {
        // one launch for the whole call; the grid is sized for the width with the most units
        CodecArgsByWidth all{};
        uint32_t most_units = 0;
        for (int k = 0; k < kNumWidths; ++k) {
            if (groups.count[k] == 0) continue;
            all.w[k] = args_for_group(a, groups, k);
            most_units = std::max(most_units, all.w[k].total_units);
        }
        all.done = static_cast<uint32_t *>(workspace) + 2;
        all.feed = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + kWsFeedOffset);
        all.entries = a.entries;
        all.n_total = n;
        all.live_meta = static_cast<llms_chunk_meta *>(device_view_of_pinned(meta));
        published = all.live_meta != nullptr;
        rc = dispatch_group(desc.group_size, [&](auto g) {
            constexpr int kG = decltype(g)::value;
            // after_kernel: the tables come from a kernel just ahead on the stream; this one may be set up while that one ends
            auto go = [&](auto kernel) {
                const int grid = grid_for(kernel, most_units);
                if (after_kernel) launch_err = launch_dependent(kernel, dim3(grid), dim3(kThreads), 0, st, all);
                else kernel<<<grid, kThreads, 0, st>>>(all);
            };
            if (a.packed) go(compress_kernel<kG, true, true>);
            else if (wide) go(compress_kernel<kG, true, false>);
            else go(compress_kernel<kG, false, false>);
        });
        if (rc) return rc;
        LLMS_CUDA_TRY(launch_err);
        LLMS_CUDA_TRY(cudaGetLastError());
    }
    // checksums back to the caller's meta (every other field is already there)
    if (published) {
        // nothing left to do
    } else if (void *live = device_view_of_pinned(meta)) {
        publish_checksums_kernel<<<(n + 255) / 256, 256, 0, st>>>(a.entries, static_cast<llms_chunk_meta *>(live), n);
        LLMS_CUDA_TRY(cudaGetLastError());
    } else {
        LLMS_CUDA_TRY(cudaMemcpyAsync(meta, a.entries, (size_t)n * sizeof(ChunkEntry), cudaMemcpyDeviceToHost, st));
    }
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
    uint64_t bytes_at[9] = {0};  // record size per bit-width, looked up once each
    uint64_t off = 0;
    for (int i = 0; i < n; ++i) {
        const uint8_t b = bits[i];
        if (b > 8) return LLMS_ERR_BAD_BITS;
        if (bytes_at[b] == 0) {
            rc = llms_record_bytes(desc, b, &bytes_at[b]);
            if (rc) return rc;
        }
        if (chunk_ids[i] >= nc || seen[chunk_ids[i]]) return LLMS_ERR_INVALID_ARG;
        seen[chunk_ids[i]] = 1;
        off += bytes_at[b];
    }
    if (off > out_bytes) return LLMS_ERR_BUF_TOO_SMALL;
    const uint32_t n_groups = (uint32_t)groups_per_chunk(*desc);
    // The device's table is built from a private copy: `meta` may be page-locked memory into which an earlier
    // call's kernel is still storing checksums, and the accumulators uploaded below have to start at zero.
    std::vector<llms_chunk_meta> staged(n);
    off = 0;
    for (int i = 0; i < n; ++i) {
        staged[i].chunk_id = chunk_ids[i];
        staged[i].bits = bits[i];
        staged[i].offset = off;
        staged[i].nbytes = bytes_at[bits[i]];
        staged[i].n_groups = n_groups;
        staged[i].checksum = 0;  // the kernel accumulates into the device copy
        meta[i] = staged[i];
        off += bytes_at[bits[i]];
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const BitGroups groups = group_by_bits(n, staged.data(), [&](int i) { return (uint32_t)bits[i]; });
    rc = upload_tables(workspace, staged.data(), groups, n, false, st);
    if (rc) return rc;
    return launch_compress(*desc, kv, out_buf, out_bytes, workspace, n, groups.first, groups.count, meta, st);
}

// The encoder over chunk tables that a kernel has already put into the workspace (llms_compress_context's stream-ordered
// path): chunks 0 .. n-1 in index order, count[k] of them at width 8, 4, 2, 1.
int llms::compress_planned(const llms_kv_desc *desc, const void *kv, int n, const int count[4], void *out_buf, uint64_t out_bytes,
                           llms_chunk_meta *meta, void *workspace, void *stream)
{
    int first[kNumWidths], cnt[kNumWidths], at = 0;
    for (int k = 0; k < kNumWidths; ++k) {
        first[k] = at;
        cnt[k] = count[k];
        at += count[k];
    }
    if (at != n) return LLMS_ERR_INVALID_ARG;
    return launch_compress(*desc, kv, out_buf, out_bytes, workspace, n, first, cnt, meta, static_cast<cudaStream_t>(stream), true);
}

int llms::check_compress_args(const llms_kv_desc *desc, int n, const void *kv, const void *out_buf, const void *workspace,
                              uint64_t workspace_bytes)
{
    int rc = check_common(desc, n, workspace, workspace_bytes);
    if (rc) return rc;
    if (n > 0 && (!kv || !out_buf)) return LLMS_ERR_INVALID_ARG;
    if (!aligned(kv, 16) || !aligned(out_buf, 256)) return LLMS_ERR_MISALIGNED;
    return LLMS_OK;
}

// live_checksums: the expected sums are read from the caller's pinned meta array by the device, in stream order
static int decompress_chunks(const llms_kv_desc *desc, const void *buf, uint64_t buf_bytes, const llms_chunk_meta *meta,
                             const uint32_t *dst_chunk_ids, int n, void *kv_out, void *workspace,
                             uint64_t workspace_bytes, void *stream, bool live_checksums)
{
    int rc = check_common(desc, n, workspace, workspace_bytes);
    if (rc) return rc;
    if (n == 0) return LLMS_OK;
    if (!buf || !meta || !kv_out) return LLMS_ERR_INVALID_ARG;
    if (!aligned(kv_out, 16) || !aligned(buf, 256)) return LLMS_ERR_MISALIGNED;
    const llms_chunk_meta *live_meta = nullptr;
    if (live_checksums) {  // only page-locked host memory is visible to the device
        live_meta = static_cast<const llms_chunk_meta *>(device_view_of_pinned(meta));
        if (!live_meta) return LLMS_ERR_INVALID_ARG;
    }
    const uint32_t nc = (uint32_t)n_chunks(*desc);
    std::vector<uint8_t> seen(nc, 0);
    std::vector<llms_chunk_meta> staged(meta, meta + n);
    uint64_t bytes_at[9] = {0};  // record size per bit-width, looked up once each
    const uint32_t n_groups = (uint32_t)groups_per_chunk(*desc);
    for (int i = 0; i < n; ++i) {
        const uint32_t b = meta[i].bits;
        if (b > 8) return LLMS_ERR_BAD_BITS;
        if (bytes_at[b] == 0) {
            rc = llms_record_bytes(desc, (int)b, &bytes_at[b]);
            if (rc) return rc;
        }
        if (meta[i].nbytes != bytes_at[b] || meta[i].n_groups != n_groups) return LLMS_ERR_INVALID_ARG;
        if (meta[i].offset % 256) return LLMS_ERR_MISALIGNED;
        // the record lies inside the buffer (nothing here can wrap around: nbytes is the size just checked)
        if (meta[i].nbytes > buf_bytes || meta[i].offset > buf_bytes - meta[i].nbytes) return LLMS_ERR_BUF_TOO_SMALL;
        const uint32_t dst = dst_chunk_ids ? dst_chunk_ids[i] : meta[i].chunk_id;
        if (dst >= nc || seen[dst]) return LLMS_ERR_INVALID_ARG;
        seen[dst] = 1;
        staged[i].chunk_id = dst;
    }
    rc = set_debug_ranges(*desc, kv_out, buf, buf_bytes, static_cast<cudaStream_t>(stream));
    if (rc) return rc;
    CodecArgs a{};
    const bool wide = wide_ok(*desc, kv_out);
    fill_args(*desc, a, n, workspace, wide);
    a.kv_out = static_cast<__half *>(kv_out);
    a.buf = const_cast<uint8_t *>(static_cast<const uint8_t *>(buf));
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t *status = static_cast<uint32_t *>(workspace);
    const BitGroups groups = group_by_bits(n, staged.data(), [&](int i) { return meta[i].bits; });
    rc = upload_tables(workspace, staged.data(), groups, n, true, st);
    if (rc) return rc;
    bool verified = false;  // the codec kernel itself checks the sums
    if (desc->quant_mode == 1) {
        for (int k = 0; k < kNumWidths; ++k) {
            if (groups.count[k] == 0) continue;
            const CodecArgs b = args_for_group(a, groups, k);
            if (k == 0) launch_decompress_cw<8>(b, desc->head_dim, desc->chunk_len, st);
            else if (k == 1) launch_decompress_cw<4>(b, desc->head_dim, desc->chunk_len, st);
            else if (k == 2) launch_decompress_cw<2>(b, desc->head_dim, desc->chunk_len, st);
            else launch_decompress_cw<1>(b, desc->head_dim, desc->chunk_len, st);
            LLMS_CUDA_TRY(cudaGetLastError());
        }
    } else {
        CodecArgsByWidth all{};
        uint32_t most_units = 0;
        for (int k = 0; k < kNumWidths; ++k) {
            if (groups.count[k] == 0) continue;
            all.w[k] = args_for_group(a, groups, k);
            most_units = std::max(most_units, all.w[k].total_units);
        }
        all.done = static_cast<uint32_t *>(workspace) + 2;
        all.feed = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(workspace) + kWsFeedOffset);
        all.entries = a.entries;
        all.sums = a.sums;
        all.status = status;
        all.n_total = n;
        all.live_meta = const_cast<llms_chunk_meta *>(live_meta);
        all.expect_live = live_meta != nullptr;
        verified = true;
        rc = dispatch_group(desc->group_size, [&](auto g) {
            constexpr int kG = decltype(g)::value;
            if (a.packed) decompress_kernel<kG, true, true><<<decode_grid(decompress_kernel<kG, true, true>, most_units), kThreads, 0, st>>>(all);
            else if (wide) decompress_kernel<kG, true, false><<<decode_grid(decompress_kernel<kG, true, false>, most_units), kThreads, 0, st>>>(all);
            else decompress_kernel<kG, false, false><<<decode_grid(decompress_kernel<kG, false, false>, most_units), kThreads, 0, st>>>(all);
        });
        if (rc) return rc;
        LLMS_CUDA_TRY(cudaGetLastError());
    }
    if (!verified) {  // channel-wise launches: the check is a kernel of its own
        verify_kernel<<<1, 256, 0, st>>>(a.entries, a.sums, n, status, live_meta);
        LLMS_CUDA_TRY(cudaGetLastError());
    }
    return LLMS_OK;
}

extern "C" int llms_decompress_chunks(const llms_kv_desc *desc, const void *buf, uint64_t buf_bytes,
                                      const llms_chunk_meta *meta, const uint32_t *dst_chunk_ids, int n, void *kv_out,
                                      void *workspace, uint64_t workspace_bytes, void *stream)
{
    return decompress_chunks(desc, buf, buf_bytes, meta, dst_chunk_ids, n, kv_out, workspace, workspace_bytes, stream, false);
}

extern "C" int llms_decompress_chunks_ordered(const llms_kv_desc *desc, const void *buf, uint64_t buf_bytes,
                                              const llms_chunk_meta *meta, const uint32_t *dst_chunk_ids, int n, void *kv_out,
                                              void *workspace, uint64_t workspace_bytes, void *stream)
{
    return decompress_chunks(desc, buf, buf_bytes, meta, dst_chunk_ids, n, kv_out, workspace, workspace_bytes, stream, true);
}

extern "C" int llms_codec_corrupt_count(const void *workspace, uint32_t *n_corrupt, void *stream)
{
    if (!workspace) return LLMS_ERR_INVALID_ARG;
    uint32_t status = 0;  // records with a wrong checksum
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    LLMS_CUDA_TRY(cudaMemcpyAsync(&status, workspace, 4, cudaMemcpyDeviceToHost, st));
    LLMS_CUDA_TRY(cudaStreamSynchronize(st));
    if (n_corrupt) *n_corrupt = status;
    return status ? LLMS_ERR_CORRUPT : LLMS_OK;
}

extern "C" int llms_debug_bounds(uint32_t *compiled_in, uint32_t *violations, uint64_t *first_address)
{
    if (!compiled_in || !violations || !first_address) return LLMS_ERR_INVALID_ARG;
    *compiled_in = 0;
    *violations = 0;
    *first_address = 0;
#ifdef LLMS_DEBUG_BOUNDS
    unsigned int count = 0;
    unsigned long long first = 0;
    LLMS_CUDA_TRY(cudaDeviceSynchronize());
    LLMS_CUDA_TRY(cudaMemcpyFromSymbol(&count, g_debug_violations, sizeof(count)));
    LLMS_CUDA_TRY(cudaMemcpyFromSymbol(&first, g_debug_first_address, sizeof(first)));
    *compiled_in = 1;
    *violations = count;
    *first_address = first;
#endif
    return LLMS_OK;
}

// ---------------------------------------------------------------------------------------------- no-allocation variant

namespace llms {

constexpr uint64_t kStaticWorkspaceBytes =
    (kWsEntriesOffset + (uint64_t)LLMS_STATIC_MAX_CHUNKS * kWsBytesPerChunk + 255) / 256 * 256;

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
