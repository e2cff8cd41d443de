// Bulk-copy (TMA) pipelines of the chunk codec for groups of at least 64 channels.
//
// Every warp runs its own pipeline over its units (one unit = one 2048-element pass over a slab):
//   - lane 0 keeps bulk asynchronous copies (cp.async.bulk, global -> shared, completion on an mbarrier) of
//     the next units in flight into a ring of kStages 4 KiB buffers, so the memory system always has work and
//     no registers are spent on prefetching;
//   - the warp reads a landed unit from shared memory, lane L taking row L (its 64 consecutive elements) as
//     eight 16-byte chunks in rotated order (chunk (k + L) mod 8 in step k), which is free of bank conflicts;
//   - results are written back into the same buffer and leave with one bulk store (shared -> global).
// The copies use this GPU's own memory only and no multicast.  Every wait is bounded: a warp whose wait runs
// out counts itself in the workspace's second status word, drains its copies and returns.
#pragma once

namespace llms {

constexpr int kStages = 3;
constexpr int kUnitBytes = kPassElems * 2;                               // 4 KiB of fp16
constexpr int kRingBytes = kStages * kUnitBytes;                         // per warp
constexpr int kBulkSmemBytes = kWarpsPerBlock * (kRingBytes + kStages * 8);
constexpr uint32_t kSpinLimit = 1u << 17;  // try_wait itself suspends for a while: far beyond any real wait, yet bounded

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait for a phase of the barrier; false when it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t spin = 0; spin < kSpinLimit; ++spin)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst_smem), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" :: "l"(dst), "r"(src_smem), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// at most N of this thread's bulk stores may still be reading shared memory
template <int N>
__device__ __forceinline__ void bulk_store_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(N) : "memory");
}
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// make this thread's shared-memory writes visible to the copy engine
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ int unit_elems(const CodecArgs &a, const UnitPos &u, int lane)
{
    const int pass_e0 = u.e0 - lane * kLaneElems;
    return min(kPassElems, a.slab_elems - pass_e0);
}

// ---------------------------------------------------------------------------------------------- quantize

// 8 values (4 words of fp16 pairs) -> BITS bytes of codes: o0 (and o1 at 8 bits).  No clamp (see quantize_piece).
template <int BITS>
__device__ __forceinline__ void quantize_chunk(const uint4 &w, float neg_zero, float inv, uint32_t &o0, uint32_t &o1)
{
    const uint32_t in[4] = {w.x, w.y, w.z, w.w};
    uint32_t t[8];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        unsigned short lo, hi;
        split_halves(in[k], lo, hi);
        t[2 * k] = __float_as_uint(__fadd_rn(__fmul_rn(add_f32_f16(lo, neg_zero), inv), kRoundMagic));
        t[2 * k + 1] = __float_as_uint(__fadd_rn(__fmul_rn(add_f32_f16(hi, neg_zero), inv), kRoundMagic));
    }
    if constexpr (BITS == 8) {
        o0 = __byte_perm(__byte_perm(t[0], t[1], 0x0040), __byte_perm(t[2], t[3], 0x0040), 0x5410);
        o1 = __byte_perm(__byte_perm(t[4], t[5], 0x0040), __byte_perm(t[6], t[7], 0x0040), 0x5410);
    } else {
        uint32_t ones = 0;
#pragma unroll
        for (int k = 0; k < 8; ++k) ones += 1u << (k * BITS);
        uint32_t acc = 0u - kRoundMagicBits * ones;  // arithmetic mod 2^32: the magic's share cancels
#pragma unroll
        for (int k = 0; k < 8; ++k) acc += t[k] << (k * BITS);
        o0 = acc;
        o1 = 0;
    }
}

// rare case (subnormal scale): with the clamp, written for size
__device__ __noinline__ void quantize_chunk_clamped(uint4 w, float neg_zero, float inv, int bits, uint32_t *o)
{
    const uint32_t in[4] = {w.x, w.y, w.z, w.w};
    const float qmax = (float)((1 << bits) - 1);
    o[0] = o[1] = 0;
    for (int k = 0; k < 8; ++k) {
        const unsigned short x = (unsigned short)(in[k >> 1] >> ((k & 1) * 16));
        const uint32_t q = (uint32_t)__float2int_rn(fminf(__fmul_rn(add_f32_f16(x, neg_zero), inv), qmax));
        o[(k * bits) >> 5] |= q << ((k * bits) & 31);
    }
}

// A warp's position among the units.  Units are numbered slab-major (pass fastest, then the launch's chunks,
// then the slab index); warp w takes units w, w + W, w + 2W, ... (W = warps of the grid), so that at any moment
// the grid works on one narrow band of addresses (measured: a contiguous run per warp was 10% slower).  The
// stride W is pre-split into (passes, chunks, slab indices), so stepping needs no division.
struct Cursor {
    uint32_t unit, s_idx, k, pass;
    int64_t plane;  // element offset of the slab index's (layer, K/V, head) plane
};

__device__ __forceinline__ int64_t plane_offset(const CodecArgs &a, uint32_t s_idx)
{
    uint32_t ls, h;
    a.div_heads.divmod(s_idx, ls, h);
    return (int64_t)(ls >> 1) * a.stride_l + (int64_t)(ls & 1) * a.stride_s + (int64_t)h * a.stride_h;
}

__device__ __forceinline__ void cursor_init(const CodecArgs &a, uint32_t unit, Cursor &c)
{
    uint32_t item;
    c.unit = unit;
    a.div_passes.divmod(unit, item, c.pass);
    a.div_n.divmod(item, c.s_idx, c.k);
    c.plane = plane_offset(a, c.s_idx);
}

__device__ __forceinline__ void cursor_next(const CodecArgs &a, Cursor &c)
{
    c.unit += a.step_units;
    c.pass += a.step_pass;
    uint32_t carry = c.pass >= (uint32_t)a.passes;
    c.pass -= carry * (uint32_t)a.passes;
    c.k += a.step_k + carry;
    carry = c.k >= (uint32_t)a.n;
    c.k -= carry * (uint32_t)a.n;
    const uint32_t ds = a.step_s + carry;
    if (ds) {
        c.s_idx += ds;
        c.plane = plane_offset(a, c.s_idx);
    }
}

// elements of the pass the cursor stands on
__device__ __forceinline__ uint32_t cursor_elems(const CodecArgs &a, const Cursor &c)
{
    return (uint32_t)min(kPassElems, a.slab_elems - (int)c.pass * kPassElems);
}

template <int BITS, int G>
__global__ void __launch_bounds__(kThreads, 2) compress_bulk_kernel(const CodecArgs a)
{
    static_assert(G >= kLaneElems, "a lane holds a whole share of one group");
    constexpr int kLanesPerGroup = G / kLaneElems;
    constexpr int kLaneBytes = kLaneElems * BITS / 8;
    extern __shared__ __align__(128) uint8_t smem[];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    uint8_t *ring = smem + wib * kRingBytes;
    const uint32_t ring_s = smem_addr(ring);
    const uint32_t bars = smem_addr(smem + kWarpsPerBlock * kRingBytes) + wib * kStages * 8;
    // this warp's units: first, first + step_units, ...
    const uint32_t first = blockIdx.x * kWarpsPerBlock + wib;
    if (first >= a.total_units) return;
    const uint32_t count = (a.total_units - first + a.step_units - 1) / a.step_units;

    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbar_init(bars + s * 8, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    Cursor load_at, at;       // the unit whose copy is issued next; the unit being encoded
    cursor_init(a, first, at);
    load_at = at;
    uint32_t issued = 0;
    // lane 0: start the copy of the unit under load_at into buffer issued % kStages
    auto issue_load = [&]() {
        const uint32_t chunk_id = a.table[load_at.k].chunk_id;
        const uint32_t bytes = cursor_elems(a, load_at) * 2;
        const uint32_t s = issued % kStages;
        mbar_expect_tx(bars + s * 8, bytes);
        bulk_load(ring_s + s * kUnitBytes,
                  a.kv_in + load_at.plane + (int64_t)chunk_id * a.chunk_stride + load_at.pass * kPassElems, bytes, bars + s * 8);
    };
    for (; issued < (uint32_t)(kStages - 1) && issued < count; ++issued) {
        if (lane == 0) issue_load();
        cursor_next(a, load_at);
    }

    uint32_t m = 0;
    bool gave_up = false;
    for (; m < count; ++m) {
        const uint32_t s = m % kStages;
        const UnitEntry ent = a.table[at.k];
        if (!__all_sync(0xffffffffu, mbar_wait(bars + s * 8, (m / kStages) & 1))) {
            gave_up = true;
            break;
        }
        uint8_t *buf = ring + s * kUnitBytes;
        const int e0 = (int)at.pass * kPassElems + lane * kLaneElems;
        const bool active = e0 < a.slab_elems;  // G >= 64: a lane is wholly inside or wholly outside the slab
        uint4 w[8];
#pragma unroll
        for (int k = 0; k < 8; ++k)
            w[k] = active ? *reinterpret_cast<const uint4 *>(buf + lane * 128 + ((k + lane) & 7) * 16) : make_uint4(0, 0, 0, 0);
        __syncwarp();  // every lane has its row: the buffer can take the codes

        // ---- group minimum and maximum
        __half2 mn = as_h2(w[0].x), mx = as_h2(w[0].x);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            mn = __hmin2(__hmin2(mn, as_h2(w[k].x)), __hmin2(as_h2(w[k].y), __hmin2(as_h2(w[k].z), as_h2(w[k].w))));
            mx = __hmax2(__hmax2(mx, as_h2(w[k].x)), __hmax2(as_h2(w[k].y), __hmax2(as_h2(w[k].z), as_h2(w[k].w))));
        }
        __half2 mm = __halves2half2(__hmin(__low2half(mn), __high2half(mn)), __hneg(__hmax(__low2half(mx), __high2half(mx))));
#pragma unroll
        for (int x = kLanesPerGroup / 2; x > 0; x >>= 1) mm = __hmin2(mm, as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mm), x)));
        const GroupParams gp = group_params<BITS>(mm);

        // ---- codes, written over the unit's own buffer at byte lane*kLaneBytes + chunk*BITS
        uint32_t sum = 0;
        uint8_t *out = buf + lane * kLaneBytes;
        const bool slow = __any_sync(0xffffffffu, gp.needs_clamp);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int c = (k + lane) & 7;
            uint32_t o[2];
            if (slow) quantize_chunk_clamped(w[k], gp.neg_zero_point, gp.inv, BITS, o);
            else quantize_chunk<BITS>(w[k], gp.neg_zero_point, gp.inv, o[0], o[1]);
            if (active) {
                if constexpr (BITS == 8) {
                    *reinterpret_cast<uint2 *>(out + c * 8) = make_uint2(o[0], o[1]);
                    sum += o[0] + o[1];
                } else if constexpr (BITS == 4) {
                    *reinterpret_cast<uint32_t *>(out + c * 4) = o[0];
                    sum += o[0];
                } else {
                    *reinterpret_cast<unsigned short *>(out + c * 2) = (unsigned short)o[0];
                    sum += o[0] << ((c & 1) * 16);  // its place in the record's 32-bit word
                }
            }
        }
        fence_async_smem();
        __syncwarp();

        uint8_t *rec = a.buf + ent.rec_off;
        const uint32_t elem0 = at.s_idx * (uint32_t)a.slab_elems + at.pass * kPassElems;  // of the unit, inside the chunk
        if (lane == 0) {
            bulk_store(rec + a.codes_off + (uint64_t)elem0 * BITS / 8, ring_s + s * kUnitBytes, cursor_elems(a, at) * BITS / 8);
            bulk_store_wait_read<1>();  // the store of the unit before this one has let go of its buffer
            if (issued < count) issue_load();
        }
        if (issued < count) {
            ++issued;
            cursor_next(a, load_at);
        }
        if (active && (lane & (kLanesPerGroup - 1)) == 0) {
            st32(reinterpret_cast<uint32_t *>(rec) + (elem0 + (uint32_t)lane * kLaneElems) / G, gp.word);
            sum += gp.word;
        }
        if (at.s_idx == 0 && at.pass == 0) zero_padding(a, rec, BITS, lane);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.entries[ent.entry].checksum, sum);
        cursor_next(a, at);
    }
    if (gave_up) {
        // copies still in flight target this warp's buffers: give each a bounded chance to land before leaving
        if (lane == 0) atomicAdd(a.gave_up, 1u);
        for (uint32_t k = m; k < issued; ++k) mbar_wait(bars + (k % kStages) * 8, (k / kStages) & 1);
    }
    if (lane == 0) bulk_store_wait_all();
}

}  // namespace llms
