// Channel-wise mode (quant_mode 1): one {scale, zero-point} per channel of a slab, taken over the chunk's tokens
// - the paper's own wording for its quantizer (Sec. 3.2).  The code stream is unchanged (memory order); only the
// groups run down the token axis instead of along it.
//
// A warp takes one slab (chunk_len x head_dim) at a time.  The slab is seen as head_dim/8 columns of 16-byte
// chunks; a lane owns one column (8 channels) for every (32 / columns)-th token, so a warp instruction still
// touches consecutive addresses.  Pass 1 takes the column minima and maxima (packed half2, then xor-shuffles over
// the lanes that share a column); pass 2 reads the slab again (it is in L1/L2 by then), quantizes each value with
// its own channel's parameters and packs 8 codes per lane and token (8, 4, 2 bytes or 1 byte).  head_dim 64, 128 or 256.
#pragma once

namespace llms {

struct CwGeo {
    int cols;  // 16-byte columns per token row
    int lpc;   // lanes per column
    int col, sub;
    __device__ __forceinline__ CwGeo(int head_dim, int lane)
    {
        cols = head_dim / 8;
        lpc = 32 / cols;
        col = lane % cols;
        sub = lane / cols;
    }
};

// item -> (entry of the launch's table, slab index): chunk fastest, as in the other kernels
__device__ __forceinline__ void cw_item(const CodecArgs &a, uint32_t item, UnitEntry &ent, uint32_t &s_idx)
{
    uint32_t k;
    a.div_n.divmod(item, s_idx, k);
    ent = a.table[k];
}

template <int BITS>
__global__ void __launch_bounds__(kThreads) compress_cw_kernel(const CodecArgs a, const int head_dim, const int chunk_len)
{
    const int lane = threadIdx.x & 31;
    const CwGeo geo(head_dim, lane);
    const uint32_t total = (uint32_t)a.n * (uint32_t)a.n_slabs;
    UnitFeed feed;   // slabs are drawn like the units of the other kernels
    feed.start(a.feed, total, lane);
    for (uint32_t item = feed.pop(lane); item < total; item = feed.pop(lane)) {
        UnitEntry ent;
        uint32_t s_idx;
        cw_item(a, item, ent, s_idx);
        const __half *src = a.kv_in + slab_offset(a, s_idx, ent.chunk_id) + geo.col * 8;
        uint8_t *rec = a.buf + ent.rec_off;

        // ---- pass 1: minima and maxima of the lane's 8 channels over its tokens, then over the column's lanes
        __half2 mn[4], mx[4];
        {
            // a lane beyond the last token starts from token 0 again: duplicates do not change a minimum or maximum
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(src + (int64_t)(geo.sub < chunk_len ? geo.sub : 0) * head_dim));
            mn[0] = mx[0] = as_h2(w.x); mn[1] = mx[1] = as_h2(w.y); mn[2] = mx[2] = as_h2(w.z); mn[3] = mx[3] = as_h2(w.w);
        }
        for (int t = geo.sub + geo.lpc; t < chunk_len; t += geo.lpc) {
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(src + (int64_t)t * head_dim));
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                mn[i] = __hmin2(mn[i], as_h2(ww[i]));
                mx[i] = __hmax2(mx[i], as_h2(ww[i]));
            }
        }
        for (int x = geo.cols; x < 32; x <<= 1) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                mn[i] = __hmin2(mn[i], as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mn[i]), x)));
                mx[i] = __hmax2(mx[i], as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mx[i]), x)));
            }
        }
        GroupParams gp[8];
        bool any_clamp = false;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            gp[2 * i] = group_params<BITS>(__halves2half2(__low2half(mn[i]), __hneg(__low2half(mx[i]))));
            gp[2 * i + 1] = group_params<BITS>(__halves2half2(__high2half(mn[i]), __hneg(__high2half(mx[i]))));
            any_clamp |= gp[2 * i].needs_clamp | gp[2 * i + 1].needs_clamp;
        }
        const bool clamp = __any_sync(0xffffffffu, any_clamp);
        uint32_t sum = 0;
        if (geo.sub == 0) {
            uint32_t *params = reinterpret_cast<uint32_t *>(rec) + (uint64_t)s_idx * head_dim + geo.col * 8;
            st128(params, gp[0].word, gp[1].word, gp[2].word, gp[3].word);
            st128(params + 4, gp[4].word, gp[5].word, gp[6].word, gp[7].word);
#pragma unroll
            for (int i = 0; i < 8; ++i) sum += gp[i].word;
        }

        // ---- pass 2: codes
        constexpr float kQmax = (float)((1 << BITS) - 1);
        uint8_t *codes = rec + a.codes_off + ((uint64_t)s_idx * a.slab_elems + geo.col * 8) * BITS / 8;
        for (int t = geo.sub; t < chunk_len; t += geo.lpc) {
            const uint4 w = __ldg(reinterpret_cast<const uint4 *>(src + (int64_t)t * head_dim));
            const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
            uint32_t tq[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                unsigned short lo, hi;
                split_halves(ww[i], lo, hi);
                float v0 = __fmul_rn(add_f32_f16(lo, gp[2 * i].neg_zero_point), gp[2 * i].inv);
                float v1 = __fmul_rn(add_f32_f16(hi, gp[2 * i + 1].neg_zero_point), gp[2 * i + 1].inv);
                if (clamp) {  // only when some scale is a subnormal fp16 number
                    v0 = fminf(v0, kQmax);
                    v1 = fminf(v1, kQmax);
                }
                tq[2 * i] = __float_as_uint(__fadd_rn(v0, kRoundMagic));
                tq[2 * i + 1] = __float_as_uint(__fadd_rn(v1, kRoundMagic));
            }
            uint8_t *dst = codes + (uint64_t)t * head_dim * BITS / 8;
            if constexpr (BITS == 8) {
                const uint32_t o0 = __byte_perm(__byte_perm(tq[0], tq[1], 0x0040), __byte_perm(tq[2], tq[3], 0x0040), 0x5410);
                const uint32_t o1 = __byte_perm(__byte_perm(tq[4], tq[5], 0x0040), __byte_perm(tq[6], tq[7], 0x0040), 0x5410);
                st64(dst, o0, o1);
                sum += o0 + o1;
            } else {
                uint32_t ones = 0;
#pragma unroll
                for (int k = 0; k < 8; ++k) ones += 1u << (k * BITS);
                uint32_t acc = 0u - kRoundMagicBits * ones;
#pragma unroll
                for (int k = 0; k < 8; ++k) acc += tq[k] << (k * BITS);
                if constexpr (BITS == 4) {
                    st32(dst, acc);
                    sum += acc;
                } else if constexpr (BITS == 2) {
                    st16(dst, acc);
                    sum += acc << ((geo.col & 1) * 16);  // its half of the record's 32-bit word
                } else {
                    asm volatile("st.global.L1::no_allocate.b8 [%1], %0;" :: "r"(acc), "l"(dst) : "memory");
                    sum += acc << ((geo.col & 3) * 8);   // its byte of the record's 32-bit word
                }
            }
        }
        if (s_idx == 0) zero_padding(a, rec, BITS, lane);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.entries[ent.entry].checksum, sum);
    }
}

// The same with the whole slab in registers, for slabs of TOK tokens per lane (chunk_len = TOK * lanes per
// column): one read of the slab, all of a warp's loads in flight at once, no second pass.  Three CTAs per SM
// measured best on the 7B shape (0.636 ms; 0.677 at two with 128 registers, 0.675 at four with spills).
template <int BITS, int TOK>
__global__ void __launch_bounds__(kThreads, 3) compress_cw_reg_kernel(const CodecArgs a, const int head_dim)
{
    const int lane = threadIdx.x & 31;
    const CwGeo geo(head_dim, lane);
    const uint32_t total = (uint32_t)a.n * (uint32_t)a.n_slabs;
    UnitFeed feed;   // slabs are drawn like the units of the other kernels
    feed.start(a.feed, total, lane);
    for (uint32_t item = feed.pop(lane); item < total; item = feed.pop(lane)) {
        UnitEntry ent;
        uint32_t s_idx;
        cw_item(a, item, ent, s_idx);
        const __half *src = a.kv_in + slab_offset(a, s_idx, ent.chunk_id) + geo.col * 8;
        uint8_t *rec = a.buf + ent.rec_off;
        uint32_t w[TOK][4];
#pragma unroll
        for (int i = 0; i < TOK; ++i) ld128(src + (int64_t)(geo.sub + i * geo.lpc) * head_dim, w[i]);

        // ---- minima and maxima of the lane's 8 channels over its tokens, then over the column's lanes
        __half2 mn[4], mx[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) mn[c] = mx[c] = as_h2(w[0][c]);
#pragma unroll
        for (int i = 1; i < TOK; ++i)
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mn[c] = __hmin2(mn[c], as_h2(w[i][c]));
                mx[c] = __hmax2(mx[c], as_h2(w[i][c]));
            }
        for (int x = geo.cols; x < 32; x <<= 1) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                mn[c] = __hmin2(mn[c], as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mn[c]), x)));
                mx[c] = __hmax2(mx[c], as_h2(__shfl_xor_sync(0xffffffffu, as_u32(mx[c]), x)));
            }
        }
        GroupParams gp[8];
        bool any_clamp = false;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            gp[2 * c] = group_params<BITS>(__halves2half2(__low2half(mn[c]), __hneg(__low2half(mx[c]))));
            gp[2 * c + 1] = group_params<BITS>(__halves2half2(__high2half(mn[c]), __hneg(__high2half(mx[c]))));
            any_clamp |= gp[2 * c].needs_clamp | gp[2 * c + 1].needs_clamp;
        }
        const bool clamp = __any_sync(0xffffffffu, any_clamp);
        uint32_t sum = 0;
        if (geo.sub == 0) {
            uint32_t *params = reinterpret_cast<uint32_t *>(rec) + (uint64_t)s_idx * head_dim + geo.col * 8;
            st128(params, gp[0].word, gp[1].word, gp[2].word, gp[3].word);
            st128(params + 4, gp[4].word, gp[5].word, gp[6].word, gp[7].word);
#pragma unroll
            for (int c = 0; c < 8; ++c) sum += gp[c].word;
        }

        // ---- codes
        constexpr float kQmax = (float)((1 << BITS) - 1);
        uint8_t *codes = rec + a.codes_off + ((uint64_t)s_idx * a.slab_elems + geo.col * 8) * BITS / 8;
#pragma unroll
        for (int i = 0; i < TOK; ++i) {
            uint32_t tq[8];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                unsigned short lo, hi;
                split_halves(w[i][c], lo, hi);
                float v0 = __fmul_rn(add_f32_f16(lo, gp[2 * c].neg_zero_point), gp[2 * c].inv);
                float v1 = __fmul_rn(add_f32_f16(hi, gp[2 * c + 1].neg_zero_point), gp[2 * c + 1].inv);
                if (clamp) {  // only when some scale is a subnormal fp16 number
                    v0 = fminf(v0, kQmax);
                    v1 = fminf(v1, kQmax);
                }
                tq[2 * c] = __float_as_uint(__fadd_rn(v0, kRoundMagic));
                tq[2 * c + 1] = __float_as_uint(__fadd_rn(v1, kRoundMagic));
            }
            uint8_t *dst = codes + (uint64_t)(geo.sub + i * geo.lpc) * head_dim * BITS / 8;
            if constexpr (BITS == 8) {
                const uint32_t o0 = __byte_perm(__byte_perm(tq[0], tq[1], 0x0040), __byte_perm(tq[2], tq[3], 0x0040), 0x5410);
                const uint32_t o1 = __byte_perm(__byte_perm(tq[4], tq[5], 0x0040), __byte_perm(tq[6], tq[7], 0x0040), 0x5410);
                st64(dst, o0, o1);
                sum += o0 + o1;
            } else {
                uint32_t ones = 0;
#pragma unroll
                for (int k = 0; k < 8; ++k) ones += 1u << (k * BITS);
                uint32_t acc = 0u - kRoundMagicBits * ones;
#pragma unroll
                for (int k = 0; k < 8; ++k) acc += tq[k] << (k * BITS);
                if constexpr (BITS == 4) {
                    st32(dst, acc);
                    sum += acc;
                } else if constexpr (BITS == 2) {
                    st16(dst, acc);
                    sum += acc << ((geo.col & 1) * 16);
                } else {
                    asm volatile("st.global.L1::no_allocate.b8 [%1], %0;" :: "r"(acc), "l"(dst) : "memory");
                    sum += acc << ((geo.col & 3) * 8);
                }
            }
        }
        if (s_idx == 0) zero_padding(a, rec, BITS, lane);
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.entries[ent.entry].checksum, sum);
    }
}

template <int BITS>
__global__ void __launch_bounds__(kThreads) decompress_cw_kernel(const CodecArgs a, const int head_dim, const int chunk_len)
{
    const int lane = threadIdx.x & 31;
    const CwGeo geo(head_dim, lane);
    constexpr float kQmax = (float)((1 << BITS) - 1);
    // fixed split: with drawn slabs this kernel, which keeps no load ahead of its stores, ran 5% slower (0.580 -> 0.611 ms)
    const uint32_t n_warps = gridDim.x * kWarpsPerBlock;
    const uint32_t total = (uint32_t)a.n * (uint32_t)a.n_slabs;
    for (uint32_t item = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); item < total; item += n_warps) {
        UnitEntry ent;
        uint32_t s_idx;
        cw_item(a, item, ent, s_idx);
        const uint8_t *rec = a.buf + ent.rec_off;
        __half *dst = a.kv_out + slab_offset(a, s_idx, ent.chunk_id) + geo.col * 8;
        uint32_t p[8];
        {
            const uint32_t *params = reinterpret_cast<const uint32_t *>(rec) + (uint64_t)s_idx * head_dim + geo.col * 8;
            ld128(params, p);
            ld128(params + 4, p + 4);
        }
        float zero[8];
        bool any_clamp = false;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            zero[i] = __half2float(__ushort_as_half((unsigned short)(p[i] >> 16)));
            any_clamp |= __fmaf_rn(kQmax, __half2float(__ushort_as_half((unsigned short)(p[i] & 0xffffu))), zero[i]) > 65504.0f;
        }
        const bool clamp = __any_sync(0xffffffffu, any_clamp);
        uint32_t sum = 0;
        if (geo.sub == 0) {
#pragma unroll
            for (int i = 0; i < 8; ++i) sum += p[i];
        }
        const uint8_t *codes = rec + a.codes_off + ((uint64_t)s_idx * a.slab_elems + geo.col * 8) * BITS / 8;
        for (int t = geo.sub; t < chunk_len; t += geo.lpc) {
            const uint8_t *src = codes + (uint64_t)t * head_dim * BITS / 8;
            uint32_t c[2] = {0, 0};
            if constexpr (BITS == 8) {
                ld64(src, c);
                sum += c[0] + c[1];
            } else if constexpr (BITS == 4) {
                ld32(src, c);
                sum += c[0];
            } else if constexpr (BITS == 2) {
                ld16(src, c);
                sum += c[0] << ((geo.col & 1) * 16);
            } else {
                asm volatile("ld.global.nc.L1::no_allocate.u8 %0, [%1];" : "=r"(c[0]) : "l"(src));
                sum += c[0] << ((geo.col & 3) * 8);
            }
            // the 8 codes as exact fp16 integers (0x6400 | q = 1024 + q), in channel order
            const __half2 k1024 = as_h2(0x64006400u);
            __half2 q[4];
            if constexpr (BITS == 8) {
                q[0] = __hsub2(as_h2(__byte_perm(c[0], 0x64646464u, 0x4140)), k1024);
                q[1] = __hsub2(as_h2(__byte_perm(c[0], 0x64646464u, 0x4342)), k1024);
                q[2] = __hsub2(as_h2(__byte_perm(c[1], 0x64646464u, 0x4140)), k1024);
                q[3] = __hsub2(as_h2(__byte_perm(c[1], 0x64646464u, 0x4342)), k1024);
            } else {
                // codes 0..3 in the low 16 bits, codes 4..7 in the high 16 bits (at 4 bits they already are)
                const uint32_t z = BITS == 4 ? c[0]
                                   : BITS == 2 ? ((c[0] & 0xFFu) | ((c[0] & 0xFF00u) << 8))
                                               : ((c[0] & 0xFu) | ((c[0] & 0xF0u) << 12));
                constexpr uint32_t kMask = BITS == 4 ? 0x000F000Fu : BITS == 2 ? 0x00030003u : 0x00010001u;
#pragma unroll
                for (int s = 0; s < 4; ++s)  // codes s (low half) and s + 4 (high half)
                    q[s] = __hsub2(as_h2(((z >> (BITS * s)) & kMask) | 0x64006400u), k1024);
            }
            float y[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                unsigned short lo, hi;
                int idx, up;
                if constexpr (BITS == 8) { idx = e / 2; up = e % 2; }
                else { idx = e % 4; up = e / 4; }
                split_halves(as_u32(q[idx]), lo, hi);
                y[e] = fma_f32_f16(up ? hi : lo, (unsigned short)(p[e] & 0xffffu), zero[e]);
                if (clamp) y[e] = fminf(y[e], 65504.0f);
            }
            st128(dst + (int64_t)t * head_dim, as_u32(__floats2half2_rn(y[0], y[1])), as_u32(__floats2half2_rn(y[2], y[3])),
                  as_u32(__floats2half2_rn(y[4], y[5])), as_u32(__floats2half2_rn(y[6], y[7])));
        }
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.sums[ent.entry], sum);
    }
}

// Decoder with all of a slab's codes fetched before the first value is produced (TOK tokens per lane).
template <int BITS, int TOK>
__global__ void __launch_bounds__(kThreads) decompress_cw_reg_kernel(const CodecArgs a, const int head_dim)
{
    const int lane = threadIdx.x & 31;
    const CwGeo geo(head_dim, lane);
    // fixed split: with drawn slabs this kernel, which keeps no load ahead of its stores, ran 5% slower (0.580 -> 0.611 ms)
    const uint32_t n_warps = gridDim.x * kWarpsPerBlock;
    const uint32_t total = (uint32_t)a.n * (uint32_t)a.n_slabs;
    for (uint32_t item = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); item < total; item += n_warps) {
        UnitEntry ent;
        uint32_t s_idx;
        cw_item(a, item, ent, s_idx);
        const uint8_t *rec = a.buf + ent.rec_off;
        __half *dst = a.kv_out + slab_offset(a, s_idx, ent.chunk_id) + geo.col * 8;
        uint32_t p[8];
        {
            const uint32_t *params = reinterpret_cast<const uint32_t *>(rec) + (uint64_t)s_idx * head_dim + geo.col * 8;
            ld128(params, p);
            ld128(params + 4, p + 4);
        }
        const uint8_t *codes = rec + a.codes_off + ((uint64_t)s_idx * a.slab_elems + geo.col * 8) * BITS / 8;
        uint32_t c[TOK][2];
#pragma unroll
        for (int i = 0; i < TOK; ++i) {
            const uint8_t *src = codes + (uint64_t)(geo.sub + i * geo.lpc) * head_dim * BITS / 8;
            c[i][1] = 0;
            if constexpr (BITS == 8) ld64(src, c[i]);
            else if constexpr (BITS == 4) ld32(src, c[i]);
            else if constexpr (BITS == 2) ld16(src, c[i]);
            else asm volatile("ld.global.nc.L1::no_allocate.u8 %0, [%1];" : "=r"(c[i][0]) : "l"(src));
        }
        float zero[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) zero[e] = __half2float(__ushort_as_half((unsigned short)(p[e] >> 16)));
        uint32_t sum = 0;
        if (geo.sub == 0) {
#pragma unroll
            for (int e = 0; e < 8; ++e) sum += p[e];
        }
        const __half2 k1024 = as_h2(0x64006400u);
#pragma unroll
        for (int i = 0; i < TOK; ++i) {
            if constexpr (BITS == 8) sum += c[i][0] + c[i][1];
            else if constexpr (BITS == 4) sum += c[i][0];
            else if constexpr (BITS == 2) sum += c[i][0] << ((geo.col & 1) * 16);
            else sum += c[i][0] << ((geo.col & 3) * 8);
            // the 8 codes as exact fp16 integers (0x6400 | q = 1024 + q), in channel order
            __half2 q[4];
            if constexpr (BITS == 8) {
                q[0] = __hsub2(as_h2(__byte_perm(c[i][0], 0x64646464u, 0x4140)), k1024);
                q[1] = __hsub2(as_h2(__byte_perm(c[i][0], 0x64646464u, 0x4342)), k1024);
                q[2] = __hsub2(as_h2(__byte_perm(c[i][1], 0x64646464u, 0x4140)), k1024);
                q[3] = __hsub2(as_h2(__byte_perm(c[i][1], 0x64646464u, 0x4342)), k1024);
            } else {
                const uint32_t z = BITS == 4 ? c[i][0]
                                   : BITS == 2 ? ((c[i][0] & 0xFFu) | ((c[i][0] & 0xFF00u) << 8))
                                               : ((c[i][0] & 0xFu) | ((c[i][0] & 0xF0u) << 12));
                constexpr uint32_t kMask = BITS == 4 ? 0x000F000Fu : BITS == 2 ? 0x00030003u : 0x00010001u;
#pragma unroll
                for (int s = 0; s < 4; ++s)  // codes s (low half) and s + 4 (high half)
                    q[s] = __hsub2(as_h2(((z >> (BITS * s)) & kMask) | 0x64006400u), k1024);
            }
            float y[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                unsigned short lo, hi;
                int idx, up;
                if constexpr (BITS == 8) { idx = e / 2; up = e % 2; }
                else { idx = e % 4; up = e / 4; }
                split_halves(as_u32(q[idx]), lo, hi);
                y[e] = fma_f32_f16(up ? hi : lo, (unsigned short)(p[e] & 0xffffu), zero[e]);
            }
            st128(dst + (int64_t)(geo.sub + i * geo.lpc) * head_dim, pack_half2_clamped(y[0], y[1]), pack_half2_clamped(y[2], y[3]),
                  pack_half2_clamped(y[4], y[5]), pack_half2_clamped(y[6], y[7]));
        }
        sum = __reduce_add_sync(0xffffffffu, sum);
        if (lane == 0) atomicAdd(&a.sums[ent.entry], sum);
    }
}

}  // namespace llms
