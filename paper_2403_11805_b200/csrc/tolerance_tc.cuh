// The logits kernel on the fifth-generation tensor cores (tcgen05), for head_dim 64 and 128 and up to 128 window
// rows per KV head.  Included by tolerance.cu.
//
// Why: the warp-level MMA kernel is bound by the latency of each warp's own instruction chain (fragment loads,
// MMAs, shuffles, one tile at a time), not by memory - with 32 rows per KV head it stays near 6.0 TB/s of K while a
// plain read stream reaches 6.9.  Here the product leaves the warps altogether:
//   * one thread feeds pairs of 128-token tiles (and, per (layer, KV head) pair, the query rows) into shared memory
//     with TMA tensor copies, 128-byte swizzled, a ring of stages ahead of the arithmetic;
//   * one thread issues the MMAs: S[128 rows x 256 tokens] = q[128 x d] K_tiles[256 x d]^T, two neighbouring tiles of
//     a pair at a time (an MMA of 256 columns holds the issuing thread hardly longer than one of 128: with one tile per
//     MMA that thread was the pacemaker of the kernel), operands read from shared memory by the tensor core, the
//     accumulator in tensor memory (two accumulators of 256 columns take turns);
//   * the other warps only do the softmax statistics: a thread reads ITS window row's consecutive tokens from tensor
//     memory, so maxima and sums over a segment of tokens stay inside the thread (one or two shuffle steps where a
//     thread holds fewer tokens than a segment has).
// A warp can only read its own quarter of an accumulator's 128 lanes, and the lanes are the rows of the product.  So
// that all four quarters (and with them all four schedulers of the SM) share a tile's statistics whatever the number of
// rows, the pair's R rows (R = 8 .. 128, a power of two) are copied 128/R times into the A operand: copy k of a row
// sits in lane k*R + row and takes tokens k*R .. k*R + R - 1 of the tile.  The tensor core multiplies 128 rows either
// way.  Rows beyond the pair's own inside R belong to other heads' queries or are zero fill; nobody stores them.  Hand-offs between the three roles go through mbarriers; every wait is bounded: a role that waits too
// long raises a flag that turns the scores of the call into NaN, and still leaves through the common exit, where
// tensor memory is given back.
//
// Measured (B200, whole launches, K bytes / time): 32K-token grouped-query shape (32 rows per KV head), one tile per MMA:
// 352.8 us against 356.9 us for the warp-level kernel; 7B shape (8 rows) 177.6 against 165.3 us - so it is used from 32
// rows per KV head on.  Taking the MMAs or the statistics out of that kernel showed the feeding side alone at the pace of
// a resident-CTA read stream (6.9 TB/s); MMAs and statistics each added their time instead of hiding behind the copies,
// whatever the number of stages (2 to 5 made no difference), and asking tiles into L2 ahead of the ring made it slower.
// Cycle counters around the waits (32K shape, per tile of 1332 cycles) then showed the issuing thread held 890 cycles by
// a tile's eight MMAs (111 each, where the tensor pipe alone needs 68) and waiting 440, the feeding thread waiting 970
// for a free stage, a statistics warp working 750 cycles on a tile of its own and waiting 4400.  With the query rows in
// tensor memory instead of shared memory (three accumulators, tcgen05.st) a tile took 1282 cycles and the same time
// (not kept); with two tiles per MMA (this kernel) the score stage of the 32K shape went from 384 to 357 us.
#pragma once

#include <cuda.h>

namespace llms {

constexpr int kTcTile = 128;                         // tokens per tile: what a statistics warp group takes at a time
constexpr int kTcWide = 2 * kTcTile;                 // tokens per MMA (N = 256): two neighbouring tiles of a pair
constexpr int kTcAcc = 4;                            // tile-wide halves of the two 256-column accumulators (all 512 columns)
constexpr int kTcEpiWarps = 4 * kTcAcc;              // per accumulator one warp for each quarter of the 128 lanes
constexpr int kTcProducerWarp = kTcEpiWarps, kTcMmaWarp = kTcEpiWarps + 1;
constexpr int kTcThreads = (kTcEpiWarps + 2) * 32;
constexpr uint32_t kTcSpinLimit = 1u << 22;          // polls (with a pause in between) before a wait is given up
constexpr uint32_t kTcGaveUp = 0x7E57DEADu;          // value of the status word after a wait was given up
constexpr int kTcBlockBytes = kTcTile * 128;         // one 64-channel block of the 128-row A operand: 128 rows x 128 bytes
constexpr int kTcWideBlockBytes = kTcWide * 128;     // one 64-channel block of the 256-row B operand (two tiles of K)

struct TcBarriers {
    unsigned long long full[8], empty[8];            // tile stages (as many as fit, at most 8)
    unsigned long long q_full[2], q_empty[2];        // query-row buffers
    unsigned long long acc_full[kTcAcc], acc_empty[kTcAcc];
    uint32_t tmem_base;
    uint32_t gave_up;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Wait for the phase of the given parity to complete; false when the wait was given up.
__device__ __forceinline__ bool mbar_wait(unsigned long long *bar, uint32_t parity, volatile uint32_t *gave_up)
{
    const uint32_t addr = smem_u32(bar);
    for (uint32_t i = 0; i < kTcSpinLimit; ++i) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(addr), "r"(parity) : "memory");
        if (done) return true;
        if (*gave_up) return false;                   // another role has given up: no point in waiting on
        if (i > 32) __nanosleep(64);
    }
    *gave_up = 1;
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, unsigned long long *bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 :: "r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, int c0, int c1, int c2, int c3,
                                            unsigned long long *bar)
{
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 :: "r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// Shared-memory operand descriptor: rows of 128 bytes (64 fp16 channels, the contraction dimension contiguous), 128-byte
// swizzle, groups of eight rows 1024 bytes apart.  Fields: address / 16 in bits 0-13, leading offset (1, unused with a
// swizzle) in bits 16-29, stride between row groups / 16 in bits 32-45, descriptor version 1 in bits 46-47, swizzle
// mode 2 (128 bytes) in bits 61-63.
__device__ __forceinline__ uint64_t tc_operand_desc(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}

// Instruction descriptor: fp32 accumulator (bits 4-5 = 1), fp16 A and B (bits 7-9, 10-12 = 0), both with the
// contraction dimension contiguous (bits 15, 16 = 0), N / 8 in bits 17-22, M / 16 in bits 24-28.
constexpr uint32_t kTcInstrDesc = (1u << 4) | ((uint32_t)(kTcWide >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(kTcInstrDesc), "r"(accumulate) : "memory");
}
// The barrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(unsigned long long *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// N (8, 16 or 32) consecutive columns of this thread's lane of tensor memory
template <int N>
__device__ __forceinline__ void tc_load(uint32_t taddr, float (&v)[N])
{
    uint32_t r[N];
    if constexpr (N == 8) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]) : "r"(taddr));
    } else if constexpr (N == 16) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                     "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                       "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                     : "r"(taddr));
    } else {
        static_assert(N == 32, "8, 16 or 32 columns");
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                     "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, "
                     "%24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
                     : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
                       "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
                       "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
                       "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                     : "r"(taddr));
    }
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < N; ++i) v[i] = __uint_as_float(r[i]);
}

// Softmax statistics of this thread's window row over its N consecutive tokens (tok0 ..), per SEG-token segment, stored
// like the MMA kernel's (see row_statistics): log2 of the segment's sum of exp and, in the last W columns, of the
// weighted sum.
// N >= SEG: whole segments inside the thread.  N < SEG: the SEG/N threads that hold a segment's pieces are N lanes
// apart (copies of the row); they combine by shuffles and the one with the first piece stores.
// run_m, run_z: the thread's running (max, sum) pair over the segment values it has stored for its row (see
// lse_accumulate).
template <int SEG, int N, bool TAIL>
__device__ __forceinline__ void tc_statistics(const TolArgs &a, const float (&dot)[N], int tok0, int last_col, bool valid, int64_t out,
                                              int lane, float &run_m, float &run_z)
{
    constexpr float kLog2e = 1.4426950408889634f;
    constexpr int kPiece = SEG < N ? SEG : N;                    // tokens of one segment that this thread holds
    const float c1 = a.inv_sqrt_d * kLog2e;
#pragma unroll
    for (int s0 = 0; s0 < N; s0 += kPiece) {
        float v[kPiece];
        float m = -INFINITY;
#pragma unroll
        for (int i = 0; i < kPiece; ++i) {
            v[i] = dot[s0 + i];
            if constexpr (TAIL) v[i] = tok0 + s0 + i <= last_col ? v[i] : -INFINITY;
            m = fmaxf(m, v[i]);
        }
#pragma unroll
        for (int d = N; d < SEG; d <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
        const float neg = -(m * c1);
        float sum = 0.0f, wsum = 0.0f;
#pragma unroll
        for (int i = 0; i < kPiece; ++i) {
            float p = ex2_approx(__fmaf_rn(v[i], c1, neg));
            if constexpr (TAIL) {
                p = v[i] == -INFINITY ? 0.0f : p;
                const int n_vis = min(a.W, max(1, a.T - (tok0 + s0 + i)));
                wsum += p * (1.0f / (float)n_vis);
            }
            sum += p;
        }
#pragma unroll
        for (int d = N; d < SEG; d <<= 1) {
            sum += __shfl_xor_sync(0xffffffffu, sum, d);
            if constexpr (TAIL) wsum += __shfl_xor_sync(0xffffffffu, wsum, d);
        }
        const bool first_piece = N >= SEG || (lane & (SEG - N)) == 0;   // lane bits N .. SEG/2 number the pieces
        if (valid && first_piece && (!TAIL || tok0 + s0 < a.T)) {
            const int seg = (tok0 + s0) / SEG;
            const float l = __fmaf_rn(m, c1, lg2_approx(sum));   // -inf where the row sees none of the segment's tokens
            a.pl[(int64_t)seg * a.rows + out] = l;
            if constexpr (TAIL)
                if (seg >= a.seg_tail0) a.pw[(int64_t)(seg - a.seg_tail0) * a.rows + out] = __fmaf_rn(m, c1, lg2_approx(wsum));
            if (!TAIL || l != -INFINITY) lse_accumulate(run_m, run_z, l);
        }
    }
}

// Where a CTA is in the sequence of all tiles (pair-major): advanced tile by tile, so that the single threads that
// feed and issue pay no division per tile (a 64-bit division per tile made them the slowest stage of the pipeline).
struct TcCursor {
    int tile, kvh, l;
    __device__ __forceinline__ void start(int64_t idx, int tiles_per_pair, int n_kv_heads)
    {
        const int pair = (int)(idx / tiles_per_pair);
        tile = (int)(idx - (int64_t)pair * tiles_per_pair);
        l = pair / n_kv_heads;
        kvh = pair - l * n_kv_heads;
    }
    __device__ __forceinline__ void next(int tiles_per_pair, int n_kv_heads)
    {
        if (++tile == tiles_per_pair) {
            tile = 0;
            if (++kvh == n_kv_heads) {
                kvh = 0;
                ++l;
            }
        }
    }
};

// R: rows of a (layer, KV head) pair rounded up to a power of two (8 .. 128)
template <int SEG, int D, int R>
__global__ void __launch_bounds__(kTcThreads, 1) logits_tc_kernel(const TolArgs a, const __grid_constant__ CUtensorMap map_k,
                                                                  const __grid_constant__ CUtensorMap map_q, int n_stages)
{
    constexpr int kBlocks = D / 64;                              // 64-channel blocks of an operand
    constexpr int kOperandBytes = kBlocks * kTcBlockBytes;       // one buffer of query rows
    constexpr int kStageBytes = kBlocks * kTcWideBlockBytes;     // two neighbouring tiles of K
    extern __shared__ __align__(1024) unsigned char tc_smem_raw[];
    // operands need 1 KiB alignment for the swizzle; the barriers sit behind them
    unsigned char *base = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *q_buf = base;                                 // [2][kOperandBytes]
    unsigned char *k_buf = base + 2 * kOperandBytes;             // [n_stages][kStageBytes]
    TcBarriers *bar = reinterpret_cast<TcBarriers *>(k_buf + (size_t)n_stages * kStageBytes);
    volatile uint32_t *gave_up = &bar->gave_up;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int n_quarters = 4;                                // every quarter of an accumulator's lanes holds copies of the rows
    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&bar->full[s], 1);
            mbar_init(&bar->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bar->q_full[b], 1);
            mbar_init(&bar->q_empty[b], 1);
        }
        for (int g = 0; g < 2; ++g) {                            // the two accumulators of 256 columns
            mbar_init(&bar->acc_full[g], 1);
            mbar_init(&bar->acc_empty[g], 2 * n_quarters);       // both halves' four statistics warps
        }
        bar->gave_up = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kTcMmaWarp) {                                    // this warp owns tensor memory: all 512 columns
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&bar->tmem_base)), "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i <= a.n_x; i += blockDim.x) a.tickets[i] = 0;   // for the column kernel of this call
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bar->tmem_base;

    // this CTA's run of the sequence of all double tiles (pair-major); a pair's last one may have only its first half
    const int n_tiles = (a.T + kTcTile - 1) / kTcTile;
    const int tiles_per_pair = (n_tiles + 1) / 2;                // double tiles of a pair
    const int64_t total = (int64_t)a.L * a.Hkv * tiles_per_pair;
    const int64_t run_begin = total * blockIdx.x / gridDim.x, run_end = total * (blockIdx.x + 1) / gridDim.x;
    const int n_items = (int)(run_end - run_begin);

    if (warp == kTcProducerWarp) {
        if (lane == 0) {
            int pair_ord = -1, stage = 0, stage_round = 0;
            TcCursor at;
            at.start(run_begin, tiles_per_pair, a.Hkv);
            for (int it = 0; it < n_items; ++it, at.next(tiles_per_pair, a.Hkv)) {
                if (it == 0 || at.tile == 0) {                   // the pair's query rows, into the buffer that is free
                    ++pair_ord;
                    const int qb = pair_ord & 1, kq = pair_ord >> 1;
                    if (!mbar_wait(&bar->q_empty[qb], (kq & 1) ^ 1, gave_up)) break;
                    mbar_expect_tx(&bar->q_full[qb], kOperandBytes);
                    const int row0 = (at.l * a.Hq + at.kvh * a.rep) * a.W;
#pragma unroll
                    for (int b = 0; b < kBlocks; ++b)
                        for (int copy = 0; copy < kTcTile / R; ++copy)       // R rows x 128 bytes each
                            tma_load_2d(smem_u32(q_buf + qb * kOperandBytes + b * kTcBlockBytes + copy * R * 128), &map_q, b * 64, row0,
                                        &bar->q_full[qb]);
                }
                const int s = stage, parity = stage_round & 1;
                if (++stage == n_stages) {
                    stage = 0;
                    ++stage_round;
                }
                if (!mbar_wait(&bar->empty[s], parity ^ 1, gave_up)) break;
                mbar_expect_tx(&bar->full[s], kStageBytes);
#pragma unroll
                for (int b = 0; b < kBlocks; ++b)
                    tma_load_4d(smem_u32(k_buf + (size_t)s * kStageBytes + b * kTcWideBlockBytes), &map_k, b * 64, at.tile * kTcWide, at.kvh,
                                at.l, &bar->full[s]);
            }
        }
    } else if (warp == kTcMmaWarp) {
        if (lane == 0) {
            int pair_ord = -1, qb = 0, stage = 0, stage_round = 0;
            int tile = (int)(run_begin % tiles_per_pair);
            for (int it = 0; it < n_items; ++it) {
                if (it == 0 || tile == 0) {
                    ++pair_ord;
                    qb = pair_ord & 1;
                    if (!mbar_wait(&bar->q_full[qb], (pair_ord >> 1) & 1, gave_up)) break;
                }
                const int s = stage;
                if (!mbar_wait(&bar->full[s], stage_round & 1, gave_up)) break;
                if (++stage == n_stages) {
                    stage = 0;
                    ++stage_round;
                }
                const int g = it & 1, ka = it >> 1;              // accumulator, its turn
                if (!mbar_wait(&bar->acc_empty[g], (ka & 1) ^ 1, gave_up)) break;
                tc_fence_after();
                const uint32_t q_addr = smem_u32(q_buf + qb * kOperandBytes), k_addr = smem_u32(k_buf + (size_t)s * kStageBytes);
#pragma unroll
                for (int b = 0; b < kBlocks; ++b)
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)               // 16 channels (32 bytes) per MMA
                        tc_mma(tmem_base + g * kTcWide, tc_operand_desc(q_addr + b * kTcBlockBytes + kk * 32),
                               tc_operand_desc(k_addr + b * kTcWideBlockBytes + kk * 32), (b | kk) != 0);
                tc_commit(&bar->empty[s]);                       // the stage is free once these MMAs have read it
                tc_commit(&bar->acc_full[g]);
                const bool pair_ends = tile == tiles_per_pair - 1;
                if (pair_ends || it == n_items - 1) tc_commit(&bar->q_empty[qb]);
                tile = pair_ends ? 0 : tile + 1;
            }
        }
    } else {
        const int g = warp >> 2, quarter = warp & 3;             // half accumulator, lanes 32*quarter .. +31 of it
        const int acc = g >> 1, half = g & 1;                    // accumulator of 256 columns, which tile of its two
        constexpr int kPiece = R < 32 ? R : 32;                  // tokens a thread takes from one load of 32 columns
        const int m_index = quarter * 32 + lane;                 // this thread's row of the product
        const int j = m_index % R;                               // ... is copy m_index / R of row j of the pair,
        const int col0 = m_index / R * R;                        // which takes tokens col0 .. col0 + R - 1 of every tile
        const int sub = R < 32 ? lane / kPiece : 0;              // with several copies in a warp: which piece of the 32 columns
        const bool valid = j < a.NR;
        const int row_in_window = j % a.W;
        // this thread's place among the statistics threads of its row (the slot of its partial sums)
        const int copy_index = g * (kTcTile / R) + m_index / R;
        const bool keep = a.n_slots > 0;
        TcCursor at;
        at.start(run_begin + acc, tiles_per_pair, a.Hkv);
        int it = acc;                                            // this thread's next double tile, counted from the run's first
        bool alive = true;
        // pair by pair: every thread leaves a (max, sum) pair for every (layer, KV head) pair the run touches, also
        // where none of the pair's tiles fell to its accumulator
        for (int64_t pair = run_begin / tiles_per_pair; alive && pair * tiles_per_pair < run_end; ++pair) {
            const int64_t next_pair = (pair + 1) * tiles_per_pair;
            const int pair_end = (int)((run_end < next_pair ? run_end : next_pair) - run_begin);
            float run_m = -INFINITY, run_z = 0.0f;
            for (; it < pair_end; it += 2) {
                const int tile = 2 * at.tile + half;
                const int64_t out = pair * a.NR + j;             // this thread's row among all rows
                const int last_col = valid ? a.T - a.W + row_in_window : -1;
#pragma unroll
                for (int k = 0; k < 2; ++k) at.next(tiles_per_pair, a.Hkv);        // where the next trip is
                if (!mbar_wait(&bar->acc_full[acc], (it >> 1) & 1, gave_up)) {
                    alive = false;
                    break;
                }
                tc_fence_after();
                const bool tail_tile = tile * kTcTile + kTcTile > a.T - a.W + 1;
                // a load's column address is the same for the whole warp: with R < 32 the warp loads its quarter's 32
                // columns and every thread keeps the piece of its copy
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + g * kTcTile + (R < 32 ? quarter * 32 : col0);
#pragma unroll
                for (int c = 0; c < (R < 32 ? 1 : R / 32) && tile < n_tiles; ++c) {   // a pair's odd last tile has no second half
                    float got[32], dot[kPiece];
                    tc_load<32>(taddr + c * 32, got);
#pragma unroll
                    for (int i = 0; i < kPiece; ++i) dot[i] = got[i];
#pragma unroll
                    for (int k = 1; k < 32 / kPiece; ++k)
                        if (sub == k) {
#pragma unroll
                            for (int i = 0; i < kPiece; ++i) dot[i] = got[k * kPiece + i];
                        }
                    const int tok0 = tile * kTcTile + col0 + c * 32;
                    if (tail_tile) tc_statistics<SEG, kPiece, true>(a, dot, tok0, last_col, valid, out, lane, run_m, run_z);
                    else tc_statistics<SEG, kPiece, false>(a, dot, tok0, last_col, valid, out, lane, run_m, run_z);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar->acc_empty[acc]);
            }
            if (alive && keep && valid) {
                const int first_cta = tc_cta_of_tile(pair * tiles_per_pair, total, (int)gridDim.x);
                a.row_part[(pair * a.NR + j) * a.n_slots + ((int)blockIdx.x - first_cta) * a.tc_spr + copy_index] = make_float2(run_m, run_z);
            }
        }
    }

    // ---- common exit: everybody comes here, also after a wait was given up (then copies may still be on their way
    // into this CTA's shared memory: they are given time to land before the memory can go to another CTA)
    grid_launch_dependents();
    if (*gave_up)
        for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    tc_fence_before();
    __syncthreads();
    if (warp == kTcMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(512) : "memory");
    }
    if (threadIdx.x == 0 && bar->gave_up) atomicExch(a.status, kTcGaveUp);
}

}  // namespace llms
