// Tolerance score (information density, Eq. 1) kernels for sm_100a.
//
// From probabilities: a column-mean reduction, one pass over the window.
// From K and the last W queries: K is streamed once.  The logits S = q K^T are a dense contraction and run on the
// tensor cores: warp-level MMAs (logits_mma_kernel) or, from 32 window rows per KV head on, tcgen05 MMAs fed by TMA
// (logits_tc_kernel, tolerance_tc.cuh); an fp32-FMA kernel with a thread per token remains for head dimensions
// neither takes.  The rows' softmax statistics are kept per *segment* of SEG neighbouring tokens (SEG = the largest
// power of two <= 32 that divides chunk_len) as one number: the base-2 logarithm of the segment's sum of exp(logit),
// its share of the row's softmax denominator (and, for the few segments that reach into the last W columns, the same
// of the 1/n_vis-weighted sum).  One kernel then turns the per-segment statistics into column sums and chunk means,
// once the rows' denominators are known: from partial sums the logits kernels keep while they run, or else from a
// pass over the statistics.  All sums run in a fixed order, so the scores - and the ranking made from them - are
// reproducible bit for bit.
#include <math.h>

#include <algorithm>

#include "llms_internal.cuh"

namespace llms {

constexpr int kTokThreads = 256;   // tokens per block in the logits kernel
constexpr int kRowTile = 8;        // query rows per pass over a key

constexpr int kMaxRowSlots = 32;   // most partial sums a logits kernel leaves per row

struct TolArgs {
    const __half *kv;
    const __half *q_win;
    int L, Hkv, Hq, d, T, W, CL;
    int rep;          // query heads per KV head
    int NR;           // rep * W query rows per KV head
    int n_seg;        // ceil(T / SEG)
    int seg_tail0;    // first segment that holds a token of the last W - 1 columns (where rows stop seeing tokens)
    int seg_per_chunk;
    int n_chunks;
    int64_t stride_l, stride_h;
    float inv_sqrt_d;
    float *pl;                // [n_seg][rows]: log2 of the sum of exp(logit) over the segment's tokens that the row sees
                              // (-inf where it sees none).  Rows are the fast index: the rows of a (layer, KV head)
                              // pair that a warp holds for one segment are then neighbours in memory (with segments
                              // as the fast index every store touched a sector per row, as many requests to L2 as
                              // the kernel's loads of K)
    float *pw;                // [n_seg - seg_tail0][rows]: the same of the 1/n_vis-weighted sum, for the segments from
                              // seg_tail0 on (before them the weighted sum is the plain one over W)
    float *row_lse;           // [rows]: log2 of a row's softmax denominator, where a kernel of its own makes it
    float2 *row_part;         // [rows][n_slots]: (max, sum of 2^(l - max)) over the segment values l of a row that one
                              // slot covers: a CTA of the MMA kernel, or a thread of a CTA of the tcgen05 kernel
    int n_slots;              // slots per row; 0: the logits kernel keeps no partial sums (row_stats_kernel follows)
    int lse_ready;            // column kernel: 1 = row_lse holds the denominators, 0 = combine the row's slots
    int tc_grid, tc_spr;      // tcgen05 kernel: its CTAs, and its statistics threads per row
    float *part;              // [Y][n_seg]
    float *colsum;            // [n_seg]: column sums over all rows
    uint32_t *tickets;        // [n_x + 1]: finished row slices per group of 32 segments, finished groups; the logits
                              // kernel of the same call clears them
    int n_x;                  // groups of 32 segments
    uint32_t *status;         // set to a magic value by a logits kernel that gave a bounded wait up: the scores of the
                              // call then come out as NaN (and the word is cleared)
    float *scores;
    float *scores_live;       // optional second destination of the scores (page-locked host memory), or NULL
    int Y, rows;
};

// ------------------------------------------------------------------ K and q -> per-segment softmax statistics

template <int SEG>
__global__ void __launch_bounds__(kTokThreads) logits_kernel(const TolArgs a)
{
    extern __shared__ float q_s[];  // [NR][d] fp32
    const int l = blockIdx.y / a.Hkv, kvh = blockIdx.y % a.Hkv;
    const __half *q_src = a.q_win + ((int64_t)(l * a.Hq + kvh * a.rep) * a.W) * a.d;
    for (int i = threadIdx.x; i < a.NR * a.d; i += blockDim.x) q_s[i] = __half2float(q_src[i]);
    __syncthreads();

    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = threadIdx.x; i <= a.n_x; i += blockDim.x) a.tickets[i] = 0;   // for the column kernel of this call
    const int t = blockIdx.x * kTokThreads + threadIdx.x;
    const bool valid = t < a.T;
    const int lane = threadIdx.x & 31;
    const uint4 *k_row = reinterpret_cast<const uint4 *>(a.kv + (int64_t)l * a.stride_l + (int64_t)kvh * a.stride_h +
                                                         (int64_t)(valid ? t : 0) * a.d);
    const int n_vis = min(a.W, a.T - (valid ? t : 0));
    const float w_col = 1.0f / (float)n_vis;
    const int seg = t / SEG;
    const int64_t row0 = (int64_t)(l * a.Hq + kvh * a.rep) * a.W;

    for (int j0 = 0; j0 < a.NR; j0 += kRowTile) {
        float acc[kRowTile];
#pragma unroll
        for (int j = 0; j < kRowTile; ++j) acc[j] = 0.0f;
        if (valid) {
            for (int c8 = 0; c8 < a.d / 8; ++c8) {
                const uint4 kk = __ldg(k_row + c8);
                const float2 k0 = __half22float2(*reinterpret_cast<const __half2 *>(&kk.x));
                const float2 k1 = __half22float2(*reinterpret_cast<const __half2 *>(&kk.y));
                const float2 k2 = __half22float2(*reinterpret_cast<const __half2 *>(&kk.z));
                const float2 k3 = __half22float2(*reinterpret_cast<const __half2 *>(&kk.w));
#pragma unroll
                for (int j = 0; j < kRowTile; ++j) {
                    if (j0 + j < a.NR) {
                        const float4 qa = *reinterpret_cast<const float4 *>(q_s + (j0 + j) * a.d + c8 * 8);
                        const float4 qb = *reinterpret_cast<const float4 *>(q_s + (j0 + j) * a.d + c8 * 8 + 4);
                        acc[j] = fmaf(k0.x, qa.x, acc[j]);
                        acc[j] = fmaf(k0.y, qa.y, acc[j]);
                        acc[j] = fmaf(k1.x, qa.z, acc[j]);
                        acc[j] = fmaf(k1.y, qa.w, acc[j]);
                        acc[j] = fmaf(k2.x, qb.x, acc[j]);
                        acc[j] = fmaf(k2.y, qb.y, acc[j]);
                        acc[j] = fmaf(k3.x, qb.z, acc[j]);
                        acc[j] = fmaf(k3.y, qb.w, acc[j]);
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < kRowTile; ++j) {
            if (j0 + j >= a.NR) break;  // uniform across the block
            const int r = (j0 + j) % a.W;
            const bool vis = valid && t <= a.T - a.W + r;
            const float logit = vis ? acc[j] * a.inv_sqrt_d : -INFINITY;
            float m = logit;
#pragma unroll
            for (int s = SEG / 2; s > 0; s >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
            const float e = vis ? expf(logit - m) : 0.0f;
            float se = e, sp = e * w_col;
#pragma unroll
            for (int s = SEG / 2; s > 0; s >>= 1) {
                se += __shfl_xor_sync(0xffffffffu, se, s);
                sp += __shfl_xor_sync(0xffffffffu, sp, s);
            }
            if (valid && (lane & (SEG - 1)) == 0) {
                constexpr float kLog2e = 1.4426950408889634f;
                const int64_t row = row0 + j0 + j;
                a.pl[(int64_t)seg * a.rows + row] = se > 0.0f ? fmaf(m, kLog2e, log2f(se)) : -INFINITY;
                if (seg >= a.seg_tail0)
                    a.pw[(int64_t)(seg - a.seg_tail0) * a.rows + row] = sp > 0.0f ? fmaf(m, kLog2e, log2f(sp)) : -INFINITY;
            }
        }
    }
}

// ------------------------------------------------------------------ the same on the tensor cores
//
// S = q K^T is a dense contraction (window rows x head_dim times head_dim x tokens): with plain fp32 fma the kernel
// is bound by instruction issue (measured 0.56 ms for the 7B shape against 0.17 ms for reading K once), so for
// head_dim 64, 128 and 256 it runs as warp-level matrix multiply-accumulate, m16n8k16 with fp16 inputs and fp32
// accumulators.  A warp owns tiles of 32 consecutive tokens of one (layer, KV head).  It copies a tile
// (32 x head_dim fp16, contiguous in memory) into shared memory with coalesced 16-byte asynchronous copies,
// swizzled by XOR-ing the 16-byte chunk index with the row index so that ldmatrix reads without bank conflicts.
//
// The window's query rows are the M side of the product (A operand, 16 rows per m-tile, rows of shared memory padded
// by 16 bytes against conflicts) and the tile's tokens the N side (B operand, four n-tiles of 8 tokens).  An
// accumulator fragment then holds, per lane, two window rows (g and g + 8) and for each of them eight tokens of the
// tile (2*q4, 2*q4 + 1 of every n-tile): the softmax statistics of a row over a segment of tokens are mostly sums
// inside a lane, finished by at most two shuffle steps.  (With the tokens on the M side, as this kernel first had
// them, every statistic took three shuffle steps per pair of values and the kernel spent two thirds of its 1180
// instructions per tile there: 0.52 ms for the 32K grouped-query shape, whose K streams past in 0.33 ms.)
constexpr int kTileTokens = 32;
constexpr int kTileWarps = 12;     // most warps a CTA is launched with; 8 when twelve tiles do not fit twice into an SM
constexpr int kTileWarpsSmall = 8;  // (measured on the 7B shape: 12 warps x 2 CTAs 0.2175 ms, 8 x 3 0.227, 4 x 6 0.269)
constexpr int kTileBuffers = 1;   // per warp; with 1 the other warps of the SM cover a warp's copy latency

// 16-byte asynchronous copy global -> shared, bypassing L1; src_bytes = 0 fills zeros instead
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// 2^x, one instruction (relative error about 2^-22; results below the normal range become 0)
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// log2(x), one instruction (absolute error about 2^-22; 0 gives -inf)
__device__ __forceinline__ float lg2_approx(float x)
{
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// (M, Z) stands for M + log2(Z), the base-2 logarithm of a sum of powers of two; add 2^l to that sum.  l is finite.
__device__ __forceinline__ void lse_accumulate(float &M, float &Z, float l)
{
    const float d = l - M;                      // +inf the first time (M = -inf, Z = 0)
    const float e = ex2_approx(-fabsf(d));
    if (d > 0.0f) {
        Z = __fmaf_rn(Z, e, 1.0f);
        M = l;
    } else {
        Z += e;
    }
}

// x[nt][e] belongs to token nt*8 + 2*q4 + e of the tile (q4 = lane & 3).  Reduce over the tokens of each SEG-token
// segment; afterwards every slot holds its segment's result.  The order of the operations is fixed by SEG alone.
template <int SEG, typename Op>
__device__ __forceinline__ void segment_reduce(float (&x)[4][2], Op op)
{
    if constexpr (SEG >= 2) {
        float r[4];
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) r[nt] = op(x[nt][0], x[nt][1]);
        if constexpr (SEG == 32) r[0] = op(op(r[0], r[1]), op(r[2], r[3]));
        if constexpr (SEG == 16) {
            r[0] = op(r[0], r[1]);
            r[2] = op(r[2], r[3]);
        }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            if ((SEG == 32 && nt) || (SEG == 16 && (nt & 1))) continue;  // folded into another slot above
            if constexpr (SEG >= 4) r[nt] = op(r[nt], __shfl_xor_sync(0xffffffffu, r[nt], 1));
            if constexpr (SEG >= 8) r[nt] = op(r[nt], __shfl_xor_sync(0xffffffffu, r[nt], 2));
        }
        if constexpr (SEG == 32) r[1] = r[2] = r[3] = r[0];
        if constexpr (SEG == 16) {
            r[1] = r[0];
            r[3] = r[2];
        }
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) x[nt][0] = x[nt][1] = r[nt];
    }
}

// Softmax statistics of one window row over the 32 tokens of a tile, from the eight dot products this lane holds
// for it.  TAIL: the tile reaches into the last W columns, where rows stop seeing tokens and 1/n_vis varies;
// everywhere else every row sees every token of the tile, and the 1/n_vis-weighted sum is the plain sum over W
// (the column kernel applies that factor), so masks and weights drop out.
//   dot[nt][e]  raw q.k of token tile*32 + nt*8 + 2*q4 + e;  j  the row's index among the KV head's rows;
//   valid  false for the zero rows that pad the last m-tile (they take part in the shuffles and store nothing);
//   last_col  (TAIL) the last token the row sees;
//   run  this warp's running (max of q.k, sum of exp relative to it) of the row over the tiles it has seen, or NULL
//        (kept for segments of 16 and 32 tokens, where one lane per row holds a tile's statistics)
template <int SEG, bool TAIL>
__device__ __forceinline__ void row_statistics(const TolArgs &a, const float (&dot)[4][2], int tile, int q4, int j, bool valid,
                                               int last_col, int64_t row0, float2 *run)
{
    constexpr float kLog2e = 1.4426950408889634f;
    const float c1 = a.inv_sqrt_d * kLog2e;                 // logit in units of log 2
    const int t0 = tile * kTileTokens + 2 * q4;             // this lane's first token of the tile
    float v[4][2], mx[4][2];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            v[nt][e] = dot[nt][e];
            if constexpr (TAIL) v[nt][e] = t0 + nt * 8 + e <= last_col ? v[nt][e] : -INFINITY;
            mx[nt][e] = v[nt][e];
        }
    segment_reduce<SEG>(mx, [](float x, float y) { return fmaxf(x, y); });
    float se[4][2], sp[4][2];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            // exp((v - max)/sqrt(d)) as 2^(v*c1 - max*c1): one fused multiply-add and one ex2
            float p = ex2_approx(__fmaf_rn(v[nt][e], c1, -(mx[nt][e] * c1)));
            if constexpr (TAIL) {
                p = v[nt][e] == -INFINITY ? 0.0f : p;       // also the segments no token of which is visible (max = -inf)
                const int n_vis = min(a.W, max(1, a.T - (t0 + nt * 8 + e)));
                sp[nt][e] = p * (1.0f / (float)n_vis);
            }
            se[nt][e] = p;
        }
    segment_reduce<SEG>(se, [](float x, float y) { return x + y; });
    if constexpr (TAIL) segment_reduce<SEG>(sp, [](float x, float y) { return x + y; });
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            if ((SEG >= 2 && e == 1) || (SEG >= 16 && (nt * 8) % SEG != 0)) continue;  // never a segment's first token
            const int t = t0 + nt * 8 + e;
            if (valid && t % SEG == 0 && t < a.T) {           // the segment's first token writes
                // -inf (no visible token: max = -inf, sum = 0) stays -inf
                const int seg = t / SEG;
                a.pl[(int64_t)seg * a.rows + row0 + j] = __fmaf_rn(mx[nt][e], c1, lg2_approx(se[nt][e]));
                if constexpr (TAIL)
                    if (seg >= a.seg_tail0)
                        a.pw[(int64_t)(seg - a.seg_tail0) * a.rows + row0 + j] = __fmaf_rn(mx[nt][e], c1, lg2_approx(sp[nt][e]));
            }
        }
    if constexpr (SEG >= 16) {
        if (run != nullptr && valid && q4 == 0) {
            float2 r = *run;
#pragma unroll
            for (int nt = 0; nt < 4; nt += SEG / 8) {
                if (TAIL && mx[nt][0] == -INFINITY) continue;                  // a segment the row does not see
                const float m_new = fmaxf(r.x, mx[nt][0]);
                r.y = r.y * ex2_approx((r.x - m_new) * c1) + se[nt][0] * ex2_approx((mx[nt][0] - m_new) * c1);
                r.x = m_new;
            }
            *run = r;
        }
    }
}

// MTG: m-tiles (16 flattened window rows each) that share one pass over a tile's B fragments - 2 where a KV head
// has more than 16 rows (grouped-query shapes), else 1.
template <int SEG, int D, int MTG>
__global__ void __launch_bounds__(kTileWarps * 32, 2) logits_mma_kernel(const TolArgs a)
{
    constexpr int kRowBytes = D * 2, kChunks = D / 8, kTileBytes = kTileTokens * kRowBytes;
    constexpr int kQRowBytes = kRowBytes + 16;                               // padded: A fragments read conflict-free
    static_assert(kTileBytes % 1024 == 0 && kRowBytes <= 1024, "tile buffers keep the alignment the swizzle relies on");
    extern __shared__ __align__(256) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int g = lane >> 2, q4 = lane & 3;
    const int n_mt = (a.NR + 15) / 16;                                       // window rows in m-tiles of 16, zero padded
    unsigned char *q_s = smem_raw;                                           // [n_mt*16][kQRowBytes]
    const int q_total = (n_mt * 16 * kQRowBytes + 255) / 256 * 256;
    int *last_col_s = reinterpret_cast<int *>(smem_raw + q_total);           // [n_mt*16]: last token a row sees
    const int lc_total = (n_mt * 16 * 4 + 255) / 256 * 256;
    // [n_mt*16][warps of the CTA]: each warp's running (max of q.k, sum of exp relative to it) of a row over its tiles
    float2 *run_s = reinterpret_cast<float2 *>(smem_raw + q_total + lc_total);
    const int run_total = (n_mt * 16 * (int)(blockDim.x >> 5) * 8 + 255) / 256 * 256;
    // this warp's tile buffers, aligned to a 1 KiB boundary whatever the base of the dynamic shared memory: every bit
    // of a chunk index then sits below the buffer's address bits and a chunk's swizzle is an XOR on the whole address
    const uint32_t tiles_s = (((uint32_t)__cvta_generic_to_shared(smem_raw) + q_total + lc_total + run_total + 1023u) & ~1023u) +
                             wib * kTileBuffers * kTileBytes;

    const int l = blockIdx.y / a.Hkv, kvh = blockIdx.y % a.Hkv;
    const __half *q_src = a.q_win + ((int64_t)(l * a.Hq + kvh * a.rep) * a.W) * D;
    for (int i = threadIdx.x; i < n_mt * 16 * kChunks; i += blockDim.x) {
        const int row = i / kChunks, c = i % kChunks;
        *reinterpret_cast<uint4 *>(q_s + row * kQRowBytes + c * 16) =
            row < a.NR ? __ldg(reinterpret_cast<const uint4 *>(q_src) + i) : make_uint4(0, 0, 0, 0);
    }
    for (int j = threadIdx.x; j < n_mt * 16; j += blockDim.x) last_col_s[j] = j < a.NR ? a.T - a.W + j % a.W : -1;
    for (int i = threadIdx.x; i < n_mt * 16 * (int)(blockDim.x >> 5); i += blockDim.x) run_s[i] = make_float2(-INFINITY, 0.0f);
    __syncthreads();

    const __half *k_plane = a.kv + (int64_t)l * a.stride_l + (int64_t)kvh * a.stride_h;
    const int n_tiles = (a.T + kTileTokens - 1) / kTileTokens;
    // this block's share of the tiles, its warps taking them in turn
    const int per_block = (n_tiles + gridDim.x - 1) / gridDim.x;
    const int tile_begin = blockIdx.x * per_block + wib;
    const int tile_end = min(n_tiles, (int)(blockIdx.x + 1) * per_block);
    const int64_t row0 = (int64_t)(l * a.Hq + kvh * a.rep) * a.W;

    // lane L copies chunk (i*32 + L) of the tile, i = 0 .. kChunks-1: consecutive lanes, consecutive addresses
    auto issue_tile = [&](int tile, int buf) {
        const __half *src = k_plane + (int64_t)tile * kTileTokens * D;
        const int valid_rows = min(kTileTokens, a.T - tile * kTileTokens);
#pragma unroll
        for (int i = 0; i < kChunks; ++i) {
            const int n = i * 32 + lane;
            const int row = n / kChunks, c = n % kChunks;
            const uint32_t dst = tiles_s + buf * kTileBytes + row * kRowBytes + ((c ^ (row & 7)) << 4);
            const bool in = row < valid_rows;
            cp_async16(dst, in ? src + n * 8 : src, in ? 16u : 0u);
        }
        cp_async_commit();
    };

    // B fragments (tokens x channels as the "column" operand): one ldmatrix x4 covers 16 tokens and 16 channels.
    // Lane L addresses token (L/16)*8 + L%8 of the 16 at channel chunk 2*ks + (L/8)%2; its row's swizzle (token & 7
    // = L & 7) and the chunk's low bit fold into a per-lane base, the rest of the chunk index is an XOR of ks << 5.
    const uint32_t b_lane = (uint32_t)((((lane >> 4) << 3) + (lane & 7)) * kRowBytes + ((((lane >> 3) & 1) ^ (lane & 7)) << 4));
    // A fragments (window rows x channels): lanes 0-15 give rows 0-15 at chunk 2*ks, lanes 16-31 at chunk 2*ks + 1
    const uint32_t a_lane = (uint32_t)__cvta_generic_to_shared(q_s) + (lane & 15) * kQRowBytes + ((lane >> 4) << 4);

    int buf = 0;
    if (kTileBuffers == 2 && tile_begin < tile_end) issue_tile(tile_begin, 0);
    const int cta_warps = blockDim.x >> 5;
    for (int tile = tile_begin; tile < tile_end; tile += cta_warps, buf ^= (kTileBuffers - 1)) {
        if (kTileBuffers == 1) {
            issue_tile(tile, 0);
            cp_async_wait<0>();
        } else if (tile + cta_warps < tile_end) {
            issue_tile(tile + cta_warps, buf ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncwarp();
        const uint32_t tile_s = tiles_s + buf * kTileBytes + b_lane;
        const bool tail_tile = tile * kTileTokens + kTileTokens > a.T - a.W + 1;
        for (int mt0 = 0; mt0 < n_mt; mt0 += MTG) {
            float acc[MTG][4][4];
#pragma unroll
            for (int m = 0; m < MTG; ++m)
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[m][nt][i] = 0.0f;
            const bool second = MTG == 2 && mt0 + 1 < n_mt;
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                uint32_t bf[2][4];      // [tokens 0-15 | 16-31]: b0, b1 of the even n-tile, b0, b1 of the odd one
                ldmatrix_x4((tile_s) ^ (ks << 5), bf[0]);
                ldmatrix_x4((tile_s + 16 * kRowBytes) ^ (ks << 5), bf[1]);
#pragma unroll
                for (int m = 0; m < MTG; ++m) {
                    if (m == 1 && !second) break;
                    uint32_t af[4];
                    ldmatrix_x4(a_lane + (mt0 + m) * 16 * kQRowBytes + ks * 32, af);
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) mma_16816(acc[m][nt], af, bf[nt >> 1][(nt & 1) * 2], bf[nt >> 1][(nt & 1) * 2 + 1]);
                }
            }
            // acc[m][nt][0..1]: window row (mt0+m)*16 + g, tokens nt*8 + 2*q4, + 1;  [2..3]: row + 8, the same tokens
#pragma unroll
            for (int m = 0; m < MTG; ++m) {
                if (m == 1 && !second) break;
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int j0 = (mt0 + m) * 16 + half * 8;
                    if (j0 >= a.NR) break;                     // only zero padding from here on (the same for every lane)
                    const int j = j0 + g;
                    float dot[4][2];
#pragma unroll
                    for (int nt = 0; nt < 4; ++nt) {
                        dot[nt][0] = acc[m][nt][2 * half];
                        dot[nt][1] = acc[m][nt][2 * half + 1];
                    }
                    float2 *run = a.n_slots > 0 ? run_s + j * cta_warps + wib : nullptr;
                    if (tail_tile) row_statistics<SEG, true>(a, dot, tile, q4, j, j < a.NR, last_col_s[j], row0, run);
                    else row_statistics<SEG, false>(a, dot, tile, q4, j, j < a.NR, 0, row0, run);
                }
            }
        }
        __syncwarp();  // the buffer is free for the copy issued two tiles from now
    }

    grid_launch_dependents();   // the kernel behind this one may be set up now (it waits for this one to complete)
    // ---- what the column kernel that follows needs from this CTA
    if (blockIdx.x == 0 && blockIdx.y == 0)
        for (int i = threadIdx.x; i <= a.n_x; i += blockDim.x) a.tickets[i] = 0;
    // Every row's (max, sum of exp) over this CTA's tiles: the warps' running pairs, combined in warp order.  The
    // column kernel combines a row's n_slots such pairs into the row's softmax denominator.
    __syncthreads();
    if (a.n_slots > 0) {
        constexpr float kLog2e = 1.4426950408889634f;
        const float c1 = a.inv_sqrt_d * kLog2e;
        for (int j = threadIdx.x; j < a.NR; j += blockDim.x) {
            float m_all = -INFINITY;
            for (int k = 0; k < cta_warps; ++k) m_all = fmaxf(m_all, run_s[j * cta_warps + k].x);
            float s_all = 0.0f;
            for (int k = 0; k < cta_warps; ++k) {
                const float2 c = run_s[j * cta_warps + k];
                if (c.x != -INFINITY) s_all += c.y * ex2_approx((c.x - m_all) * c1);
            }
            a.row_part[(row0 + j) * a.n_slots + blockIdx.x] = make_float2(m_all * c1, s_all);
        }
    }
}

// Which CTA of the tcgen05 kernel has tile x of the sequence of all `total` tiles in its run (CTA c has the tiles
// from total * c / grid up to, not including, total * (c + 1) / grid).
__host__ __device__ inline int tc_cta_of_tile(int64_t x, int64_t total, int grid)
{
    return (int)(((x + 1) * grid - 1) / total);
}

}  // namespace llms

#include "tolerance_tc.cuh"

namespace llms {

// block = 32 neighbouring rows x 32 segment lanes: log2 of every row's softmax denominator from its segment values.
// A warp reads 32 neighbouring rows of one segment (128 consecutive bytes); four segments per trip are in flight.
__global__ void __launch_bounds__(1024) row_stats_kernel(const TolArgs a)
{
    __shared__ float red[32][33];
    grid_dependency_wait();
    const int row = blockIdx.x * 32 + threadIdx.x;
    const bool in = row < a.rows;
    const float *pl = a.pl + row;
    float m = -INFINITY;
    if (in) {
        int s = threadIdx.y;
        for (; s + 96 < a.n_seg; s += 128) {
            float v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = pl[(int64_t)(s + 32 * u) * a.rows];
            m = fmaxf(fmaxf(m, fmaxf(v[0], v[1])), fmaxf(v[2], v[3]));
        }
        for (; s < a.n_seg; s += 32) m = fmaxf(m, pl[(int64_t)s * a.rows]);
    }
    red[threadIdx.y][threadIdx.x] = m;
    __syncthreads();
#pragma unroll
    for (int y = 0; y < 32; ++y) m = fmaxf(m, red[y][threadIdx.x]);
    __syncthreads();
    float sum = 0.0f;
    if (in) {
        int s = threadIdx.y;
        for (; s + 96 < a.n_seg; s += 128) {   // the terms of a lane are added in segment order
            float v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = pl[(int64_t)(s + 32 * u) * a.rows];
#pragma unroll
            for (int u = 0; u < 4; ++u) sum += exp2f(v[u] - m);   // -inf (a segment the row does not see) adds 0
        }
        for (; s < a.n_seg; s += 32) sum += exp2f(pl[(int64_t)s * a.rows] - m);
    }
    red[threadIdx.y][threadIdx.x] = sum;
    grid_launch_dependents();
    __syncthreads();
    if (threadIdx.y == 0 && in) {
        float total = 0.0f;
#pragma unroll
        for (int y = 0; y < 32; ++y) total += red[y][threadIdx.x];
        a.row_lse[row] = m + log2f(total);
    }
}

// log2 of a row's softmax denominator from its n <= 32 (max, sum) pairs, by a whole warp: lane k takes pair k, the
// lanes are combined in a fixed tree.  Every lane returns the result.
__device__ __forceinline__ float row_lse_from_pair(float2 c)   // c: this lane's pair, (-inf, 0) if it has none
{
    float m = c.x;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    float sum = c.x != -INFINITY ? c.y * exp2f(c.x - m) : 0.0f;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
    return m + log2f(sum);
}
__device__ __forceinline__ float row_lse_from_slots(const float2 *rp, int n, int lane)
{
    return row_lse_from_pair(lane < n ? rp[lane] : make_float2(-INFINITY, 0.0f));
}
static_assert(kMaxRowSlots <= 32, "a lane per slot");

// The tcgen05 kernel leaves, per row, one (max, sum) pair for every statistics thread of every CTA that had tiles of
// the row's (layer, KV head) pair: a warp per row adds them up.
__global__ void __launch_bounds__(256) row_combine_kernel(const TolArgs a)
{
    grid_dependency_wait();
    grid_launch_dependents();
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= a.rows) return;
    const int tiles_per_pair = ((a.T + 127) / 128 + 1) / 2;      // the tcgen05 kernel's double tiles
    const int64_t total = (int64_t)a.L * a.Hkv * tiles_per_pair;
    const int64_t first = (int64_t)(row / a.NR) * tiles_per_pair;
    const int n = (tc_cta_of_tile(first + tiles_per_pair - 1, total, a.tc_grid) - tc_cta_of_tile(first, total, a.tc_grid) + 1) * a.tc_spr;
    const float lse = row_lse_from_slots(a.row_part + (int64_t)row * a.n_slots, n, lane);
    if (lane == 0) a.row_lse[row] = lse;
}

// True in every thread of exactly one of the `expected` blocks that pass through with this counter: the one that comes
// last.  What the others wrote to global memory before is then visible to loads that bypass L1.  Nobody waits.
__device__ __forceinline__ bool arrives_last(uint32_t *counter, uint32_t expected)
{
    __shared__ uint32_t ticket;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0 && threadIdx.y == 0) ticket = atomicAdd(counter, 1u);
    __syncthreads();
    const bool last = ticket == expected - 1;
    if (last) __threadfence();
    return last;
}

constexpr int kMaxSliceRows = 1024;   // rows of one slice of the column kernel (their denominators sit in shared memory)

// Column sums, then chunk means, in one launch.  Block (32 row lanes x 8 segment lanes) over 32 segments; blockIdx.y
// picks a slice of rows.
// A block first makes its rows' softmax denominators (from the per-CTA pairs the MMA kernel left, or copies them
// where a kernel of its own made them), then adds up its rows' normalised, 1/n_vis-weighted probabilities per segment.
// The last slice to finish a group of 32 segments adds the slices in index order; the last group to finish adds
// every chunk's segments.  All sums run in a fixed order: the scores do not depend on which block came last.
__global__ void __launch_bounds__(256) column_chunk_kernel(const TolArgs a)
{
    __shared__ float red[8][33];
    __shared__ float rl_s[kMaxSliceRows];
    grid_dependency_wait();
    const int tid = threadIdx.y * 32 + threadIdx.x;
    const int seg = blockIdx.x * 32 + threadIdx.x;
    const int rows_per_slice = (a.rows + a.Y - 1) / a.Y;
    const int r_begin = blockIdx.y * rows_per_slice;
    const int r_end = min(a.rows, r_begin + rows_per_slice);
    if (a.lse_ready) {
        for (int r = r_begin + tid; r < r_end; r += 256) rl_s[r - r_begin] = a.row_lse[r];
    } else {   // a warp per row, a lane per pair; eight rows per trip so that their loads are in flight together
        for (int r0 = r_begin + threadIdx.y; r0 < r_end; r0 += 64) {
            float2 c[8];
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                const int r = r0 + 8 * v;
                c[v] = r < r_end && threadIdx.x < a.n_slots ? a.row_part[(int64_t)r * a.n_slots + threadIdx.x] : make_float2(-INFINITY, 0.0f);
            }
#pragma unroll
            for (int v = 0; v < 8; ++v) {
                const float lse = row_lse_from_pair(c[v]);
                if (threadIdx.x == 0 && r0 + 8 * v < r_end) rl_s[r0 + 8 * v - r_begin] = lse;
            }
        }
    }
    __syncthreads();
    // Row lane x takes rows r_begin + x, + 32, ...; segment lane y takes the block's segments y, y + 8, y + 16, y + 24.
    // A segment's probability mass in a row is 2^(its value - the row's log2 denominator).  Before the last W columns
    // every row sees every token: the column weight 1/W is applied to the finished sum.  Four rows per trip: sixteen
    // loads in flight per thread (with four the kernel waited on one round trip to memory after another).
    float acc4[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int row0 = r_begin + threadIdx.x; row0 < r_end; row0 += 128) {
        float rl[4], ls[4][4];
#pragma unroll
        for (int v = 0; v < 4; ++v) {
            const int row = row0 + 32 * v;
            const bool in = row < r_end;
            rl[v] = in ? rl_s[row - r_begin] : 0.0f;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int sg = blockIdx.x * 32 + u * 8 + threadIdx.y;
                if (!in || sg >= a.n_seg) ls[v][u] = -INFINITY;
                else if (sg >= a.seg_tail0) ls[v][u] = a.pw[(int64_t)(sg - a.seg_tail0) * a.rows + row];
                else ls[v][u] = a.pl[(int64_t)sg * a.rows + row];
            }
        }
#pragma unroll
        for (int v = 0; v < 4; ++v)
#pragma unroll
            for (int u = 0; u < 4; ++u) acc4[u] += exp2f(ls[v][u] - rl[v]);   // rows in rising order; -inf adds 0
    }
    // the 32 row lanes of a segment, added in a fixed tree
#pragma unroll
    for (int u = 0; u < 4; ++u) {
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) acc4[u] += __shfl_xor_sync(0xffffffffu, acc4[u], d);
        const int sg = blockIdx.x * 32 + u * 8 + threadIdx.y;
        if (threadIdx.x == 0 && sg < a.n_seg)
            a.part[(int64_t)blockIdx.y * a.n_seg + sg] = sg >= a.seg_tail0 ? acc4[u] : acc4[u] * (1.0f / (float)a.W);
    }
    float acc = 0.0f;
    grid_launch_dependents();
    if (!arrives_last(a.tickets + blockIdx.x, gridDim.y)) return;

    // ---- this group's column sums: row lane y adds slices y, y + 8, ... in order, then the eight lanes are added in order
    acc = 0.0f;
    if (seg < a.n_seg) {
        for (int y0 = threadIdx.y; y0 < a.Y; y0 += 64) {   // eight loads in flight, added in slice order
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = y0 + 8 * k < a.Y ? __ldcg(a.part + (int64_t)(y0 + 8 * k) * a.n_seg + seg) : 0.0f;
#pragma unroll
            for (int k = 0; k < 8; ++k) acc += v[k];
        }
    }
    __syncthreads();
    red[threadIdx.y][threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.y == 0 && seg < a.n_seg) {
        float s = 0.0f;
#pragma unroll
        for (int y = 0; y < 8; ++y) s += red[y][threadIdx.x];
        a.colsum[seg] = s;
    }
    if (!arrives_last(a.tickets + a.n_x, gridDim.x)) return;

    // ---- every chunk's mean over its tokens, layers and heads
    const float norm = (float)a.CL * (float)a.L * (float)a.Hq;
    const bool gave_up = *reinterpret_cast<volatile uint32_t *>(a.status) == kTcGaveUp;   // the logits kernel did not finish
    __syncthreads();
    if (tid == 0 && gave_up) *a.status = 0;
    for (int c = tid; c < a.n_chunks; c += 256) {
        float tot = 0.0f;
        for (int sg = c * a.seg_per_chunk; sg < (c + 1) * a.seg_per_chunk; ++sg) tot += __ldcg(a.colsum + sg);
        const float score = gave_up ? __int_as_float(0x7fc00000) : tot / norm;
        a.scores[c] = score;
        if (a.scores_live) a.scores_live[c] = score;
    }
}

// ------------------------------------------------------------------ probabilities -> scores

struct ProbArgs {
    const float *probs;
    int LH, W, T, CL, n_chunks, chunks_per_block;
    float *part;   // [LH][n_chunks]
    float *scores;
    float inv_norm;
};

// block = (a run of whole chunks) x (one layer-head); thread per column, then one thread per chunk
__global__ void __launch_bounds__(256) probs_column_kernel(const ProbArgs a)
{
    extern __shared__ float tok_s[];
    const int lh = blockIdx.y;
    const int c0 = blockIdx.x * a.chunks_per_block;
    const int nc = min(a.chunks_per_block, a.n_chunks - c0);
    const int col0 = c0 * a.CL, ncol = nc * a.CL;
    const float *P = a.probs + (int64_t)lh * a.W * a.T;
    for (int i = threadIdx.x; i < ncol; i += blockDim.x) {
        const int col = col0 + i;
        const int n_vis = min(a.W, a.T - col);
        float s = 0.0f;
        for (int r = a.W - n_vis; r < a.W; ++r) s += __ldg(P + (int64_t)r * a.T + col);  // rows at position >= col
        tok_s[i] = s / (float)n_vis;
    }
    __syncthreads();
    for (int c = threadIdx.x; c < nc; c += blockDim.x) {
        float s = 0.0f;
        for (int i = 0; i < a.CL; ++i) s += tok_s[c * a.CL + i];
        a.part[(int64_t)lh * a.n_chunks + c0 + c] = s;
    }
}

__global__ void probs_final_kernel(const ProbArgs a)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= a.n_chunks) return;
    float s = 0.0f;
    for (int lh = 0; lh < a.LH; ++lh) s += a.part[(int64_t)lh * a.n_chunks + c];
    a.scores[c] = s * a.inv_norm;
}

static int seg_len(int chunk_len)
{
    int s = 1;
    while (s < 32 && chunk_len % (s * 2) == 0) s *= 2;
    return s;
}

// slices of rows in the column kernel: enough blocks to fill the GPU - with many rows about 512 blocks over the n_x
// groups of 32 segments (measured: 64 slices at 8 groups, 16 at 32 groups; 8 or 128 slices cost 3-10% of the stage) -
// and no slice longer than the kernel's arrays
static int row_slices(int rows, int n_x)
{
    const int y = rows >= 4096 ? std::min(64, std::max(16, 512 / std::max(1, n_x))) : (rows >= 512 ? 16 : (rows >= 64 ? 4 : 1));
    return std::max(y, (rows + kMaxSliceRows - 1) / kMaxSliceRows);
}


struct TolLayout {
    int SEG, n_seg, seg_tail0, rows, Y, n_x;
    uint64_t off_pl, off_pw, off_rlse, off_part, off_rpart, off_colsum, off_tickets, total;
};

static TolLayout tol_layout(const llms_kv_desc &d, int W)
{
    TolLayout t;
    t.SEG = seg_len(d.chunk_len);
    t.n_seg = (d.n_tokens + t.SEG - 1) / t.SEG;
    t.seg_tail0 = std::min(t.n_seg, (d.n_tokens - W + 1) / t.SEG);
    t.rows = d.n_layers * d.n_q_heads * W;
    t.n_x = (t.n_seg + 31) / 32;
    t.Y = row_slices(t.rows, t.n_x);
    t.off_pl = 0;
    t.off_pw = round_up((uint64_t)t.rows * t.n_seg * 4, 256);
    t.off_rlse = t.off_pw + round_up((uint64_t)t.rows * (t.n_seg - t.seg_tail0) * 4, 256);
    t.off_part = t.off_rlse + round_up((uint64_t)t.rows * 4, 256);
    t.off_rpart = t.off_part + round_up((uint64_t)t.Y * t.n_seg * 4, 256);
    t.off_colsum = t.off_rpart + round_up((uint64_t)t.rows * kMaxRowSlots * sizeof(float2), 256);
    t.off_tickets = t.off_colsum + round_up((uint64_t)t.n_seg * 4, 256);
    t.total = t.off_tickets + round_up((uint64_t)(t.n_x + 2) * 4, 256);   // tickets, then the status word
    return t;
}

// ---- launching the tcgen05 kernel

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn tensor_map_encoder()
{
    static EncodeTiledFn fn = [] {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult found;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &found) != cudaSuccess ||
            found != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

static int tc_rows(const TolArgs &a)
{
    int r = 8;
    while (r < a.NR) r *= 2;
    return r;
}

// The tcgen05 kernel takes head_dim 64 or 128, up to 128 rows per KV head and segments of 16 or 32 tokens (chunk_len a
// multiple of 16).  It is used from 32 rows per KV head on (grouped-query shapes), where it is the faster one.
static bool tc_path_ok(const TolArgs &a, int SEG)
{
    return (a.d == 64 || a.d == 128) && a.NR >= 32 && a.NR <= 128 && SEG >= 16 && tensor_map_encoder() != nullptr;
}

template <int SEG, int D, int R>
static int launch_logits_tc_inst(const TolArgs &a, const CUtensorMap &map_k, const CUtensorMap &map_q, cudaStream_t st)
{
    const size_t operand = (size_t)(D / 64) * kTcBlockBytes, stage = (size_t)(D / 64) * kTcWideBlockBytes;
    const int n_stages = (int)std::min<size_t>(8, (227 * 1024 - 2 * operand - sizeof(TcBarriers) - 1024) / stage);
    const size_t smem = 1024 + 2 * operand + (size_t)n_stages * stage + sizeof(TcBarriers);
    LLMS_CUDA_TRY(cudaFuncSetAttribute(logits_tc_kernel<SEG, D, R>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    logits_tc_kernel<SEG, D, R><<<a.tc_grid, kTcThreads, smem, st>>>(a, map_k, map_q, n_stages);
    return LLMS_OK;
}

template <int SEG, int D>
static int launch_logits_tc_rows(const TolArgs &a, int R, const CUtensorMap &map_k, const CUtensorMap &map_q, cudaStream_t st)
{
    switch (R) {
    case 8: return launch_logits_tc_inst<SEG, D, 8>(a, map_k, map_q, st);
    case 16: return launch_logits_tc_inst<SEG, D, 16>(a, map_k, map_q, st);
    case 32: return launch_logits_tc_inst<SEG, D, 32>(a, map_k, map_q, st);
    case 64: return launch_logits_tc_inst<SEG, D, 64>(a, map_k, map_q, st);
    case 128: return launch_logits_tc_inst<SEG, D, 128>(a, map_k, map_q, st);
    default: return LLMS_ERR_UNSUPPORTED;
    }
}

static int launch_logits_tc(const TolArgs &a, int SEG, cudaStream_t st)
{
    EncodeTiledFn encode = tensor_map_encoder();
    if (!encode) return LLMS_ERR_UNSUPPORTED;
    const int R = tc_rows(a);
    // K as a 4-D tensor (channel, token, KV head, layer), tiles of 64 channels x 128 tokens, 128-byte swizzle; tokens past
    // the end of the context read as zeros
    CUtensorMap map_k, map_q;
    {
        const cuuint64_t dims[4] = {(cuuint64_t)a.d, (cuuint64_t)a.T, (cuuint64_t)a.Hkv, (cuuint64_t)a.L};
        const cuuint64_t strides[3] = {(cuuint64_t)a.d * 2, (cuuint64_t)a.stride_h * 2, (cuuint64_t)a.stride_l * 2};
        const cuuint32_t box[4] = {64, (cuuint32_t)kTcWide, 1, 1}, elem[4] = {1, 1, 1, 1};
        if (encode(&map_k, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, const_cast<__half *>(a.kv), dims, strides, box, elem,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LLMS_ERR_UNSUPPORTED;
    }
    {   // the query window as a matrix of (layer, head, row) x channel, R rows at a time
        const cuuint64_t dims[2] = {(cuuint64_t)a.d, (cuuint64_t)a.L * a.Hq * a.W};
        const cuuint64_t strides[1] = {(cuuint64_t)a.d * 2};
        const cuuint32_t box[2] = {64, (cuuint32_t)R}, elem[2] = {1, 1};
        if (encode(&map_q, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<__half *>(a.q_win), dims, strides, box, elem,
                   CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                   CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return LLMS_ERR_UNSUPPORTED;
    }
    if (SEG == 16) return a.d == 64 ? launch_logits_tc_rows<16, 64>(a, R, map_k, map_q, st) : launch_logits_tc_rows<16, 128>(a, R, map_k, map_q, st);
    if (SEG == 32) return a.d == 64 ? launch_logits_tc_rows<32, 64>(a, R, map_k, map_q, st) : launch_logits_tc_rows<32, 128>(a, R, map_k, map_q, st);
    return LLMS_ERR_UNSUPPORTED;
}

static int check_tol(const llms_kv_desc *desc, int W)
{
    int rc = check_desc(desc);
    if (rc) return rc;
    if (W <= 0 || W > desc->n_tokens) return LLMS_ERR_INVALID_ARG;
    if ((int64_t)desc->n_layers * desc->n_q_heads * W > 0x7fffffff / 4) return LLMS_ERR_UNSUPPORTED;
    return LLMS_OK;
}

}  // namespace llms

using namespace llms;

extern "C" int llms_tolerance_workspace_bytes(const llms_kv_desc *desc, int W, uint64_t *nbytes)
{
    int rc = check_tol(desc, W);
    if (rc) return rc;
    if (!nbytes) return LLMS_ERR_INVALID_ARG;
    const uint64_t from_q = tol_layout(*desc, W).total;
    const uint64_t from_p = round_up((uint64_t)desc->n_layers * desc->n_q_heads * (uint64_t)n_chunks(*desc) * 4, 256);
    *nbytes = from_q > from_p ? from_q : from_p;
    return LLMS_OK;
}

extern "C" int llms_chunk_tolerance(const llms_kv_desc *desc, const void *kv, const void *q_win, int W,
                                    float *scores, void *workspace, uint64_t workspace_bytes, void *stream)
{
    return llms::chunk_tolerance_impl(desc, kv, q_win, W, scores, nullptr, workspace, workspace_bytes, stream);
}

int llms::chunk_tolerance_impl(const llms_kv_desc *desc, const void *kv, const void *q_win, int W, float *scores,
                               float *scores_live, void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_tol(desc, W);
    if (rc) return rc;
    if (!kv || !q_win || !scores || !workspace) return LLMS_ERR_INVALID_ARG;
    if (desc->head_dim % 8 || (desc->stride_l | desc->stride_h) % 8) return LLMS_ERR_MISALIGNED;
    if (!aligned(kv, 16) || !aligned(q_win, 16) || !aligned(workspace, 256) || !aligned(scores, 4)) return LLMS_ERR_MISALIGNED;
    if (n_chunks(*desc) == 0) return LLMS_OK;
    const TolLayout t = tol_layout(*desc, W);
    if (workspace_bytes < t.total) return LLMS_ERR_BUF_TOO_SMALL;
    TolArgs a{};
    a.kv = static_cast<const __half *>(kv);
    a.q_win = static_cast<const __half *>(q_win);
    a.L = desc->n_layers; a.Hkv = desc->n_kv_heads; a.Hq = desc->n_q_heads; a.d = desc->head_dim;
    a.T = desc->n_tokens; a.W = W; a.CL = desc->chunk_len;
    a.rep = a.Hq / a.Hkv;
    a.NR = a.rep * W;
    a.n_seg = t.n_seg;
    a.seg_tail0 = t.seg_tail0;
    a.seg_per_chunk = a.CL / t.SEG;
    a.n_chunks = n_chunks(*desc);
    a.stride_l = desc->stride_l; a.stride_h = desc->stride_h;
    a.inv_sqrt_d = (float)(1.0 / sqrt((double)a.d));
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    a.pl = reinterpret_cast<float *>(ws + t.off_pl);
    a.pw = reinterpret_cast<float *>(ws + t.off_pw);
    a.row_lse = reinterpret_cast<float *>(ws + t.off_rlse);
    a.part = reinterpret_cast<float *>(ws + t.off_part);
    a.row_part = reinterpret_cast<float2 *>(ws + t.off_rpart);
    a.colsum = reinterpret_cast<float *>(ws + t.off_colsum);
    a.tickets = reinterpret_cast<uint32_t *>(ws + t.off_tickets);
    a.n_x = t.n_x;
    a.status = a.tickets + t.n_x + 1;
    a.scores = scores;
    a.scores_live = scores_live;
    a.Y = t.Y; a.rows = t.rows;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((unsigned)(a.L * a.Hkv) > 65535u || a.Y > 65535) return LLMS_ERR_UNSUPPORTED;
    if (tc_path_ok(a, t.SEG)) {
        // one CTA per SM, each with an equal run of the sequence of all 128-token tiles.  Every statistics thread
        // keeps the partial sums of its row while it runs, if a row's slots - threads per row x the most CTAs that
        // share a (layer, KV head) pair - fit; else a pass over the statistics follows.
        const int tiles_per_pair = ((a.T + kTcTile - 1) / kTcTile + 1) / 2;      // double tiles: what an MMA takes
        const int64_t total = (int64_t)a.L * a.Hkv * tiles_per_pair;
        a.tc_grid = (int)std::min<int64_t>(total, sm_count());
        a.tc_spr = kTcAcc * (kTcTile / tc_rows(a));
        int most_ctas = 1;
        for (int64_t pair = 0; pair < (int64_t)a.L * a.Hkv; ++pair)
            most_ctas = std::max(most_ctas, tc_cta_of_tile((pair + 1) * tiles_per_pair - 1, total, a.tc_grid) -
                                                tc_cta_of_tile(pair * tiles_per_pair, total, a.tc_grid) + 1);
        a.n_slots = a.tc_spr * most_ctas <= kMaxRowSlots ? a.tc_spr * most_ctas : 0;
        rc = launch_logits_tc(a, t.SEG, st);
        if (rc) return rc;
        goto tail;
    }
    {
    const size_t padded_rows = (size_t)(a.NR + 15) / 16 * 16;                            // whole m-tiles
    const size_t mma_q_bytes = (padded_rows * (a.d * 2 + 16) + 255) / 256 * 256 +
                               (padded_rows * 4 + 255) / 256 * 256 +                     // query rows, each row's last visible
                               (padded_rows * kTileWarps * 8 + 255) / 256 * 256 + 1024;  // token, the warps' running row sums,
                                                                                         // room to align the tiles
    const size_t tile_bytes = (size_t)kTileBuffers * kTileTokens * a.d * 2;
    // twelve warps per CTA when two such CTAs fit into an SM's shared memory, else eight
    const int cta_warps = 2 * (mma_q_bytes + kTileWarps * tile_bytes + 1024) <= 227 * 1024 ? kTileWarps : kTileWarpsSmall;
    const size_t mma_smem = mma_q_bytes + (size_t)cta_warps * tile_bytes;
    if ((a.d == 64 || a.d == 128 || a.d == 256) && mma_smem <= 200 * 1024) {
        // enough blocks per (layer, KV head) to fill the GPU a few times over - many times over where a block then still
        // has two tiles per warp: the blocks are handed out as earlier ones leave, and the shorter they are the less the
        // last ones leave idle (7B shape, 1024 pairs of 128 tiles: 1 / 2 / 3 / 4 / 6 blocks per pair 193.6 / 193.4 /
        // 191.5 / 191.5 / 195.6 us for the stage; 1024 pairs of 32 tiles: 1 / 3 blocks 72.7 / 75.2 us)
        const int n_tiles = (a.T + kTileTokens - 1) / kTileTokens;
        const int pairs = a.L * a.Hkv;
        int splits = (sm_count() * 6 + pairs - 1) / pairs;
        const int more = (sm_count() * 18 + pairs - 1) / pairs;
        if (n_tiles / more >= 2 * cta_warps) splits = more;
        splits = std::max(1, std::min({splits, (n_tiles + cta_warps - 1) / cta_warps, kMaxRowSlots}));
        // With up to 16 rows per KV head and segments of 16 or 32 tokens every CTA leaves its rows' (max, sum of exp)
        // for the column kernel (7B shape: 2 us more in this kernel, 6 us of row_stats_kernel and a launch less).
        // Elsewhere the denominators come from a pass of row_stats_kernel over all statistics: with 32 rows per KV
        // head the running sums made this kernel 24 us slower (32K grouped-query shape), more than that pass costs.
        a.n_slots = t.SEG >= 16 && a.NR <= 16 ? splits : 0;
        const dim3 grid(splits, pairs);
#define LLMS_LAUNCH_MMA_G(S, DD, G)                                                                                                  \
    do {                                                                                                                             \
        LLMS_CUDA_TRY(cudaFuncSetAttribute(logits_mma_kernel<S, DD, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mma_smem)); \
        logits_mma_kernel<S, DD, G><<<grid, cta_warps * 32, mma_smem, st>>>(a);                                                     \
    } while (0)
#define LLMS_LAUNCH_MMA(S, DD)                        \
    do {                                              \
        if (a.NR > 16) LLMS_LAUNCH_MMA_G(S, DD, 2);   \
        else LLMS_LAUNCH_MMA_G(S, DD, 1);             \
    } while (0)
#define LLMS_LAUNCH_MMA_SEG(S)                                                      \
    case S:                                                                         \
        if (a.d == 64) LLMS_LAUNCH_MMA(S, 64);                                      \
        else if (a.d == 128) LLMS_LAUNCH_MMA(S, 128);                               \
        else LLMS_LAUNCH_MMA(S, 256);                                               \
        break;
        switch (t.SEG) {
            LLMS_LAUNCH_MMA_SEG(1)
            LLMS_LAUNCH_MMA_SEG(2)
            LLMS_LAUNCH_MMA_SEG(4)
            LLMS_LAUNCH_MMA_SEG(8)
            LLMS_LAUNCH_MMA_SEG(16)
            LLMS_LAUNCH_MMA_SEG(32)
        default: return LLMS_ERR_UNSUPPORTED;
        }
#undef LLMS_LAUNCH_MMA_SEG
#undef LLMS_LAUNCH_MMA
#undef LLMS_LAUNCH_MMA_G
    } else {
        const size_t q_bytes = (size_t)a.NR * a.d * sizeof(float);
        if (q_bytes > 200 * 1024) return LLMS_ERR_UNSUPPORTED;
        const dim3 grid((a.T + kTokThreads - 1) / kTokThreads, a.L * a.Hkv);
#define LLMS_LAUNCH_LOGITS(S)                                                                                   \
    case S:                                                                                                     \
        LLMS_CUDA_TRY(cudaFuncSetAttribute(logits_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)q_bytes)); \
        logits_kernel<S><<<grid, kTokThreads, q_bytes, st>>>(a);                                                \
        break;
        switch (t.SEG) {
            LLMS_LAUNCH_LOGITS(1)
            LLMS_LAUNCH_LOGITS(2)
            LLMS_LAUNCH_LOGITS(4)
            LLMS_LAUNCH_LOGITS(8)
            LLMS_LAUNCH_LOGITS(16)
            LLMS_LAUNCH_LOGITS(32)
        default: return LLMS_ERR_UNSUPPORTED;
        }
#undef LLMS_LAUNCH_LOGITS
    }
    }
tail:
    LLMS_CUDA_TRY(cudaGetLastError());
    if (a.n_slots == 0) {  // no partial row sums were left: a pass over all statistics makes the denominators
        LLMS_CUDA_TRY(launch_dependent(row_stats_kernel, dim3((a.rows + 31) / 32), dim3(32, 32), 0, st, a));
        a.lse_ready = 1;
    } else if (a.tc_grid > 0) {  // one pair per statistics thread and CTA: added up per row first
        LLMS_CUDA_TRY(launch_dependent(row_combine_kernel, dim3((a.rows + 7) / 8), dim3(256), 0, st, a));
        a.lse_ready = 1;
    }
    LLMS_CUDA_TRY(launch_dependent(column_chunk_kernel, dim3(a.n_x, a.Y), dim3(32, 8), 0, st, a));
    return LLMS_OK;
}

extern "C" int llms_chunk_tolerance_from_probs(const llms_kv_desc *desc, const float *probs, int W,
                                               float *scores, void *workspace, uint64_t workspace_bytes, void *stream)
{
    int rc = check_tol(desc, W);
    if (rc) return rc;
    if (!probs || !scores || !workspace) return LLMS_ERR_INVALID_ARG;
    if (!aligned(probs, 4) || !aligned(scores, 4) || !aligned(workspace, 4)) return LLMS_ERR_MISALIGNED;
    ProbArgs a{};
    a.probs = probs;
    a.LH = desc->n_layers * desc->n_q_heads;
    a.W = W; a.T = desc->n_tokens; a.CL = desc->chunk_len;
    a.n_chunks = n_chunks(*desc);
    if (a.n_chunks == 0) return LLMS_OK;
    if (workspace_bytes < (uint64_t)a.LH * a.n_chunks * 4) return LLMS_ERR_BUF_TOO_SMALL;
    if (a.CL > 8192 || a.LH > 65535) return LLMS_ERR_UNSUPPORTED;
    a.chunks_per_block = a.CL >= 256 ? 1 : 256 / a.CL;
    a.part = static_cast<float *>(workspace);
    a.scores = scores;
    a.inv_norm = 1.0f / ((float)a.CL * (float)desc->n_layers * (float)desc->n_q_heads);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const dim3 grid((a.n_chunks + a.chunks_per_block - 1) / a.chunks_per_block, a.LH);
    const size_t smem = (size_t)a.chunks_per_block * a.CL * sizeof(float);
    probs_column_kernel<<<grid, 256, smem, st>>>(a);
    LLMS_CUDA_TRY(cudaGetLastError());
    probs_final_kernel<<<(a.n_chunks + 127) / 128, 128, 0, st>>>(a);
    LLMS_CUDA_TRY(cudaGetLastError());
    return LLMS_OK;
}
