// Tolerance score (information density, Eq. 1) kernels for sm_100a.
//
// From probabilities: a column-mean reduction, one pass over the window.
// From K and the last W queries: K is streamed once.  A thread owns one token (one column of the attention
// window), dots its key with every query row of the KV head, and the rows' softmax statistics are kept per
// *segment* of SEG neighbouring tokens (SEG = the largest power of two <= 32 that divides chunk_len), as
// (segment max, sum of exp, 1/n_vis-weighted sum of exp).  Three small kernels then turn the per-segment
// statistics into row normalisers, column means and chunk means.  All sums run in a fixed order, so the
// scores - and the ranking made from them - are reproducible bit for bit.
#include <math.h>

#include <algorithm>

#include "llms_internal.cuh"

namespace llms {

constexpr int kTokThreads = 256;   // tokens per block in the logits kernel
constexpr int kRowTile = 8;        // query rows per pass over a key

struct TolArgs {
    const __half *kv;
    const __half *q_win;
    int L, Hkv, Hq, d, T, W, CL;
    int rep;          // query heads per KV head
    int NR;           // rep * W query rows per KV head
    int n_seg;        // ceil(T / SEG)
    int seg_per_chunk;
    int n_chunks;
    int64_t stride_l, stride_h;
    float inv_sqrt_d;
    float *pm, *ps, *pp;      // [rows][n_seg]: segment max, sum exp, weighted sum exp
    float *row_max, *row_inv; // [rows]
    float *part;              // [Y][n_seg]
    float *scores;
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
                const int64_t o = (row0 + j0 + j) * a.n_seg + seg;
                a.pm[o] = m;
                a.ps[o] = se;
                a.pp[o] = sp;
            }
        }
    }
}

// ------------------------------------------------------------------ the same, staged through shared memory
//
// For head_dim 64, 128 or 256.  A warp owns tiles of 32 consecutive tokens of one (layer, KV head).  It copies
// a tile (32 x head_dim fp16, contiguous in memory) into shared memory with coalesced 16-byte asynchronous
// copies (cp.async, two buffers: the next tile lands while this one is used), swizzled by XOR-ing the 16-byte
// chunk index with the row index so that lane t can then read row t without bank conflicts.  The dot products
// use the sm_100 mixed-precision fma (fp16 x fp16 + fp32, one rounding; the products are exact), so neither K
// nor q is ever converted, and q stays in shared memory as fp16, read as warp-wide broadcasts: 8 fma per
// 16-byte load.
constexpr int kTileTokens = 32;
constexpr int kTileWarps = 4;

__device__ __forceinline__ float fma_f32_f16(unsigned short x, unsigned short y, float c)
{
    float d;
    asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(d) : "h"(x), "h"(y), "f"(c));
    return d;
}
__device__ __forceinline__ void split_halves(uint32_t w, unsigned short &lo, unsigned short &hi)
{
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(w));
}
// 16-byte asynchronous copy global -> shared, bypassing L1; src_bytes = 0 fills zeros instead
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void *src, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory"); }

template <int RT, int D>
__global__ void __launch_bounds__(kTileWarps * 32) logits_tile_kernel(const TolArgs a, const int seg_len)
{
    constexpr int kRowBytes = D * 2, kChunks = D / 8, kTileBytes = kTileTokens * kRowBytes;
    constexpr int kUnrollChunks = 64 / RT;                                   // 512 fma per unrolled trip
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
    const int nr_pad = (a.NR + RT - 1) / RT * RT;                            // rows padded with zeros to whole row tiles
    __half *q_s = reinterpret_cast<__half *>(smem_raw);                      // [nr_pad][D] fp16
    unsigned char *tiles = smem_raw + nr_pad * kRowBytes + wib * 2 * kTileBytes;  // this warp's two buffers
    const uint32_t tiles_s = (uint32_t)__cvta_generic_to_shared(tiles);

    const int l = blockIdx.y / a.Hkv, kvh = blockIdx.y % a.Hkv;
    const __half *q_src = a.q_win + ((int64_t)(l * a.Hq + kvh * a.rep) * a.W) * D;
    for (int i = threadIdx.x; i < nr_pad * kChunks; i += blockDim.x)
        reinterpret_cast<uint4 *>(q_s)[i] = i < a.NR * kChunks ? __ldg(reinterpret_cast<const uint4 *>(q_src) + i) : make_uint4(0, 0, 0, 0);
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

    int buf = 0;
    if (tile_begin < tile_end) issue_tile(tile_begin, 0);
    for (int tile = tile_begin; tile < tile_end; tile += kTileWarps, buf ^= 1) {
        if (tile + kTileWarps < tile_end) {
            issue_tile(tile + kTileWarps, buf ^ 1);
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncwarp();
        const int t = tile * kTileTokens + lane;
        const bool valid = t < a.T;
        const int n_vis = min(a.W, a.T - (valid ? t : 0));
        const float w_col = 1.0f / (float)n_vis;
        const int seg = t / seg_len;
        const unsigned char *my_row = tiles + buf * kTileBytes + lane * kRowBytes;
        const int swz = (lane & 7) << 4;
        for (int j0 = 0; j0 < a.NR; j0 += RT) {
            float acc[RT];
#pragma unroll
            for (int j = 0; j < RT; ++j) acc[j] = 0.0f;
            const __half *q_tile = q_s + j0 * D;
#pragma unroll kUnrollChunks
            for (int c = 0; c < kChunks; ++c) {
                const uint4 kk = *reinterpret_cast<const uint4 *>(my_row + ((c << 4) ^ swz));
                const uint32_t kw[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                for (int j = 0; j < RT; ++j) {
                    const uint4 qq = *reinterpret_cast<const uint4 *>(q_tile + j * D + c * 8);
                    const uint32_t qw[4] = {qq.x, qq.y, qq.z, qq.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        unsigned short k0, k1, q0, q1;
                        split_halves(kw[i], k0, k1);
                        split_halves(qw[i], q0, q1);
                        acc[j] = fma_f32_f16(k0, q0, acc[j]);
                        acc[j] = fma_f32_f16(k1, q1, acc[j]);
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < RT; ++j) {
                if (j0 + j >= a.NR) break;  // uniform
                const int r = (j0 + j) % a.W;
                const bool vis = valid && t <= a.T - a.W + r;
                const float logit = vis ? acc[j] * a.inv_sqrt_d : -INFINITY;
                float m = logit;
                for (int s = seg_len / 2; s > 0; s >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
                const float e = vis ? expf(logit - m) : 0.0f;
                float se = e, sp = e * w_col;
                for (int s = seg_len / 2; s > 0; s >>= 1) {
                    se += __shfl_xor_sync(0xffffffffu, se, s);
                    sp += __shfl_xor_sync(0xffffffffu, sp, s);
                }
                if (valid && (lane & (seg_len - 1)) == 0) {
                    const int64_t o = (row0 + j0 + j) * a.n_seg + seg;
                    a.pm[o] = m;
                    a.ps[o] = se;
                    a.pp[o] = sp;
                }
            }
        }
        __syncwarp();  // the buffer is free for the copy issued two tiles from now
    }
}

// one warp per row: global max and 1 / sum of exp
__global__ void row_stats_kernel(const TolArgs a)
{
    const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= a.rows) return;
    const int lane = threadIdx.x & 31;
    const float *pm = a.pm + (int64_t)row * a.n_seg;
    const float *ps = a.ps + (int64_t)row * a.n_seg;
    float m = -INFINITY;
    for (int s = lane; s < a.n_seg; s += 32) m = fmaxf(m, pm[s]);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, s));
    float sum = 0.0f;
    for (int s = lane; s < a.n_seg; s += 32) {
        const float ms = pm[s];
        if (ms != -INFINITY) sum += ps[s] * expf(ms - m);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, s);
    if (lane == 0) {
        a.row_max[row] = m;
        a.row_inv[row] = 1.0f / sum;
    }
}

// block (32 segments x 8 row lanes); blockIdx.y picks a slice of rows
__global__ void __launch_bounds__(256) column_sum_kernel(const TolArgs a)
{
    __shared__ float red[8][33];
    const int seg = blockIdx.x * 32 + threadIdx.x;
    const int rows_per_slice = (a.rows + a.Y - 1) / a.Y;
    const int r_begin = blockIdx.y * rows_per_slice;
    const int r_end = min(a.rows, r_begin + rows_per_slice);
    float acc = 0.0f;
    if (seg < a.n_seg) {
        for (int row = r_begin + threadIdx.y; row < r_end; row += 8) {
            const int64_t o = (int64_t)row * a.n_seg + seg;
            const float ms = a.pm[o];
            if (ms != -INFINITY) acc += a.pp[o] * expf(ms - a.row_max[row]) * a.row_inv[row];
        }
    }
    red[threadIdx.y][threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.y == 0 && seg < a.n_seg) {
        float s = 0.0f;
#pragma unroll
        for (int y = 0; y < 8; ++y) s += red[y][threadIdx.x];
        a.part[(int64_t)blockIdx.y * a.n_seg + seg] = s;
    }
}

// thread per chunk: sum the row slices and the chunk's segments, scale to the mean
__global__ void chunk_mean_kernel(const TolArgs a)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= a.n_chunks) return;
    float tot = 0.0f;
    for (int s = c * a.seg_per_chunk; s < (c + 1) * a.seg_per_chunk; ++s) {
        float col = 0.0f;
        for (int y = 0; y < a.Y; ++y) col += a.part[(int64_t)y * a.n_seg + s];
        tot += col;
    }
    a.scores[c] = tot / ((float)a.CL * (float)a.L * (float)a.Hq);
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

static int row_slices(int rows) { return rows >= 512 ? 16 : (rows >= 64 ? 4 : 1); }

struct TolLayout {
    int SEG, n_seg, rows, Y;
    uint64_t off_pm, off_ps, off_pp, off_rmax, off_rinv, off_part, total;
};

static TolLayout tol_layout(const llms_kv_desc &d, int W)
{
    TolLayout t;
    t.SEG = seg_len(d.chunk_len);
    t.n_seg = (d.n_tokens + t.SEG - 1) / t.SEG;
    t.rows = d.n_layers * d.n_q_heads * W;
    t.Y = row_slices(t.rows);
    const uint64_t stat = round_up((uint64_t)t.rows * t.n_seg * 4, 256);
    t.off_pm = 0;
    t.off_ps = stat;
    t.off_pp = 2 * stat;
    t.off_rmax = 3 * stat;
    t.off_rinv = t.off_rmax + round_up((uint64_t)t.rows * 4, 256);
    t.off_part = t.off_rinv + round_up((uint64_t)t.rows * 4, 256);
    t.total = t.off_part + round_up((uint64_t)t.Y * t.n_seg * 4, 256);
    return t;
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
    a.seg_per_chunk = a.CL / t.SEG;
    a.n_chunks = n_chunks(*desc);
    a.stride_l = desc->stride_l; a.stride_h = desc->stride_h;
    a.inv_sqrt_d = (float)(1.0 / sqrt((double)a.d));
    uint8_t *ws = static_cast<uint8_t *>(workspace);
    a.pm = reinterpret_cast<float *>(ws + t.off_pm);
    a.ps = reinterpret_cast<float *>(ws + t.off_ps);
    a.pp = reinterpret_cast<float *>(ws + t.off_pp);
    a.row_max = reinterpret_cast<float *>(ws + t.off_rmax);
    a.row_inv = reinterpret_cast<float *>(ws + t.off_rinv);
    a.part = reinterpret_cast<float *>(ws + t.off_part);
    a.scores = scores;
    a.Y = t.Y; a.rows = t.rows;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if ((unsigned)(a.L * a.Hkv) > 65535u) return LLMS_ERR_UNSUPPORTED;
    const int rt = a.NR <= 8 ? 8 : (a.NR <= 16 ? 16 : 32);
    const size_t tile_q_bytes = (size_t)((a.NR + rt - 1) / rt * rt) * a.d * 2;
    const size_t tile_smem = tile_q_bytes + (size_t)kTileWarps * 2 * kTileTokens * a.d * 2;
    if ((a.d == 64 || a.d == 128 || a.d == 256) && tile_smem <= 200 * 1024) {
        // tiles through shared memory; enough blocks per (layer, KV head) to fill the GPU a few times over
        const int n_tiles = (a.T + kTileTokens - 1) / kTileTokens;
        const int pairs = a.L * a.Hkv;
        int splits = (sm_count() * 6 + pairs - 1) / pairs;
        splits = std::max(1, std::min(splits, (n_tiles + kTileWarps - 1) / kTileWarps));
        const dim3 grid(splits, pairs);
#define LLMS_LAUNCH_TILE(R, DD)                                                                                                   \
    do {                                                                                                                          \
        LLMS_CUDA_TRY(cudaFuncSetAttribute(logits_tile_kernel<R, DD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tile_smem)); \
        logits_tile_kernel<R, DD><<<grid, kTileWarps * 32, tile_smem, st>>>(a, t.SEG);                                            \
    } while (0)
#define LLMS_LAUNCH_TILE_D(R)                                                       \
    do {                                                                            \
        if (a.d == 64) LLMS_LAUNCH_TILE(R, 64);                                     \
        else if (a.d == 128) LLMS_LAUNCH_TILE(R, 128);                              \
        else LLMS_LAUNCH_TILE(R, 256);                                              \
    } while (0)
        if (rt == 8) LLMS_LAUNCH_TILE_D(8);
        else if (rt == 16) LLMS_LAUNCH_TILE_D(16);
        else LLMS_LAUNCH_TILE_D(32);
#undef LLMS_LAUNCH_TILE_D
#undef LLMS_LAUNCH_TILE
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
    LLMS_CUDA_TRY(cudaGetLastError());
    row_stats_kernel<<<(a.rows + 7) / 8, 256, 0, st>>>(a);
    LLMS_CUDA_TRY(cudaGetLastError());
    column_sum_kernel<<<dim3((a.n_seg + 31) / 32, a.Y), dim3(32, 8), 0, st>>>(a);
    LLMS_CUDA_TRY(cudaGetLastError());
    chunk_mean_kernel<<<(a.n_chunks + 127) / 128, 128, 0, st>>>(a);
    LLMS_CUDA_TRY(cudaGetLastError());
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
