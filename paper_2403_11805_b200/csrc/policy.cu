// Host-side policies: rank -> bit-width (Eq. 2), the thresholds of Eq. 3 and the LCTRU eviction order (Sec. 3.4 ii);
// and the call that strings score, ranking and compression of a whole context together.
#include <algorithm>
#include <cmath>
#include <numeric>
#include <vector>

#include "llms_internal.cuh"

extern "C" int llms_assign_levels(const float *scores, int n, const float frac[3], const uint8_t levels[3],
                                  uint8_t *bits_out, uint32_t *order_out)
{
    if (n < 0 || !frac || !levels || (n > 0 && (!scores || !bits_out))) return LLMS_ERR_INVALID_ARG;
    for (int w = 0; w < 3; ++w)
        if (llms::check_bits(levels[w])) return LLMS_ERR_BAD_BITS;
    if (!(levels[0] > levels[1] && levels[1] > levels[2])) return LLMS_ERR_INVALID_ARG;
    const double f_top = frac[0], f_mid = frac[1], f_low = frac[2];
    if (!(f_top >= 0) || !(f_mid >= 0) || !(f_low >= 0) || std::fabs(f_top + f_mid + f_low - 1.0) > 1e-3) return LLMS_ERR_INVALID_ARG;
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    // densest first; equal densities keep index order
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return scores[a] > scores[b]; });
    long n_top = (long)std::floor(f_top * n + 0.5);
    long n_top_mid = (long)std::floor((f_top + f_mid) * n + 0.5);
    n_top = std::min<long>(n_top, n);
    n_top_mid = std::max(std::min<long>(n_top_mid, n), n_top);
    for (long r = 0; r < n; ++r) {
        bits_out[order[r]] = r < n_top ? levels[0] : (r < n_top_mid ? levels[1] : levels[2]);
        if (order_out) order_out[r] = order[r];
    }
    return LLMS_OK;
}

extern "C" int llms_assign_bits(const float *scores, int n, const float frac[3], uint8_t *bits_out, uint32_t *order_out)
{
    static const uint8_t kLevels[3] = {8, 4, 2};
    return llms_assign_levels(scores, n, frac, kLevels, bits_out, order_out);
}

extern "C" int llms_optimize_thresholds_levels(const float *scores, int n, float ratio_global, const uint8_t levels[3],
                                               float frac_out[3])
{
    if (n <= 0 || !scores || !levels || !frac_out) return LLMS_ERR_INVALID_ARG;
    for (int w = 0; w < 3; ++w)
        if (llms::check_bits(levels[w])) return LLMS_ERR_BAD_BITS;
    if (!(levels[0] > levels[1] && levels[1] > levels[2])) return LLMS_ERR_INVALID_ARG;
    // a chunk at the middle / low level keeps r1 / r2 of the top level's bytes, and of its density's weight
    const double r1 = (double)levels[1] / (double)levels[0], r2 = (double)levels[2] / (double)levels[0];
    const double R = (double)ratio_global;
    if (!(R >= r2 && R <= 1.0)) return LLMS_ERR_INVALID_ARG;
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return scores[a] > scores[b]; });
    // prefix[k] = density of the k densest chunks, added in rank order
    std::vector<double> prefix(n + 1, 0.0);
    for (int k = 0; k < n; ++k) prefix[k + 1] = prefix[k] + (double)scores[order[k]];
    long best_top = -1, best_low = 0;
    double best = 0.0;
    for (long n_top = 0; n_top <= n; ++n_top) {
        // shares: f0 + f1 + f2 = 1 and f0 + r1 f1 + r2 f2 = R  =>  f2 = ((1 - r1) f0 + r1 - R) / (r1 - r2)
        const long n_low = (long)std::floor(((1.0 - r1) * n_top + (r1 - R) * n) / (r1 - r2) + 0.5);
        if (n_low < 0 || n_top + n_low > n) continue;
        const double info = prefix[n_top] + (prefix[n - n_low] - prefix[n_top]) * r1 + (prefix[n] - prefix[n - n_low]) * r2;
        if (best_top < 0 || info > best) {
            best_top = n_top;
            best_low = n_low;
            best = info;
        }
    }
    if (best_top < 0) return LLMS_ERR_INVALID_ARG;
    frac_out[0] = (float)((double)best_top / n);
    frac_out[1] = (float)((double)(n - best_top - best_low) / n);
    frac_out[2] = (float)((double)best_low / n);
    return LLMS_OK;
}

extern "C" int llms_optimize_thresholds(const float *scores, int n, float ratio_global, float frac_out[3])
{
    static const uint8_t kLevels[3] = {8, 4, 2};
    return llms_optimize_thresholds_levels(scores, n, ratio_global, kLevels, frac_out);
}

extern "C" int llms_lctru_order(const llms_chunk_state *table, int n, uint32_t *order_out)
{
    if (n < 0 || (n > 0 && (!table || !order_out))) return LLMS_ERR_INVALID_ARG;
    int m = 0;
    for (int i = 0; i < n; ++i) {
        if (table[i].resident && !table[i].locked) {
            if (llms::check_bits((int)table[i].bits)) return LLMS_ERR_BAD_BITS;
            order_out[m++] = (uint32_t)i;
        }
    }
    // concatenated sub-queues: 8-bit chunks first, then 4, then 2; least recently used first inside each
    std::sort(order_out, order_out + m, [&](uint32_t x, uint32_t y) {
        const llms_chunk_state &a = table[x], &b = table[y];
        if (a.bits != b.bits) return a.bits > b.bits;
        if (a.last_access_step != b.last_access_step) return a.last_access_step < b.last_access_step;
        if (a.ctx_id != b.ctx_id) return a.ctx_id < b.ctx_id;
        if (a.chunk_id != b.chunk_id) return a.chunk_id < b.chunk_id;
        return x < y;
    });
    return m;
}

namespace llms {

// Eq. 2 and the chunk tables of the encoder on the device, for a context whose scores have just been computed on the
// same stream (one CTA; n <= kPlanMaxChunks).  The chunks are ranked in the order "denser first, equal densities by
// index" - exactly the order the host's stable sort produces - so levels and record offsets equal those of
// llms_assign_levels followed by llms_compress_chunks on the same score bits.
constexpr int kPlanMaxChunks = 4096;
constexpr int kPlanThreads = 1024;
constexpr int kPlanCountChunks = 256;   // up to here ranks are counted, above the keys are sorted

struct PlanArgs {
    const float *scores;       // device, n
    int n, n_top, n_top_mid;   // ranks below n_top keep levels[0], below n_top_mid levels[1], the rest levels[2]
    uint32_t levels[3];
    uint64_t rec_bytes[3];     // record size per level
    uint32_t n_groups;
    int first[4];              // where the chunks of width 8, 4, 2, 1 start in the grouped order
    uint8_t *workspace;        // codec workspace: header, entries, unit table, grouped order
    llms_chunk_meta *meta;     // the caller's page-locked meta array (device view)
    uint8_t *bits_out;         // the caller's page-locked level array (device view)
};

__device__ __forceinline__ int width_class(uint32_t bits) { return bits == 8 ? 0 : (bits == 4 ? 1 : (bits == 2 ? 2 : 3)); }

// inclusive scan of one value per thread over the CTA (kPlanThreads threads), fixed order
template <typename T>
__device__ __forceinline__ T block_inclusive_scan(T v, T *warp_totals)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const T up = __shfl_up_sync(0xffffffffu, v, d);
        if (lane >= d) v += up;
    }
    if (lane == 31) warp_totals[w] = v;
    __syncthreads();
    if (w == 0) {
        T t = warp_totals[lane];
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const T up = __shfl_up_sync(0xffffffffu, t, d);
            if (lane >= d) t += up;
        }
        warp_totals[lane] = t;
    }
    __syncthreads();
    const T before = w > 0 ? warp_totals[w - 1] : T(0);
    __syncthreads();
    return v + before;
}

__global__ void __launch_bounds__(kPlanThreads) plan_context_kernel(const PlanArgs a)
{
    __shared__ unsigned long long s_key[kPlanMaxChunks];       // (descending score, ascending index) as one rising key
    __shared__ uint8_t s_level[kPlanMaxChunks];                // index into levels[]
    __shared__ unsigned long long s_scan[32];
    grid_dependency_wait();
    const int n = a.n;
    int n2 = 2;                                                // keys are sorted in a power-of-two array
    while (n2 < n) n2 *= 2;
    for (int i = threadIdx.x; i < n2; i += kPlanThreads) {
        // the bits of a float as an unsigned number that rises with the float (for scores, which are not negative,
        // this only sets the top bit), inverted so that the densest chunk gets the smallest key; padding sorts last
        unsigned long long key = ~0ull;
        if (i < n) {
            uint32_t b = __float_as_uint(a.scores[i]);
            if (b == 0x80000000u) b = 0;                       // -0 and +0 are one density
            const uint32_t rising = b ^ ((b >> 31) ? 0xffffffffu : 0x80000000u);
            key = ((unsigned long long)(~rising) << 32) | (uint32_t)i;
        }
        s_key[i] = key;
    }
    // the header: status word, spare, finished-CTA count, work-split counters
    for (int i = threadIdx.x; i < (int)(kWsEntriesOffset / 4); i += blockDim.x) reinterpret_cast<uint32_t *>(a.workspace)[i] = 0;
    __syncthreads();
    if (n <= kPlanCountChunks) {
        // Few chunks: the rank of a chunk is the number of keys below its own, counted by `parts` neighbouring lanes
        // that split the array among them (a power of two, at most 32, so that they sit in one warp).
        int parts = 1;
        while (parts < 32 && n * parts * 2 <= kPlanThreads) parts *= 2;
        const int i = (int)threadIdx.x / parts, p = threadIdx.x % parts;
        int rank = 0;
        if (i < n) {
            const unsigned long long mine = s_key[i];
            for (int j = p; j < n; j += parts) rank += s_key[j] < mine;
        }
        for (int d = 1; d < parts; d <<= 1) rank += __shfl_xor_sync(0xffffffffu, rank, d);
        if (i < n && p == 0) s_level[i] = rank < a.n_top ? 0 : (rank < a.n_top_mid ? 1 : 2);
    } else {
        // Bitonic sort; a thread per comparator, and only the warps that have one take part in the barriers between
        // the stages.  Position r of the sorted array then names the chunk of rank r.  (Counting takes n / 4 trips
        // through the array per thread from 1024 chunks on: 6 us of this kernel's 20 at 512 chunks, growing with
        // the square of n; the sort's 45 stages take 2 us there, but more than counting does up to 256 chunks.)
        const int comparators = n2 / 2;
        const int sort_threads = min(kPlanThreads, (comparators + 31) / 32 * 32);
        if ((int)threadIdx.x < sort_threads) {
            for (int k = 2; k <= n2; k <<= 1) {
                for (int j = k >> 1; j > 0; j >>= 1) {
                    for (int t = threadIdx.x; t < comparators; t += sort_threads) {
                        const int lo = ((t & ~(j - 1)) << 1) | (t & (j - 1));   // comparator t: the positions lo and lo + j
                        const int hi = lo | j;
                        const unsigned long long x = s_key[lo], y = s_key[hi];
                        if ((x > y) == ((lo & k) == 0)) {
                            s_key[lo] = y;
                            s_key[hi] = x;
                        }
                    }
                    asm volatile("bar.sync 1, %0;" :: "r"(sort_threads) : "memory");
                }
            }
            for (int r = threadIdx.x; r < n; r += sort_threads)
                s_level[(uint32_t)s_key[r]] = r < a.n_top ? 0 : (r < a.n_top_mid ? 1 : 2);
        }
    }
    __syncthreads();
    // every thread owns a run of consecutive chunks: record bytes and per-width counts before each chunk by two scans
    const int per = (n + kPlanThreads - 1) / kPlanThreads;
    const int begin = min(n, (int)threadIdx.x * per), end = min(n, begin + per);
    unsigned long long bytes = 0, counts = 0;                  // counts: four 16-bit fields, one per width class
    for (int i = begin; i < end; ++i) {
        bytes += a.rec_bytes[s_level[i]];
        counts += 1ull << (16 * width_class(a.levels[s_level[i]]));
    }
    unsigned long long off = block_inclusive_scan(bytes, s_scan) - bytes;
    unsigned long long seen = block_inclusive_scan(counts, s_scan) - counts;
    ChunkEntry *entries = reinterpret_cast<ChunkEntry *>(a.workspace + kWsEntriesOffset);
    UnitEntry *table = reinterpret_cast<UnitEntry *>(a.workspace + ws_table_offset(n));
    uint32_t *order = reinterpret_cast<uint32_t *>(a.workspace + ws_order_offset(n));
    for (int i = begin; i < end; ++i) {
        const int lv = s_level[i];
        const uint32_t bits = a.levels[lv];
        const int k = width_class(bits);
        ChunkEntry e;
        e.chunk_id = (uint32_t)i;
        e.bits = bits;
        e.offset = off;
        e.nbytes = a.rec_bytes[lv];
        e.n_groups = a.n_groups;
        e.checksum = 0;                                        // the encoder accumulates into the device copy
        entries[i] = e;
        const int at = a.first[k] + (int)((seen >> (16 * k)) & 0xffffu);
        order[at] = (uint32_t)i;
        UnitEntry u;
        u.chunk_id = (uint32_t)i;
        u.entry = (uint32_t)i;
        u.rec_off = off;
        table[at] = u;
        off += a.rec_bytes[lv];
        seen += 1ull << (16 * k);
    }
    grid_launch_dependents();   // the encoder may be set up now; it waits for this kernel to complete before it reads the tables
    // The caller's meta and level arrays lie across the host link, where every store instruction of a lane is a
    // transaction of its own: they are written as whole warps of neighbouring 16-byte pieces (the meta entries are the
    // bytes of the entries just laid down, read back through L2).
    __syncthreads();
    const uint4 *from = reinterpret_cast<const uint4 *>(entries);
    uint4 *to = reinterpret_cast<uint4 *>(a.meta);
    for (int i = threadIdx.x; i < 2 * n; i += kPlanThreads) to[i] = __ldcg(from + i);
    if ((reinterpret_cast<uintptr_t>(a.bits_out) & 15) == 0) {
        for (int i0 = threadIdx.x * 16; i0 < n; i0 += kPlanThreads * 16) {
            uint32_t w[4] = {0, 0, 0, 0};
            for (int k = 0; k < 16 && i0 + k < n; ++k) w[k >> 2] |= a.levels[s_level[i0 + k]] << (8 * (k & 3));
            if (i0 + 16 <= n) {
                *reinterpret_cast<uint4 *>(a.bits_out + i0) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
                for (int k = 0; i0 + k < n; ++k) a.bits_out[i0 + k] = (uint8_t)(w[k >> 2] >> (8 * (k & 3)));
            }
        }
    } else {
        for (int i = threadIdx.x; i < n; i += kPlanThreads) a.bits_out[i] = (uint8_t)a.levels[s_level[i]];
    }
}

// The counts of Eq. 2's three levels for n chunks: the first n_top ranks, then up to n_top_mid.
static void level_counts(int n, const float frac[3], long &n_top, long &n_top_mid)
{
    const double f_top = frac[0], f_mid = frac[1];
    n_top = std::min<long>((long)std::floor(f_top * n + 0.5), n);
    n_top_mid = std::max(std::min<long>((long)std::floor((f_top + f_mid) * n + 0.5), n), n_top);
}

}  // namespace llms

// Score -> levels -> records for all chunks of a context: the three calls a swap-out makes, without the host
// round trips between them.
extern "C" int llms_compress_context(const llms_kv_desc *desc, const void *kv, const void *q_win, int W,
                                     const float frac[3], const uint8_t levels[3],
                                     float *scores_dev, float *scores_host, uint8_t *bits_out,
                                     void *out_buf, uint64_t out_bytes, llms_chunk_meta *meta,
                                     void *tolerance_workspace, uint64_t tolerance_workspace_bytes,
                                     void *codec_workspace, uint64_t codec_workspace_bytes,
                                     void *after_scores, void *stream)
{
    using namespace llms;
    if (!desc || !scores_dev || !scores_host || !bits_out || !frac || !levels || !meta) return LLMS_ERR_INVALID_ARG;
    // ---- everything that can be wrong is found before the first launch
    int rc = check_desc(desc);
    if (rc) return rc;
    const int n = (int)n_chunks(*desc);
    for (int w = 0; w < 3; ++w)
        if (check_bits(levels[w])) return LLMS_ERR_BAD_BITS;
    if (!(levels[0] > levels[1] && levels[1] > levels[2])) return LLMS_ERR_INVALID_ARG;
    if (!(frac[0] >= 0) || !(frac[1] >= 0) || !(frac[2] >= 0) || std::fabs((double)frac[0] + frac[1] + frac[2] - 1.0) > 1e-3)
        return LLMS_ERR_INVALID_ARG;
    rc = check_compress_args(desc, n, kv, out_buf, codec_workspace, codec_workspace_bytes);
    if (rc) return rc;
    long n_top, n_top_mid;
    level_counts(n, frac, n_top, n_top_mid);
    uint64_t rec_bytes[3], need = 0;
    for (int w = 0; w < 3; ++w) {
        rc = llms_record_bytes(desc, levels[w], &rec_bytes[w]);
        if (rc) return rc;
    }
    need = (uint64_t)n_top * rec_bytes[0] + (uint64_t)(n_top_mid - n_top) * rec_bytes[1] + (uint64_t)(n - n_top_mid) * rec_bytes[2];
    if (need > out_bytes) return LLMS_ERR_BUF_TOO_SMALL;      // the levels' counts follow from frac and n alone

    // Into page-locked memory the last score kernel stores the scores itself (a copy after the kernels costs a switch to
    // the copy engine and back: about 15 us per context); pageable memory gets them by a copy.
    float *scores_live = static_cast<float *>(device_view_of_pinned(scores_host));
    uint8_t *bits_live = static_cast<uint8_t *>(device_view_of_pinned(bits_out));
    llms_chunk_meta *meta_live = static_cast<llms_chunk_meta *>(device_view_of_pinned(meta));
    rc = chunk_tolerance_impl(desc, kv, q_win, W, scores_dev, scores_live, tolerance_workspace, tolerance_workspace_bytes, stream);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n == 0) return LLMS_OK;

    if (scores_live && bits_live && meta_live && n <= kPlanMaxChunks) {
        // ---- stream-ordered: a kernel ranks the chunks and lays the encoder's tables down; nothing waits for the host
        PlanArgs p{};
        p.scores = scores_dev;
        p.n = n;
        p.n_top = (int)n_top;
        p.n_top_mid = (int)n_top_mid;
        int count[4] = {0, 0, 0, 0};
        const long level_n[3] = {n_top, n_top_mid - n_top, n - n_top_mid};
        for (int w = 0; w < 3; ++w) {
            p.levels[w] = levels[w];
            p.rec_bytes[w] = rec_bytes[w];
            count[levels[w] == 8 ? 0 : (levels[w] == 4 ? 1 : (levels[w] == 2 ? 2 : 3))] = (int)level_n[w];
        }
        for (int k = 0, at = 0; k < 4; ++k) {
            p.first[k] = at;
            at += count[k];
        }
        p.n_groups = (uint32_t)groups_per_chunk(*desc);
        p.workspace = static_cast<uint8_t *>(codec_workspace);
        p.meta = meta_live;
        p.bits_out = bits_live;
        LLMS_CUDA_TRY(launch_dependent(plan_context_kernel, dim3(1), dim3(kPlanThreads), 0, st, p));
        if (after_scores) LLMS_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(after_scores), st));
        return compress_planned(desc, kv, n, count, out_buf, out_bytes, meta, codec_workspace, stream);
    }

    // ---- the ranking as a host step: one synchronisation, when the scores have reached the host
    if (!scores_live)
        LLMS_CUDA_TRY(cudaMemcpyAsync(scores_host, scores_dev, (size_t)n * sizeof(float), cudaMemcpyDeviceToHost, st));
    if (after_scores) LLMS_CUDA_TRY(cudaEventRecord(static_cast<cudaEvent_t>(after_scores), st));
    LLMS_CUDA_TRY(cudaStreamSynchronize(st));
    rc = llms_assign_levels(scores_host, n, frac, levels, bits_out, nullptr);
    if (rc) return rc;
    std::vector<uint32_t> ids(n);
    std::iota(ids.begin(), ids.end(), 0u);
    return llms_compress_chunks(desc, kv, ids.data(), bits_out, n, out_buf, out_bytes, meta, codec_workspace,
                                codec_workspace_bytes, stream);
}
