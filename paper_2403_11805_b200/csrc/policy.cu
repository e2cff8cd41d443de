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
    if (!desc || !scores_dev || !scores_host || !bits_out) return LLMS_ERR_INVALID_ARG;
    // Into page-locked memory the last score kernel stores the scores itself (a copy after the kernels costs a switch to
    // the copy engine and back: about 15 us per context); pageable memory gets them by a copy.
    float *scores_live = static_cast<float *>(llms::device_view_of_pinned(scores_host));
    int rc = llms::chunk_tolerance_impl(desc, kv, q_win, W, scores_dev, scores_live, tolerance_workspace,
                                        tolerance_workspace_bytes, stream);
    if (rc) return rc;
    const int n = (int)llms::n_chunks(*desc);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
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
