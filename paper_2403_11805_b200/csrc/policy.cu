// Host-side policies: rank -> bit-width (Eq. 2) and the LCTRU eviction order (Sec. 3.4 ii).
#include <algorithm>
#include <cmath>
#include <numeric>
#include <vector>

#include "llms_internal.cuh"

extern "C" int llms_assign_bits(const float *scores, int n, const float frac[3], uint8_t *bits_out, uint32_t *order_out)
{
    if (n < 0 || !frac || (n > 0 && (!scores || !bits_out))) return LLMS_ERR_INVALID_ARG;
    const double f8 = frac[0], f4 = frac[1], f2 = frac[2];
    if (!(f8 >= 0) || !(f4 >= 0) || !(f2 >= 0) || std::fabs(f8 + f4 + f2 - 1.0) > 1e-3) return LLMS_ERR_INVALID_ARG;
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    // densest first; equal densities keep index order
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return scores[a] > scores[b]; });
    long n8 = (long)std::floor(f8 * n + 0.5);
    long n84 = (long)std::floor((f8 + f4) * n + 0.5);
    n8 = std::min<long>(n8, n);
    n84 = std::max(std::min<long>(n84, n), n8);
    for (long r = 0; r < n; ++r) {
        bits_out[order[r]] = r < n8 ? 8 : (r < n84 ? 4 : 2);
        if (order_out) order_out[r] = order[r];
    }
    return LLMS_OK;
}

extern "C" int llms_optimize_thresholds(const float *scores, int n, float ratio_global, float frac_out[3])
{
    if (n <= 0 || !scores || !frac_out) return LLMS_ERR_INVALID_ARG;
    const double R = (double)ratio_global;
    if (!(R >= 0.25 && R <= 1.0)) return LLMS_ERR_INVALID_ARG;
    std::vector<uint32_t> order(n);
    std::iota(order.begin(), order.end(), 0u);
    std::stable_sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return scores[a] > scores[b]; });
    // prefix[k] = density of the k densest chunks, added in rank order
    std::vector<double> prefix(n + 1, 0.0);
    for (int k = 0; k < n; ++k) prefix[k + 1] = prefix[k] + (double)scores[order[k]];
    long best8 = -1, best2 = 0;
    double best = 0.0;
    for (long n8 = 0; n8 <= n; ++n8) {
        // shares: f8 + f4 + f2 = 1 and f8 + f4/2 + f2/4 = R  =>  f2 = 2 f8 + 2 - 4R
        const long n2 = (long)std::floor(2.0 * n8 + (2.0 - 4.0 * R) * n + 0.5);
        if (n2 < 0 || n8 + n2 > n) continue;
        const double info = prefix[n8] + (prefix[n - n2] - prefix[n8]) / 2.0 + (prefix[n] - prefix[n - n2]) / 4.0;
        if (best8 < 0 || info > best) {
            best8 = n8;
            best2 = n2;
            best = info;
        }
    }
    if (best8 < 0) return LLMS_ERR_INVALID_ARG;
    frac_out[0] = (float)((double)best8 / n);
    frac_out[1] = (float)((double)(n - best8 - best2) / n);
    frac_out[2] = (float)((double)best2 / n);
    return LLMS_OK;
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
