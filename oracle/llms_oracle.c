/*
 * CPU oracle for the LLMS chunk codec and tolerance score.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, step-by-step
 * statement of what the GPU library has to compute.  It is built and called
 * by the tests, by the smoke check and by the benchmark's CPU-baseline leg,
 * and by nothing else; the GPU library neither includes nor links it, and it
 * includes nothing of the GPU library.
 *
 * Paper passages followed (LLMS, arXiv 2403.11805):
 *   - Sec. 3.1 "context memory model": a chunk = a fixed number of tokens of
 *     the KV cache (all layers and heads), one compression ratio per chunk.
 *   - Sec. 3.2 Eq. 1: information density D_i of a chunk from attention.
 *   - Sec. 3.2 Eq. 2: rank of D_i inside a context decides the ratio level.
 *   - Sec. 3.2 "Compressing chunks": linear quantization to lower bit-width,
 *     levels {8/8, 4/8, 2/8}.
 *   - Sec. 4: sub-byte codes packed into bytes with bit shifts.
 *   - Sec. 3.4 (ii): LCTRU queue = concatenated per-ratio sub-queues, each
 *     ordered by last access; working-set lock.
 *
 * Arithmetic.  The codec is an encoding, so its decisions are taken in the
 * precision the encoding is defined in: IEEE binary32, round to nearest even,
 * no fused multiply-add, no flush to zero; binary16 conversions are done in
 * integer arithmetic below.  The score (Eq. 1) is evaluated in binary64.
 * Build with -ffp-contract=off.
 *
 * Pins: every function here is pinned by tests/test_oracle_*.py (hand-worked
 * groups, the paper's worked density example, closed forms, brute force).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ types */

/* KV cache of one context (or one pool of chunk slots):
 *   element (l, s, h, t, c) lives at  l*stride_l + s*stride_s + h*stride_h + t*head_dim + c
 * s = 0 for K, 1 for V; strides in elements; values are binary16 bit patterns. */
typedef struct {
    int32_t n_layers, n_kv_heads, n_q_heads, head_dim;
    int32_t n_tokens, chunk_len, group_size, quant_mode; /* 0: groups of G channels of one token; 1: one group per channel across the chunk's tokens */
    int64_t stride_l, stride_s, stride_h;
} orc_kv_desc;

typedef struct {
    uint32_t chunk_id, bits;
    uint64_t offset, nbytes;
    uint32_t n_groups, checksum;
} orc_chunk_meta;

typedef struct {
    uint32_t ctx_id, chunk_id, bits, resident, locked, pad_;
    uint64_t last_access_step;
} orc_chunk_state;

enum { ORC_OK = 0, ORC_ERR_ARG = -1, ORC_ERR_BITS = -2, ORC_ERR_SMALL = -4 };

/* ----------------------------------------------------- binary16 <-> binary32 */

/* binary16 -> binary32, exact. */
float orc_f16_to_f32(uint16_t h)
{
    uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
    uint32_t e = (h >> 10) & 0x1fu;
    uint32_t m = h & 0x3ffu;
    uint32_t out;
    if (e == 0) {
        if (m == 0) {
            out = sign;
        } else { /* subnormal: m * 2^-24, normalise */
            int sh = 0;
            while ((m & 0x400u) == 0) { m <<= 1; ++sh; }
            m &= 0x3ffu;
            out = sign | ((uint32_t)(127 - 14 - sh) << 23) | (m << 13);
        }
    } else if (e == 31) {
        out = sign | 0x7f800000u | (m << 13);
    } else {
        out = sign | ((e + 127 - 15) << 23) | (m << 13);
    }
    float f;
    memcpy(&f, &out, 4);
    return f;
}

/* binary32 -> binary16, round to nearest, ties to even, subnormals kept,
 * overflow to infinity. */
uint16_t orc_f32_to_f16(float f)
{
    uint32_t x;
    memcpy(&x, &f, 4);
    uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
    uint32_t a = x & 0x7fffffffu;
    if (a >= 0x7f800000u) { /* inf / nan */
        if (a == 0x7f800000u) return (uint16_t)(sign | 0x7c00u);
        return (uint16_t)(sign | 0x7e00u | ((a >> 13) & 0x3ffu));
    }
    int32_t e = (int32_t)(a >> 23) - 127;
    uint32_t m24 = (a & 0x7fffffu) | 0x800000u; /* 1.m as a 24-bit integer, value m24 * 2^(e-23) */
    if ((a >> 23) == 0) return sign;             /* binary32 subnormal: far below half of 2^-24 */
    uint32_t q, rem, half;
    if (e >= -14) {
        if (e > 15) return (uint16_t)(sign | 0x7c00u);
        q = ((uint32_t)(e + 15) << 10) | ((m24 >> 13) & 0x3ffu);
        rem = m24 & 0x1fffu;
        half = 0x1000u;
    } else {
        int sh = -e - 1; /* result unit is 2^-24: q = m24 * 2^(e+1) */
        if (sh > 24) return sign;
        q = m24 >> sh;
        rem = m24 & ((1u << sh) - 1u);
        half = 1u << (sh - 1);
    }
    if (rem > half || (rem == half && (q & 1u))) ++q; /* a carry walks into the exponent, up to 0x7c00 = inf */
    return (uint16_t)(sign | q);
}

/* ----------------------------------------------------------- record layout */

static int desc_ok(const orc_kv_desc *d)
{
    if (!d) return 0;
    if (d->n_layers <= 0 || d->n_kv_heads <= 0 || d->n_q_heads <= 0 || d->head_dim <= 0) return 0;
    if (d->n_tokens <= 0 || d->chunk_len <= 0) return 0;
    if (d->n_q_heads % d->n_kv_heads) return 0;
    if (d->quant_mode == 0) {
        if (d->group_size <= 0 || d->head_dim % d->group_size) return 0;
    } else if (d->quant_mode != 1) {
        return 0;
    }
    return 1;
}

static int64_t n_slabs(const orc_kv_desc *d) { return (int64_t)d->n_layers * 2 * d->n_kv_heads; }

/* groups per chunk */
static uint64_t groups_per_chunk(const orc_kv_desc *d)
{
    if (d->quant_mode == 0)
        return (uint64_t)n_slabs(d) * d->chunk_len * (d->head_dim / d->group_size);
    return (uint64_t)n_slabs(d) * d->head_dim;
}

static uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

/* Record of one chunk:
 *   [n_groups x {u16 scale, u16 zero}]  padded with zero bytes to a multiple of 16
 *   [codes: element e of the chunk (memory order: slab, token, channel) occupies
 *           bits [e*b, (e+1)*b) of a little-endian bit stream]
 *   zero bytes up to a multiple of 256. */
int orc_record_layout(const orc_kv_desc *d, int bits, uint64_t *codes_off, uint64_t *nbytes)
{
    if (!desc_ok(d)) return ORC_ERR_ARG;
    if (bits != 1 && bits != 2 && bits != 4 && bits != 8) return ORC_ERR_BITS;
    uint64_t ng = groups_per_chunk(d);
    uint64_t n_elem = (uint64_t)n_slabs(d) * d->chunk_len * d->head_dim;
    if ((n_elem * bits) % 8) return ORC_ERR_ARG;
    uint64_t co = round_up(ng * 4, 16);
    if (codes_off) *codes_off = co;
    if (nbytes) *nbytes = round_up(co + n_elem * bits / 8, 256);
    return ORC_OK;
}

int orc_record_bytes(const orc_kv_desc *d, int bits, uint64_t *out)
{
    return orc_record_layout(d, bits, NULL, out);
}

int orc_compressed_size(const orc_kv_desc *d, const uint8_t *bits, int n, uint64_t *out)
{
    uint64_t tot = 0;
    for (int i = 0; i < n; ++i) {
        uint64_t nb;
        int rc = orc_record_bytes(d, bits[i], &nb);
        if (rc) return rc;
        tot += nb;
    }
    *out = tot;
    return ORC_OK;
}

/* ------------------------------------------------------------ quantization */

/* Steps Q1-Q4 on one group: x[0..n) at stride `step` (binary16 bit patterns).
 * Writes scale/zero bit patterns and one code per element. */
void orc_quantize_group(const uint16_t *x, int64_t step, int n, int bits,
                        uint16_t *scale_h, uint16_t *zero_h, uint8_t *codes)
{
    const int qmax = (1 << bits) - 1;
    float mn = orc_f16_to_f32(x[0]), mx = mn;
    uint16_t mn_h = x[0];
    for (int k = 1; k < n; ++k) { /* Q1: exact min / max */
        float v = orc_f16_to_f32(x[(int64_t)k * step]);
        if (v < mn) { mn = v; mn_h = x[(int64_t)k * step]; }
        if (v > mx) mx = v;
    }
    if (mn == 0.0f) mn_h = 0; /* -0 and +0 compare equal: store +0 */
    /* Q2: scale = binary16( (max - min) / (2^b - 1) ), zero-point = min */
    volatile float range = mx - mn;
    volatile float sc32 = range / (float)qmax;
    *scale_h = orc_f32_to_f16(sc32);
    if (*scale_h == 0x7C00) *scale_h = 0x7BFF; /* a range above 65504 (possible at 1 bit only) keeps the largest finite scale */
    *zero_h = mn_h;
    /* Q3 */
    float s = orc_f16_to_f32(*scale_h);
    if (s == 0.0f) {
        for (int k = 0; k < n; ++k) codes[k] = 0;
        return;
    }
    volatile float inv = 1.0f / s;
    float zero = orc_f16_to_f32(mn_h);
    for (int k = 0; k < n; ++k) { /* Q4 */
        volatile float diff = orc_f16_to_f32(x[(int64_t)k * step]) - zero;
        volatile float v = diff * inv;
        float r = rintf(v); /* ties to even in the default rounding mode */
        int q = (int)r;
        if (q < 0) q = 0;
        if (q > qmax) q = qmax;
        codes[k] = (uint8_t)q;
    }
}

/* Q5: code e occupies bits [e*b, (e+1)*b) of a little-endian bit stream. */
void orc_pack_codes(const uint8_t *codes, uint64_t n, int bits, uint8_t *out)
{
    uint64_t nbytes = (n * bits + 7) / 8;
    memset(out, 0, nbytes);
    for (uint64_t e = 0; e < n; ++e) {
        uint64_t bitpos = e * (uint64_t)bits;
        out[bitpos >> 3] |= (uint8_t)((codes[e] & ((1u << bits) - 1u)) << (bitpos & 7));
    }
}

void orc_unpack_codes(const uint8_t *in, uint64_t n, int bits, uint8_t *codes)
{
    for (uint64_t e = 0; e < n; ++e) {
        uint64_t bitpos = e * (uint64_t)bits;
        codes[e] = (uint8_t)((in[bitpos >> 3] >> (bitpos & 7)) & ((1u << bits) - 1u));
    }
}

/* y = binary16( zero + q * scale ): q*scale is exact in binary32 (8-bit times
 * 11-bit significand), so one binary32 rounding, then one binary16 rounding.
 * A result beyond the largest finite binary16 saturates instead of becoming
 * infinite (finite input must decode to finite output). */
uint16_t orc_dequantize_one(uint16_t scale_h, uint16_t zero_h, uint8_t q)
{
    float s = orc_f16_to_f32(scale_h);
    float z = orc_f16_to_f32(zero_h);
    volatile float prod = (float)q * s;
    volatile float v = z + prod;
    float w = v;
    if (w > 65504.0f) w = 65504.0f;
    if (w < -65504.0f) w = -65504.0f;
    return orc_f32_to_f16(w);
}

static uint32_t checksum_words(const uint8_t *p, uint64_t nbytes)
{
    uint32_t s = 0;
    for (uint64_t i = 0; i + 4 <= nbytes; i += 4)
        s += (uint32_t)p[i] | ((uint32_t)p[i + 1] << 8) | ((uint32_t)p[i + 2] << 16) | ((uint32_t)p[i + 3] << 24);
    return s;
}

static int64_t slab_base(const orc_kv_desc *d, int64_t s_idx, uint32_t chunk)
{
    int64_t h = s_idx % d->n_kv_heads;
    int64_t s = (s_idx / d->n_kv_heads) % 2;
    int64_t l = s_idx / (2 * d->n_kv_heads);
    return l * d->stride_l + s * d->stride_s + h * d->stride_h + (int64_t)chunk * d->chunk_len * d->head_dim;
}

/* Swap-out encoder (Reclaim's compression half): for each listed chunk, in
 * list order, quantize every group and lay its record down at the running
 * offset.  kv holds binary16 bit patterns.  meta[i] is filled in. */
int orc_compress_chunks(const orc_kv_desc *d, const uint16_t *kv, const uint32_t *chunk_ids,
                        const uint8_t *bits, int n, uint8_t *out_buf, uint64_t out_bytes,
                        orc_chunk_meta *meta)
{
    if (!desc_ok(d) || n < 0) return ORC_ERR_ARG;
    const uint32_t n_chunks = (uint32_t)(d->n_tokens / d->chunk_len);
    uint64_t off = 0;
    for (int i = 0; i < n; ++i) {
        uint64_t co, nb;
        int rc = orc_record_layout(d, bits[i], &co, &nb);
        if (rc) return rc;
        if (chunk_ids[i] >= n_chunks) return ORC_ERR_ARG;
        if (off + nb > out_bytes) return ORC_ERR_SMALL;
        meta[i].chunk_id = chunk_ids[i];
        meta[i].bits = bits[i];
        meta[i].offset = off;
        meta[i].nbytes = nb;
        meta[i].n_groups = (uint32_t)groups_per_chunk(d);
        off += nb;
    }
    const int64_t S = n_slabs(d);
    const int CL = d->chunk_len, D = d->head_dim;
    const int64_t slab_elems = (int64_t)CL * D;
    for (int i = 0; i < n; ++i) {
        const int b = bits[i];
        uint64_t co, nb;
        orc_record_layout(d, b, &co, &nb);
        uint8_t *rec = out_buf + meta[i].offset;
        memset(rec, 0, nb);
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
        for (int64_t s_idx = 0; s_idx < S; ++s_idx) {
            const uint16_t *x = kv + slab_base(d, s_idx, chunk_ids[i]);
            uint8_t *codes = (uint8_t *)malloc((size_t)slab_elems);
            if (d->quant_mode == 0) {
                const int G = d->group_size, gpt = D / G;
                for (int t = 0; t < CL; ++t)
                    for (int j = 0; j < gpt; ++j) {
                        uint64_t g = ((uint64_t)s_idx * CL + t) * gpt + j;
                        uint16_t sc, ze;
                        orc_quantize_group(x + (int64_t)t * D + (int64_t)j * G, 1, G, b, &sc, &ze,
                                           codes + (int64_t)t * D + (int64_t)j * G);
                        rec[4 * g + 0] = (uint8_t)(sc & 0xff);
                        rec[4 * g + 1] = (uint8_t)(sc >> 8);
                        rec[4 * g + 2] = (uint8_t)(ze & 0xff);
                        rec[4 * g + 3] = (uint8_t)(ze >> 8);
                    }
            } else {
                uint8_t *col = (uint8_t *)malloc((size_t)CL);
                for (int c = 0; c < D; ++c) {
                    uint64_t g = (uint64_t)s_idx * D + c;
                    uint16_t sc, ze;
                    orc_quantize_group(x + c, D, CL, b, &sc, &ze, col);
                    for (int t = 0; t < CL; ++t) codes[(int64_t)t * D + c] = col[t];
                    rec[4 * g + 0] = (uint8_t)(sc & 0xff);
                    rec[4 * g + 1] = (uint8_t)(sc >> 8);
                    rec[4 * g + 2] = (uint8_t)(ze & 0xff);
                    rec[4 * g + 3] = (uint8_t)(ze >> 8);
                }
                free(col);
            }
            /* a slab's codes start on a byte boundary whenever slab_elems*b is a multiple of 8 */
            if (((uint64_t)slab_elems * b) % 8 == 0) {
                orc_pack_codes(codes, (uint64_t)slab_elems, b, rec + co + (uint64_t)s_idx * slab_elems * b / 8);
            } else {
#ifdef _OPENMP
#pragma omp critical
#endif
                for (int64_t e = 0; e < slab_elems; ++e) {
                    uint64_t bitpos = ((uint64_t)s_idx * slab_elems + e) * b;
                    rec[co + (bitpos >> 3)] |= (uint8_t)(codes[e] << (bitpos & 7));
                }
            }
            free(codes);
        }
        meta[i].checksum = checksum_words(rec, nb);
    }
    return ORC_OK;
}

/* Swap-in decoder (Load's decompression half).  Record i is written to chunk
 * slot dst_ids[i] of kv_out (dst_ids == NULL: meta[i].chunk_id). */
int orc_decompress_chunks(const orc_kv_desc *d, const uint8_t *buf, const orc_chunk_meta *meta,
                          const uint32_t *dst_ids, int n, uint16_t *kv_out)
{
    if (!desc_ok(d) || n < 0) return ORC_ERR_ARG;
    const uint32_t n_chunks = (uint32_t)(d->n_tokens / d->chunk_len);
    const int64_t S = n_slabs(d);
    const int CL = d->chunk_len, D = d->head_dim;
    const int64_t slab_elems = (int64_t)CL * D;
    for (int i = 0; i < n; ++i) {
        const int b = (int)meta[i].bits;
        uint64_t co, nb;
        int rc = orc_record_layout(d, b, &co, &nb);
        if (rc) return rc;
        uint32_t chunk = dst_ids ? dst_ids[i] : meta[i].chunk_id;
        if (chunk >= n_chunks) return ORC_ERR_ARG;
        const uint8_t *rec = buf + meta[i].offset;
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
        for (int64_t s_idx = 0; s_idx < S; ++s_idx) {
            uint16_t *y = kv_out + slab_base(d, s_idx, chunk);
            for (int64_t e = 0; e < slab_elems; ++e) {
                uint64_t bitpos = ((uint64_t)s_idx * slab_elems + e) * b;
                uint8_t q = (uint8_t)((rec[co + (bitpos >> 3)] >> (bitpos & 7)) & ((1u << b) - 1u));
                uint64_t g;
                if (d->quant_mode == 0) {
                    int t = (int)(e / D), c = (int)(e % D);
                    g = ((uint64_t)s_idx * CL + t) * (D / d->group_size) + c / d->group_size;
                } else {
                    g = (uint64_t)s_idx * D + (uint64_t)(e % D);
                }
                uint16_t sc = (uint16_t)(rec[4 * g] | (rec[4 * g + 1] << 8));
                uint16_t ze = (uint16_t)(rec[4 * g + 2] | (rec[4 * g + 3] << 8));
                y[e] = orc_dequantize_one(sc, ze, q);
            }
        }
    }
    return ORC_OK;
}

uint32_t orc_checksum(const uint8_t *p, uint64_t nbytes) { return checksum_words(p, nbytes); }

/* ----------------------------------------------------- Eq. 1: tolerance score */

/* Number of window rows that can see column col.  Row r of a W-row window
 * sits at absolute position T - W + r and sees columns 0..position. */
static int n_visible(int T, int W, int col)
{
    int v = T - col;
    return v < W ? v : W;
}

/* Eq. 1 from attention probabilities.
 * probs[l][h][r][col], l < L, h < Hq, r < W, col < T, binary64; entries with
 * col > T - W + r are masked (ignored, treated as 0).  W = T gives the paper's
 * full lower-triangular R x C matrix.
 *   tok(l,h,col) = (1 / n_vis(col)) * sum over rows that see col of A[r][col]
 *   D_i = mean over the chunk's tokens, layers and heads of tok
 * scores[i], i < floor(T / chunk_len). */
int orc_chunk_tolerance_from_probs(const orc_kv_desc *d, const double *probs, int W, double *scores)
{
    if (!desc_ok(d) || W <= 0 || W > d->n_tokens) return ORC_ERR_ARG;
    const int L = d->n_layers, H = d->n_q_heads, T = d->n_tokens, CL = d->chunk_len;
    const int nc = T / CL;
    for (int i = 0; i < nc; ++i) {
        double over_tokens = 0.0;
        for (int col = i * CL; col < (i + 1) * CL; ++col) {
            double over_layers = 0.0;
            for (int l = 0; l < L; ++l) {
                double over_heads = 0.0;
                for (int h = 0; h < H; ++h) {
                    const double *A = probs + (((int64_t)l * H + h) * W) * (int64_t)T;
                    double colsum = 0.0;
                    for (int r = 0; r < W; ++r)
                        if (col <= T - W + r) colsum += A[(int64_t)r * T + col];
                    over_heads += colsum / (double)n_visible(T, W, col);
                }
                over_layers += over_heads / (double)H;
            }
            over_tokens += over_layers / (double)L;
        }
        scores[i] = over_tokens / (double)CL;
    }
    return ORC_OK;
}

/* A = softmax(mask(Q K^T / sqrt(d_k))) for the last W query positions.
 * q_win[l][h][r][c] binary16 bit patterns; K is the s = 0 half of kv; query
 * head h reads KV head h / (Hq / Hkv).  probs as in the function above. */
int orc_attention_window(const orc_kv_desc *d, const uint16_t *kv, const uint16_t *q_win, int W, double *probs)
{
    if (!desc_ok(d) || W <= 0 || W > d->n_tokens) return ORC_ERR_ARG;
    const int L = d->n_layers, H = d->n_q_heads, T = d->n_tokens, D = d->head_dim;
    const int rep = H / d->n_kv_heads;
    const double inv_sqrt_d = 1.0 / sqrt((double)D);
#ifdef _OPENMP
#pragma omp parallel for collapse(2) schedule(dynamic)
#endif
    for (int l = 0; l < L; ++l)
        for (int h = 0; h < H; ++h) {
            const uint16_t *K = kv + (int64_t)l * d->stride_l + (int64_t)(h / rep) * d->stride_h;
            for (int r = 0; r < W; ++r) {
                const uint16_t *q = q_win + ((((int64_t)l * H + h) * W) + r) * D;
                double *A = probs + ((((int64_t)l * H + h) * W) + r) * (int64_t)T;
                const int pos = T - W + r;
                double mx = -INFINITY;
                for (int col = 0; col <= pos; ++col) {
                    double dot = 0.0;
                    for (int c = 0; c < D; ++c)
                        dot += (double)orc_f16_to_f32(q[c]) * (double)orc_f16_to_f32(K[(int64_t)col * D + c]);
                    A[col] = dot * inv_sqrt_d;
                    if (A[col] > mx) mx = A[col];
                }
                double sum = 0.0;
                for (int col = 0; col <= pos; ++col) { A[col] = exp(A[col] - mx); sum += A[col]; }
                for (int col = 0; col <= pos; ++col) A[col] /= sum;
                for (int col = pos + 1; col < T; ++col) A[col] = 0.0;
            }
        }
    return ORC_OK;
}

/* Eq. 1 from K and the last W queries: the attention window, then the
 * reduction above.  Allocates the L*Hq*W*T window. */
int orc_chunk_tolerance(const orc_kv_desc *d, const uint16_t *kv, const uint16_t *q_win, int W, double *scores)
{
    if (!desc_ok(d) || W <= 0 || W > d->n_tokens) return ORC_ERR_ARG;
    size_t n = (size_t)d->n_layers * d->n_q_heads * W * (size_t)d->n_tokens;
    double *probs = (double *)malloc(n * sizeof(double));
    if (!probs) return ORC_ERR_SMALL;
    int rc = orc_attention_window(d, kv, q_win, W, probs);
    if (!rc) rc = orc_chunk_tolerance_from_probs(d, probs, W, scores);
    free(probs);
    return rc;
}

/* ------------------------------------------------------ Eq. 2: rank -> bits */

/* order_out: chunk indices by density, most informative first (ties: lower
 * index first).  levels = {top, middle, low} bit-widths, e.g. {8, 4, 2}, or
 * {4, 2, 1} atop a 4-bit base (Sec. 3.2).  The first n_top chunks keep the top
 * level, the next n_mid get the middle one, the rest the low one: low density =
 * high tolerance = fewer bits.  Counts round to nearest:
 *   n_top = floor(f_top*n + 1/2), n_top + n_mid = floor((f_top+f_mid)*n + 1/2). */
int orc_assign_levels(const float *scores, int n, const float frac[3], const uint8_t levels[3], uint8_t *bits_out,
                      uint32_t *order_out)
{
    if (n < 0 || !frac || !levels) return ORC_ERR_ARG;
    for (int w = 0; w < 3; ++w)
        if (levels[w] != 1 && levels[w] != 2 && levels[w] != 4 && levels[w] != 8) return ORC_ERR_BITS;
    if (!(levels[0] > levels[1] && levels[1] > levels[2])) return ORC_ERR_ARG;
    double f8 = frac[0], f4 = frac[1], f2 = frac[2];
    if (f8 < 0 || f4 < 0 || f2 < 0 || fabs(f8 + f4 + f2 - 1.0) > 1e-3) return ORC_ERR_ARG;
    uint32_t *ord = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(n > 0 ? n : 1));
    for (int i = 0; i < n; ++i) ord[i] = (uint32_t)i;
    for (int i = 1; i < n; ++i) { /* insertion sort: stable, so equal scores stay in index order */
        uint32_t k = ord[i];
        int j = i - 1;
        while (j >= 0 && scores[ord[j]] < scores[k]) { ord[j + 1] = ord[j]; --j; }
        ord[j + 1] = k;
    }
    long n8 = (long)floor(f8 * n + 0.5);
    long n84 = (long)floor((f8 + f4) * n + 0.5);
    if (n8 > n) n8 = n;
    if (n84 > n) n84 = n;
    if (n84 < n8) n84 = n8;
    for (int r = 0; r < n; ++r) {
        uint8_t b = r < n8 ? levels[0] : (r < n84 ? levels[1] : levels[2]);
        bits_out[ord[r]] = b;
        if (order_out) order_out[r] = ord[r];
    }
    free(ord);
    return ORC_OK;
}

/* Eq. 2 with the levels of the paper's experiments, {8, 4, 2}. */
int orc_assign_bits(const float *scores, int n, const float frac[3], uint8_t *bits_out, uint32_t *order_out)
{
    static const uint8_t k842[3] = {8, 4, 2};
    return orc_assign_levels(scores, n, frac, k842, bits_out, order_out);
}

/* ------------------------------------------------------ Eq. 3: thresholds */

/* Thresholds of Eq. 2 chosen as Eq. 3 asks: maximise the context's information
 *   ctxInfo = sum over levels w of weight_w * (sum of D_i of the chunks at level w)
 * under a global average ratio, for the three levels {8/8, 4/8, 2/8} (Sec. 3.2: with three levels
 * one free variable is left).  Reading: weight_w = ratio_w (a chunk kept at more bits keeps more
 * of its information); the printed 1/ratio_w would reward compressing the densest chunks most.
 * With shares f8 + f4 + f2 = 1 and f8 + f4/2 + f2/4 = R:  f2 = 2*f8 + 2 - 4R.
 * Chunks are taken in density order (as in orc_assign_bits); for every count n8 = 0..n the count
 * n2 = floor(2*n8 + (2 - 4R)*n + 1/2) follows, n4 is the rest, and with prefix sums
 * P[k] = D(rank 0) + ... + D(rank k-1) (added in that order, binary64)
 *   ctxInfo(n8) = P[n8] + (P[n-n2] - P[n8])/2 + (P[n] - P[n-n2])/4.
 * The largest wins, the smaller n8 on a tie.  counts_out = {n8, n4, n2}; frac_out = counts / n. */
int orc_optimize_thresholds_levels(const float *scores, int n, float ratio_global, const uint8_t levels[3],
                                   float frac_out[3], int counts_out[3]);

int orc_optimize_thresholds(const float *scores, int n, float ratio_global, float frac_out[3], int counts_out[3])
{
    static const uint8_t k842[3] = {8, 4, 2};
    return orc_optimize_thresholds_levels(scores, n, ratio_global, k842, frac_out, counts_out);
}

/* The same for any level set {top, middle, low} of bit-widths (Sec. 3.2: the levels are a parameter).  With
 * r1 = middle/top and r2 = low/top the two conditions f0 + f1 + f2 = 1 and f0 + r1*f1 + r2*f2 = R leave
 *   f2 = ((1 - r1)*f0 + r1 - R) / (r1 - r2),
 * so n_low = floor(((1 - r1)*n_top + (r1 - R)*n) / (r1 - r2) + 1/2) for every n_top = 0..n, and
 *   ctxInfo(n_top) = P[n_top] + r1*(P[n-n_low] - P[n_top]) + r2*(P[n] - P[n-n_low]).
 * R in [r2, 1].  For {8, 4, 2} this is the formula above, term by term. */
int orc_optimize_thresholds_levels(const float *scores, int n, float ratio_global, const uint8_t levels[3],
                                   float frac_out[3], int counts_out[3])
{
    if (n <= 0 || !scores || !levels) return ORC_ERR_ARG;
    for (int w = 0; w < 3; ++w)
        if (levels[w] != 1 && levels[w] != 2 && levels[w] != 4 && levels[w] != 8) return ORC_ERR_BITS;
    if (!(levels[0] > levels[1] && levels[1] > levels[2])) return ORC_ERR_ARG;
    const double r1 = (double)levels[1] / (double)levels[0], r2 = (double)levels[2] / (double)levels[0];
    const double R = (double)ratio_global;
    if (!(R >= r2 && R <= 1.0)) return ORC_ERR_ARG;
    uint32_t *ord = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)n);
    double *P = (double *)malloc(sizeof(double) * (size_t)(n + 1));
    for (int i = 0; i < n; ++i) ord[i] = (uint32_t)i;
    for (int i = 1; i < n; ++i) {
        uint32_t k = ord[i];
        int j = i - 1;
        while (j >= 0 && scores[ord[j]] < scores[k]) { ord[j + 1] = ord[j]; --j; }
        ord[j + 1] = k;
    }
    P[0] = 0.0;
    for (int k = 0; k < n; ++k) P[k + 1] = P[k] + (double)scores[ord[k]];
    int best_top = -1, best_low = 0;
    double best = 0.0;
    for (int n_top = 0; n_top <= n; ++n_top) {
        const double x = ((1.0 - r1) * n_top + (r1 - R) * n) / (r1 - r2);
        const long n_low = (long)floor(x + 0.5);
        if (n_low < 0 || n_top + n_low > n) continue;
        const double info = P[n_top] + (P[n - n_low] - P[n_top]) * r1 + (P[n] - P[n - n_low]) * r2;
        if (best_top < 0 || info > best) { best_top = n_top; best_low = (int)n_low; best = info; }
    }
    free(ord);
    free(P);
    if (best_top < 0) return ORC_ERR_ARG;
    counts_out[0] = best_top;
    counts_out[1] = n - best_top - best_low;
    counts_out[2] = best_low;
    for (int w = 0; w < 3; ++w) frac_out[w] = (float)((double)counts_out[w] / (double)n);
    return ORC_OK;
}

/* ------------------------------------------------------------- LCTRU order */

static int lctru_before(const orc_chunk_state *a, const orc_chunk_state *b)
{
    if (a->bits != b->bits) return a->bits > b->bits;                                   /* heavy sub-queue first */
    if (a->last_access_step != b->last_access_step) return a->last_access_step < b->last_access_step; /* least recently used */
    if (a->ctx_id != b->ctx_id) return a->ctx_id < b->ctx_id;
    return a->chunk_id < b->chunk_id;
}

/* Eviction order over resident, unlocked table rows.  order_out receives row
 * indices; returns their count (>= 0) or an error (< 0). */
int orc_lctru_order(const orc_chunk_state *table, int n, uint32_t *order_out)
{
    if (n < 0) return ORC_ERR_ARG;
    int m = 0;
    for (int i = 0; i < n; ++i)
        if (table[i].resident && !table[i].locked) order_out[m++] = (uint32_t)i;
    for (int i = 1; i < m; ++i) {
        uint32_t k = order_out[i];
        int j = i - 1;
        while (j >= 0 && lctru_before(&table[k], &table[order_out[j]])) { order_out[j + 1] = order_out[j]; --j; }
        order_out[j + 1] = k;
    }
    return m;
}

/* Timing aid for the CPU baseline (not part of the method): threads the slab loops may use. */
void orc_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
