/*
 * fp64 CPU oracle for chunked-prefill attention.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain definition the GPU library is checked against.
 * It shares no code, header, table or constant with the CUDA path and must
 * never be linked into or called from the product library.
 *
 * What it computes (the paper's Eq. 1 with the causal rule of its Transformer
 * background section, applied to one chunk of a chunked prefill as described
 * in its "Chunked Prefill Pipeline Parallelism" background section):
 *
 *   request r has prefix_len P and chunk_len C; query row i (0 <= i < C) of
 *   q-head h sits at absolute position p = P + i and attends to every cached
 *   key j with 0 <= j <= p (itself included) of kv-head g = h / (Hq / Hkv):
 *
 *     s_j  = scale * sum_d Q[r,i,h,d] * K[r,j,g,d]
 *     m    = max_j s_j,   l = sum_j exp(s_j - m)
 *     out  = (1/l) * sum_j exp(s_j - m) * V[r,j,g,:Dv]
 *     lse  = m + ln l
 *
 * All inputs are bf16 bit patterns (uint16) widened exactly to double; every
 * sum runs in double in index order.  No blocking, no online softmax.
 *
 * Pins (tests/test_oracle_pins.py): chunked == unchunked full causal
 * attention, identical keys -> running mean of V, single key -> that V row,
 * split + merge == unsplit, hand-evaluated tiny cases, zero queries, shift
 * invariance, causality, block-table shuffling, and float64
 * torch scaled_dot_product_attention with an explicit mask.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t b)
{
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Address (in elements) of cache row `j` of request `r`, kv-head `g`.
 * Paged: block_table[r][j / B] names the physical block, j % B the slot.
 * Contiguous (block_table == NULL): request r is "block" r and slot = j. */
static int64_t cache_row(const int32_t *block_table, int32_t max_blocks_per_req,
                         int32_t block_size, int64_t block_stride,
                         int64_t token_stride, int64_t head_stride,
                         int32_t r, int64_t j, int32_t g)
{
    int64_t blk, slot;
    if (block_table) {
        blk = block_table[(int64_t)r * max_blocks_per_req + j / block_size];
        slot = j % block_size;
    } else {
        blk = r;
        slot = j;
    }
    return blk * block_stride + slot * token_stride + (int64_t)g * head_stride;
}

/*
 * rows: n_rows triples (request, row-in-chunk, q-head).
 * Keys are restricted to kv_lo <= j < kv_hi as well as j <= p (pass kv_lo = 0,
 * kv_hi < 0 for "all visible keys").  A row with no key in range gets
 * out = 0 and lse = -inf (used only by the split/merge pin).
 * q is packed request-major: rows of request r start at sum_{r'<r} chunk_len[r'].
 * out: double [n_rows, Dv]; lse: double [n_rows].
 * Returns 0, or -1 on an out-of-range row triple.
 */
int ref_chunk_attn_rows(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                        int64_t k_block_stride, int64_t k_token_stride, int64_t k_head_stride,
                        int64_t v_block_stride, int64_t v_token_stride, int64_t v_head_stride,
                        const int32_t *block_table, int32_t max_blocks_per_req, int32_t block_size,
                        const int32_t *prefix_len, const int32_t *chunk_len, int32_t num_reqs,
                        int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim_qk,
                        int32_t head_dim_v, double scale,
                        const int32_t *rows, int64_t n_rows, int64_t kv_lo, int64_t kv_hi,
                        double *out, double *lse)
{
    const int32_t group = num_q_heads / num_kv_heads;
    int64_t *q_start = (int64_t *)malloc(sizeof(int64_t) * (size_t)(num_reqs + 1));
    q_start[0] = 0;
    for (int32_t r = 0; r < num_reqs; ++r) q_start[r + 1] = q_start[r] + chunk_len[r];

    int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t n = 0; n < n_rows; ++n) {
        const int32_t r = rows[3 * n + 0], i = rows[3 * n + 1], h = rows[3 * n + 2];
        if (r < 0 || r >= num_reqs || i < 0 || i >= chunk_len[r] || h < 0 || h >= num_q_heads) {
#pragma omp atomic write
            bad = 1;
            continue;
        }
        const int32_t g = h / group;
        const int64_t p = (int64_t)prefix_len[r] + i;
        const int64_t lo = kv_lo > 0 ? kv_lo : 0;
        int64_t hi = p + 1;
        if (kv_hi >= 0 && kv_hi < hi) hi = kv_hi;
        double *o = out + n * head_dim_v;
        for (int32_t d = 0; d < head_dim_v; ++d) o[d] = 0.0;
        if (hi <= lo) {
            lse[n] = -INFINITY;
            continue;
        }
        const uint16_t *qrow = q + ((q_start[r] + i) * num_q_heads + h) * (int64_t)head_dim_qk;
        double *s = (double *)malloc(sizeof(double) * (size_t)(hi - lo));
        double m = -INFINITY;
        for (int64_t j = lo; j < hi; ++j) {
            const uint16_t *krow = k_cache + cache_row(block_table, max_blocks_per_req, block_size,
                                                       k_block_stride, k_token_stride, k_head_stride, r, j, g);
            double acc = 0.0;
            for (int32_t d = 0; d < head_dim_qk; ++d) acc += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
            s[j - lo] = scale * acc;
            if (s[j - lo] > m) m = s[j - lo];
        }
        double l = 0.0;
        for (int64_t j = lo; j < hi; ++j) {
            const double w = exp(s[j - lo] - m);
            l += w;
            const uint16_t *vrow = v_cache + cache_row(block_table, max_blocks_per_req, block_size,
                                                       v_block_stride, v_token_stride, v_head_stride, r, j, g);
            for (int32_t d = 0; d < head_dim_v; ++d) o[d] += w * bf16_to_double(vrow[d]);
        }
        for (int32_t d = 0; d < head_dim_v; ++d) o[d] /= l;
        lse[n] = m + log(l);
        free(s);
    }
    free(q_start);
    return bad ? -1 : 0;
}

/*
 * Merge of per-split partial results over disjoint key sets:
 *   lse = M + ln sum_s exp(lse_s - M),  M = max_s lse_s
 *   out = sum_s exp(lse_s - lse) * o_s
 * A split with lse_s = -inf (no keys) contributes nothing.  If every split is
 * empty the row gets out = 0, lse = -inf.
 * o_parts: double [S, n, Dv]; lse_parts: double [S, n].
 */
void ref_lse_merge(const double *o_parts, const double *lse_parts, int32_t num_splits,
                   int64_t n, int32_t head_dim_v, double *out, double *lse)
{
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < n; ++t) {
        double M = -INFINITY;
        for (int32_t s = 0; s < num_splits; ++s)
            if (lse_parts[(int64_t)s * n + t] > M) M = lse_parts[(int64_t)s * n + t];
        double *o = out + t * head_dim_v;
        for (int32_t d = 0; d < head_dim_v; ++d) o[d] = 0.0;
        if (M == -INFINITY) {
            lse[t] = -INFINITY;
            continue;
        }
        double z = 0.0;
        for (int32_t s = 0; s < num_splits; ++s) z += exp(lse_parts[(int64_t)s * n + t] - M);
        const double L = M + log(z);
        for (int32_t s = 0; s < num_splits; ++s) {
            const double ls = lse_parts[(int64_t)s * n + t];
            if (ls == -INFINITY) continue;
            const double w = exp(ls - L);
            const double *os = o_parts + ((int64_t)s * n + t) * head_dim_v;
            for (int32_t d = 0; d < head_dim_v; ++d) o[d] += w * os[d];
        }
        lse[t] = L;
    }
}
