/*
 * CPU oracle for the chunk-attention path of HAT's cloud-side middle submodel.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA library is checked against.  It shares no code with the CUDA library,
 * and nothing in the library may call it.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg load it.
 *
 * What it defines (fp64 throughout; 16-bit inputs are widened exactly):
 *
 *   hat_oracle_kv_append        the KV cache store of Sec. 2.1 (KV cache),
 *                               addressed through a block table (the paged
 *                               attention named in Sec. 4.1): logical token p
 *                               of request r lives
 *                               at page block_table[r][p / page_size], slot
 *                               p % page_size.
 *   hat_oracle_attention_rows   scaled dot-product attention (Sec. 2.1, the
 *                               self-attention module of a decoder layer) of
 *                               one query row against the keys it may see:
 *                               all cached tokens of its request plus the
 *                               chunk's own tokens up to and including itself.
 *                               This one mask covers both a prompt chunk
 *                               (Sec. 2.1 Batched Inference; Sec. 3.3) and a draft
 *                               sequence verified in a single inference step
 *                               (Sec. 2.1 Speculative Decoding; Sec. 3.4).
 *   hat_oracle_chunk_attention  the same for every (row, head) of a batch.
 *
 *   Two extensions beyond the paper's own models, both optional:
 *     grouped query heads   num_q_heads = G * num_heads: query head h reads the
 *                           K/V head h / G (the paper's models have G = 1:
 *                           32 and 40 attention heads, Sec. 4.1).
 *     tree_mask             for a chunk of at most 16 rows, word t of tree_mask
 *                           (one per packed row) replaces the causal rule
 *                           INSIDE the chunk: row t sees chunk position c iff
 *                           bit c is set; the cached prefix stays fully
 *                           visible.  This is the token-tree verification of
 *                           the U-Medusa comparison system (Sec. 4.1, tree
 *                           size 8); HAT's own drafts are a linear sequence
 *                           (Sec. 3.4), i.e. the causal rule.  Longer chunks
 *                           are prompt chunks and stay causal.
 *   hat_oracle_merge            combination of attention results computed over
 *                               disjoint key sets (exact identity of softmax;
 *                               not in the paper, used by split-KV kernels).
 *
 * Pins (tests/test_oracle_pins.py): brute-force single-row softmax in pure
 * Python, the Q=0 closed form, chunk-size invariance, draft-verify ==
 * sequential decode, page-permutation invariance, split/merge identity, a
 * library SDPA cross-check.  End-to-end values against the paper: parity
 * unpinned (the paper prints no attention-level numbers).
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { HAT_ORACLE_FP16 = 0, HAT_ORACLE_BF16 = 1 };
enum { HAT_ORACLE_TREE_MAX_ROWS = 16 };

/* IEEE 754 binary16 -> double, exact. */
static double half_bits_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int expo = (h >> 10) & 0x1F;
    int frac = h & 0x3FF;
    double v;
    if (expo == 0)
        v = ldexp((double)frac, -24);              /* subnormal: frac * 2^-10 * 2^-14 */
    else if (expo == 31)
        v = frac ? NAN : INFINITY;
    else
        v = ldexp(1.0 + (double)frac / 1024.0, expo - 15);
    return sign ? -v : v;
}

/* bfloat16 = the upper 16 bits of an IEEE binary32 -> double, exact. */
static double bf16_bits_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double widen(uint16_t bits, int dtype)
{
    return dtype == HAT_ORACLE_BF16 ? bf16_bits_to_double(bits) : half_bits_to_double(bits);
}

/* Exposed so a test can compare all 65536 patterns with an independent decoder. */
double hat_oracle_widen(uint16_t bits, int dtype) { return widen(bits, dtype); }

/* Element offset of (logical token p of request r, head h) inside a pool. */
static int64_t slot_offset(const int32_t *block_table, int max_pages, int page_size,
                           int64_t stride_page, int64_t stride_token, int64_t stride_head,
                           int r, int64_t p, int h)
{
    int32_t page = block_table[(int64_t)r * max_pages + p / page_size];
    int64_t slot = p % page_size;
    return (int64_t)page * stride_page + slot * stride_token + (int64_t)h * stride_head;
}

/*
 * KV append.  For request r and chunk row i (packed row cu_chunk[r] + i), the
 * 16-bit patterns k_new[row][h][:] and v_new[row][h][:] are stored at logical
 * position prefix_len[r] + i.  Slots before prefix_len[r] are not touched;
 * slots at or after it are overwritten (this is how drafts rejected in an
 * earlier round disappear: the caller restarts from the accepted length,
 * Sec. 3.4).
 */
void hat_oracle_kv_append(uint16_t *k_pool, uint16_t *v_pool,
                          int64_t stride_page, int64_t stride_token, int64_t stride_head,
                          int page_size, int num_heads, int head_dim,
                          int num_requests, const int32_t *cu_chunk,
                          const int32_t *prefix_len, const int32_t *chunk_len,
                          const int32_t *block_table, int max_pages,
                          const uint16_t *k_new, const uint16_t *v_new)
{
    for (int r = 0; r < num_requests; ++r) {
        for (int i = 0; i < chunk_len[r]; ++i) {
            int64_t row = (int64_t)cu_chunk[r] + i;
            int64_t p = (int64_t)prefix_len[r] + i;
            for (int h = 0; h < num_heads; ++h) {
                int64_t dst = slot_offset(block_table, max_pages, page_size, stride_page,
                                          stride_token, stride_head, r, p, h);
                int64_t src = (row * num_heads + h) * head_dim;
                for (int c = 0; c < head_dim; ++c) {
                    k_pool[dst + c] = k_new[src + c];
                    v_pool[dst + c] = v_new[src + c];
                }
            }
        }
    }
}

/*
 * One query row.  Keys j in [j_begin, j_end) intersected with the visible set
 * [0, prefix_len[r] + i] are used (pass j_begin = 0, j_end = -1 for "all
 * visible"); K and V rows are fetched through the block table.  With
 *   s_j = sm_scale * <q, k_j>,  m = max_j s_j,  w_j = exp(s_j - m),  l = sum_j w_j
 * the results are  out[c] = sum_j w_j v_j[c] / l  and  lse = m + ln l.
 * An empty key set gives out = 0, lse = -inf.
 */
static void attend_one(const uint16_t *k_pool, const uint16_t *v_pool, int dtype,
                       int64_t stride_page, int64_t stride_token, int64_t stride_head,
                       int page_size, int num_heads, int num_q_heads, int head_dim,
                       const int32_t *cu_chunk, const int32_t *prefix_len, const int32_t *chunk_len,
                       const int32_t *block_table, int max_pages,
                       const uint16_t *q, const uint32_t *tree_mask, double sm_scale,
                       int r, int i, int h, int64_t j_begin, int64_t j_end,
                       double *out, double *lse)
{
    int64_t P = prefix_len[r];
    int64_t visible_end = P + i + 1;                            /* causal: keys 0 .. prefix+i */
    int use_tree = tree_mask != NULL && chunk_len[r] <= HAT_ORACLE_TREE_MAX_ROWS;
    uint32_t bits = 0;
    if (use_tree) {
        bits = tree_mask[(int64_t)cu_chunk[r] + i];
        visible_end = P + chunk_len[r];                         /* any chunk position may be named */
    }
    if (j_begin < 0) j_begin = 0;
    if (j_end < 0 || j_end > visible_end) j_end = visible_end;
    int64_t n = j_end - j_begin;
    for (int c = 0; c < head_dim; ++c) out[c] = 0.0;
    *lse = -INFINITY;
    if (n <= 0) return;

    int group = num_q_heads / num_heads;                        /* query heads per K/V head */
    int hk = h / group;
    const uint16_t *qrow = q + (((int64_t)cu_chunk[r] + i) * num_q_heads + h) * head_dim;
    double *s = (double *)malloc((size_t)n * sizeof(double));
    char *seen = (char *)malloc((size_t)n);

    double m = -INFINITY;
    int64_t count = 0;
    for (int64_t j = j_begin; j < j_end; ++j) {
        seen[j - j_begin] = (char)(!use_tree || j < P || ((bits >> (j - P)) & 1u));
        if (!seen[j - j_begin]) continue;
        int64_t off = slot_offset(block_table, max_pages, page_size, stride_page,
                                  stride_token, stride_head, r, j, hk);
        double dot = 0.0;
        for (int c = 0; c < head_dim; ++c)
            dot += widen(qrow[c], dtype) * widen(k_pool[off + c], dtype);
        s[j - j_begin] = sm_scale * dot;
        if (s[j - j_begin] > m) m = s[j - j_begin];
        ++count;
    }
    if (count > 0) {
        double l = 0.0;
        for (int64_t j = j_begin; j < j_end; ++j) {
            if (!seen[j - j_begin]) continue;
            int64_t off = slot_offset(block_table, max_pages, page_size, stride_page,
                                      stride_token, stride_head, r, j, hk);
            double w = exp(s[j - j_begin] - m);
            l += w;
            for (int c = 0; c < head_dim; ++c)
                out[c] += w * widen(v_pool[off + c], dtype);
        }
        for (int c = 0; c < head_dim; ++c) out[c] /= l;
        *lse = m + log(l);
    }
    free(seen);
    free(s);
}

/*
 * Attention for a list of sampled rows.  sample[5*t + {0,1,2,3,4}] =
 * (request, row within chunk, query head, j_begin, j_end); out is [num_samples,
 * head_dim], lse is [num_samples].  q is [T, num_q_heads, head_dim]; tree_mask
 * is NULL or [T].
 */
void hat_oracle_attention_rows(const uint16_t *k_pool, const uint16_t *v_pool, int dtype,
                               int64_t stride_page, int64_t stride_token, int64_t stride_head,
                               int page_size, int num_heads, int num_q_heads, int head_dim,
                               const int32_t *cu_chunk, const int32_t *prefix_len,
                               const int32_t *chunk_len,
                               const int32_t *block_table, int max_pages,
                               const uint16_t *q, const uint32_t *tree_mask, double sm_scale,
                               int64_t num_samples, const int64_t *sample,
                               double *out, double *lse)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t t = 0; t < num_samples; ++t) {
        const int64_t *sm = sample + 5 * t;
        attend_one(k_pool, v_pool, dtype, stride_page, stride_token, stride_head, page_size,
                   num_heads, num_q_heads, head_dim, cu_chunk, prefix_len, chunk_len, block_table,
                   max_pages, q, tree_mask, sm_scale,
                   (int)sm[0], (int)sm[1], (int)sm[2], sm[3], sm[4],
                   out + t * head_dim, lse + t);
    }
}

/*
 * Attention for every (row, query head) of a batch.  out is [T, num_q_heads,
 * head_dim], lse is [T, num_q_heads], T = cu_chunk[num_requests].  The cache
 * must already hold the chunk's own K/V (append first, then attend).
 */
void hat_oracle_chunk_attention(const uint16_t *k_pool, const uint16_t *v_pool, int dtype,
                                int64_t stride_page, int64_t stride_token, int64_t stride_head,
                                int page_size, int num_heads, int num_q_heads, int head_dim,
                                int num_requests, const int32_t *cu_chunk,
                                const int32_t *prefix_len, const int32_t *chunk_len,
                                const int32_t *block_table, int max_pages,
                                const uint16_t *q, const uint32_t *tree_mask, double sm_scale,
                                double *out, double *lse)
{
    for (int r = 0; r < num_requests; ++r) {
        int64_t units = (int64_t)chunk_len[r] * num_q_heads;
#pragma omp parallel for schedule(dynamic, 1)
        for (int64_t u = 0; u < units; ++u) {
            int i = (int)(u / num_q_heads);
            int h = (int)(u % num_q_heads);
            int64_t row = (int64_t)cu_chunk[r] + i;
            attend_one(k_pool, v_pool, dtype, stride_page, stride_token, stride_head, page_size,
                       num_heads, num_q_heads, head_dim, cu_chunk, prefix_len, chunk_len,
                       block_table, max_pages, q, tree_mask, sm_scale, r, i, h, 0, -1,
                       out + (row * num_q_heads + h) * head_dim, lse + row * num_q_heads + h);
        }
    }
}

/*
 * Merge of attention results over disjoint key sets:
 *   lse = ln sum_s exp(lse_s),   out = sum_s exp(lse_s - lse) * out_s.
 * parts_out is [num_parts, head_dim], parts_lse is [num_parts]; a part with
 * lse = -inf (empty key set) contributes nothing.
 */
void hat_oracle_merge(int num_parts, int head_dim, const double *parts_out,
                      const double *parts_lse, double *out, double *lse)
{
    double m = -INFINITY;
    for (int s = 0; s < num_parts; ++s)
        if (parts_lse[s] > m) m = parts_lse[s];
    for (int c = 0; c < head_dim; ++c) out[c] = 0.0;
    if (m == -INFINITY) { *lse = -INFINITY; return; }
    double l = 0.0;
    for (int s = 0; s < num_parts; ++s) l += exp(parts_lse[s] - m);
    *lse = m + log(l);
    for (int s = 0; s < num_parts; ++s) {
        double w = exp(parts_lse[s] - *lse);
        for (int c = 0; c < head_dim; ++c) out[c] += w * parts_out[(int64_t)s * head_dim + c];
    }
}

/* Number of worker threads the batch entry points use (for the benchmark report). */
#ifdef _OPENMP
#include <omp.h>
int hat_oracle_threads(void) { return omp_get_max_threads(); }
#else
int hat_oracle_threads(void) { return 1; }
#endif
