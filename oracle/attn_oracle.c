/*
 * Reference ("oracle") implementation of one decode step of paged-KV grouped-query
 * attention, in plain single-threaded C with fp64 arithmetic.
 *
 * THIS IS TEST INFRASTRUCTURE. It exists so that the CUDA library can be checked
 * against something obviously correct; it is slow on purpose, shares no code with
 * the CUDA path, and must never be called from the product path.
 *
 * What is computed. The paper (arXiv 2510.07356, "ConCuR") generates ~9e4 long
 * reasoning traces with 32B-class GQA models (Sec. 3.3; Sec. 4.1 gives the 32,768
 * token limit; Table 3 the trace lengths) but gives no attention formula; the
 * operation is the textbook one, written out as its definition:
 *
 *   for sequence b, query head h, KV head g = h / (Hq/Hkv), n = seq_lens[b]:
 *     token j lives at page = block_table[b][j / P], slot = j % P
 *     s_j   = scale * sum_c q[b][h][c] * K[page][g][slot][c]
 *     m     = max_j s_j ;  w_j = exp(s_j - m) ;  l = sum_j w_j
 *     out_c = (sum_j w_j * V[page][g][slot][c]) / l
 *     lse   = m + ln(l)                       (natural log, scale included)
 *   n == 0  ->  out = 0, lse = -inf.
 *
 * Two passes over a materialised score vector; no online softmax, no blocking,
 * no splitting.  Inputs are bf16 bit patterns (uint16_t) widened exactly to
 * double; `scale` is the caller's fp32 value widened to double.
 *
 * Pins (tests/test_oracle_pins.py): n == 1 returns the V row exactly; constant
 * scores return the mean of V and lse = s + ln n; a geometric-series closed
 * form; the 1/4 : 3/4 two-token case; page-permutation invariance (bit-exact);
 * token-order invariance; shift invariance; split consistency through
 * oracle_lse_merge; convexity bounds; brute force on tiny inputs against a
 * separately written routine; torch fp64 softmax/matmul as a library second
 * opinion.  Every function here is pinned by at least one of those.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t bits) {
    uint32_t w = ((uint32_t)bits) << 16; /* bf16 is the top half of an IEEE fp32 */
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

typedef struct {
    int32_t num_q_heads;   /* Hq  */
    int32_t num_kv_heads;  /* Hkv */
    int32_t head_dim;      /* D   */
    int32_t page_size;     /* P   */
    int32_t block_table_stride; /* ints per block_table row */
} oracle_geom_t;

/* Address of the first element of token j of sequence b, KV head g, in a pool laid
 * out [num_pages][Hkv][P][D]. */
static const uint16_t* kv_row(const uint16_t* pool, const int32_t* block_table,
                              const oracle_geom_t* ge, int32_t b, int32_t g, int64_t j) {
    int64_t page = block_table[(int64_t)b * ge->block_table_stride + j / ge->page_size];
    int64_t slot = j % ge->page_size;
    return pool + ((page * ge->num_kv_heads + g) * ge->page_size + slot) * (int64_t)ge->head_dim;
}

/*
 * Attention of query head h of sequence b over the cached tokens j0 <= j < j1
 * (the definition above restricted to a token range; j0 = 0, j1 = n is the whole
 * operation).  out_bh has D doubles.  An empty range gives out = 0, lse = -inf.
 * Returns 0, or -1 if the score buffer cannot be allocated.
 */
int oracle_attn_range(const uint16_t* q, const uint16_t* k_pages, const uint16_t* v_pages,
                      const int32_t* block_table, const oracle_geom_t* ge, float scale,
                      int32_t b, int32_t h, int64_t j0, int64_t j1,
                      double* out_bh, double* lse_bh) {
    const int32_t D = ge->head_dim;
    const int32_t g = h / (ge->num_q_heads / ge->num_kv_heads);
    const uint16_t* qv = q + ((int64_t)b * ge->num_q_heads + h) * D;
    for (int32_t c = 0; c < D; ++c) out_bh[c] = 0.0;
    if (j1 <= j0) { *lse_bh = -INFINITY; return 0; }

    double* s = (double*)malloc((size_t)(j1 - j0) * sizeof(double));
    if (!s) return -1;

    /* pass 1: scores and their maximum */
    double m = -INFINITY;
    for (int64_t j = j0; j < j1; ++j) {
        const uint16_t* kr = kv_row(k_pages, block_table, ge, b, g, j);
        double dot = 0.0;
        for (int32_t c = 0; c < D; ++c) dot += bf16_to_double(qv[c]) * bf16_to_double(kr[c]);
        s[j - j0] = (double)scale * dot;
        if (s[j - j0] > m) m = s[j - j0];
    }
    /* pass 2: weights, normaliser, weighted sum of V */
    double l = 0.0;
    for (int64_t j = j0; j < j1; ++j) {
        double w = exp(s[j - j0] - m);
        l += w;
        const uint16_t* vr = kv_row(v_pages, block_table, ge, b, g, j);
        for (int32_t c = 0; c < D; ++c) out_bh[c] += w * bf16_to_double(vr[c]);
    }
    for (int32_t c = 0; c < D; ++c) out_bh[c] /= l;
    *lse_bh = m + log(l);
    free(s);
    return 0;
}

/*
 * The whole operation for sequences b_begin <= b < b_end and query heads
 * h_begin <= h < h_end.  out is [batch][Hq][D] doubles, lse is [batch][Hq]
 * doubles; only the selected entries are written.
 */
int oracle_decode_attn(const uint16_t* q, const uint16_t* k_pages, const uint16_t* v_pages,
                       const int32_t* block_table, const int32_t* seq_lens,
                       const oracle_geom_t* ge, float scale,
                       int32_t b_begin, int32_t b_end, int32_t h_begin, int32_t h_end,
                       double* out, double* lse) {
    for (int32_t b = b_begin; b < b_end; ++b)
        for (int32_t h = h_begin; h < h_end; ++h) {
            int64_t idx = (int64_t)b * ge->num_q_heads + h;
            int rc = oracle_attn_range(q, k_pages, v_pages, block_table, ge, scale, b, h, 0,
                                       seq_lens[b], out + idx * ge->head_dim, lse + idx);
            if (rc) return rc;
        }
    return 0;
}

/*
 * Merge of `parts` partial results over disjoint token ranges of one (b, h):
 *   L = ln sum_s exp(lse_s);  out = sum_s exp(lse_s - L) * out_s;  lse = L.
 * A part with lse = -inf (empty range) has weight 0; all parts empty gives
 * out = 0, lse = -inf.  part_out is [parts][D], part_lse is [parts].
 * This is the definition the combine step of a split-KV kernel must reproduce;
 * it is pinned by the split-consistency test (merge of ranges == whole range).
 */
void oracle_lse_merge(const double* part_out, const double* part_lse, int32_t parts, int32_t D,
                      double* out, double* lse) {
    double m = -INFINITY;
    for (int32_t s = 0; s < parts; ++s)
        if (part_lse[s] > m) m = part_lse[s];
    for (int32_t c = 0; c < D; ++c) out[c] = 0.0;
    if (m == -INFINITY) { *lse = -INFINITY; return; }
    double z = 0.0;
    for (int32_t s = 0; s < parts; ++s) z += exp(part_lse[s] - m);
    double L = m + log(z);
    for (int32_t s = 0; s < parts; ++s) {
        if (part_lse[s] == -INFINITY) continue;
        double w = exp(part_lse[s] - L);
        for (int32_t c = 0; c < D; ++c) out[c] += w * part_out[(int64_t)s * D + c];
    }
    *lse = L;
}
