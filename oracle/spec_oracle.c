/*
 * CPU oracle for the SparseSpec-L attention hot path.  TEST INFRASTRUCTURE ONLY:
 * it is imported by the tests, the smoke check and the bench's cpu_baseline /
 * reference arm, never by the product path, and it shares no code with the CUDA
 * library.
 *
 * Everything here is the plain definition written out, in fp64, from the exact
 * values of the bf16 inputs:
 *   - oracle_verify_attn : causal softmax attention of the n_q = k+1 speculated
 *     query rows over the whole dense KV cache ("Full Verification Stage"), plus
 *     the importance score of Eq. 3 (column sum of the attention weights of the
 *     most recent W query rows), aggregated per KV head.
 *   - oracle_select_recall : the index set of Eq. 4 (sink + TopK over the middle
 *     span + recent), ties going to the lower position, emitted ascending.
 *   - oracle_sparse_draft_attn : attention over Gather(K, I), Gather(V, I) of
 *     Eq. 5 plus the dense tail of tokens drafted in the current round.
 *
 * Pin status: verify/statistic, select and draft are pinned by the CPU tests
 * (library fp64 softmax attention, closed forms for identical keys, one-hot
 * limit, brute-force full sort, torch.topk on distinct values, budget >= context
 * reduces draft to dense).  Three readings the paper leaves open are choices and
 * therefore "parity unpinned": aggregation of the score over the GQA group
 * (summed), inclusion of rows of drafts that are later rejected (included), and
 * the values of K_sink / K_recent (parameters).
 *
 * KV cache addressing (shared by all three calls): element (layer, b, pos, h, d)
 * lives at
 *     layer*layer_stride + phys*page_stride + h*head_stride + slot*slot_stride + d
 * with page = pos / page_size, slot = pos % page_size and
 * phys = page_table ? page_table[b*max_pages + page] : b*max_pages + page.
 * Positions are 0-based (the paper counts from 1).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    const void *k, *v; /* bf16 bit patterns, or fp8 (e4m3) bytes when kv_fp8 is set */
    int64_t layer_stride, page_stride, head_stride, slot_stride; /* in elements */
    int32_t n_layers, page_size;
    const int32_t *page_table;
    int32_t max_pages, batch, n_q_heads, n_kv_heads, head_dim;
    double sm_scale; /* <= 0 means 1/sqrt(head_dim) */
    /* 8-bit cache: an element is e4m3 (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; exponent 0 is
     * the denormal range m / 8 * 2^-6; no infinities, S.1111.111 is NaN) times a per-(layer, KV head)
     * scale, k_scale / v_scale [n_layers, n_kv_heads] (NULL: 1).  The attention is then the plain
     * definition on those dequantised values. */
    int32_t kv_fp8;
    const float *k_scale, *v_scale;
} oracle_kv_t;

static double bf16_to_double(uint16_t bits)
{
    uint32_t u = (uint32_t)bits << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double e4m3_to_double(uint8_t b)
{
    const int sign = b >> 7, e = (b >> 3) & 15, m = b & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/* element `off` of K (which = 0) or V (which = 1) of (layer, KV head h), dequantised */
static double kv_elem(const oracle_kv_t *kv, int which, int layer, int h, int64_t off)
{
    const void *base = which ? kv->v : kv->k;
    if (!kv->kv_fp8) return bf16_to_double(((const uint16_t *)base)[off]);
    const float *sc = which ? kv->v_scale : kv->k_scale;
    const double scale = sc ? (double)sc[(int64_t)layer * kv->n_kv_heads + h] : 1.0;
    return e4m3_to_double(((const uint8_t *)base)[off]) * scale;
}

/* decoder exposed for the pins */
double oracle_e4m3_to_double(int byte) { return e4m3_to_double((uint8_t)byte); }

static int64_t kv_row_offset(const oracle_kv_t *kv, int layer, int b, int64_t pos, int h)
{
    int64_t page = pos / kv->page_size, slot = pos % kv->page_size;
    int64_t phys = kv->page_table ? kv->page_table[(int64_t)b * kv->max_pages + page]
                                  : (int64_t)b * kv->max_pages + page;
    return layer * kv->layer_stride + phys * kv->page_stride + h * kv->head_stride +
           slot * kv->slot_stride;
}

static double scale_of(const oracle_kv_t *kv)
{
    return kv->sm_scale > 0.0 ? kv->sm_scale : 1.0 / sqrt((double)kv->head_dim);
}

int oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* scaled logit of one query row against one cached key */
static double logit(const oracle_kv_t *kv, const uint16_t *qrow, int layer, int b, int64_t pos,
                    int h, double scale)
{
    const int64_t krow = kv_row_offset(kv, layer, b, pos, h);
    double s = 0.0;
    for (int d = 0; d < kv->head_dim; ++d) s += bf16_to_double(qrow[d]) * kv_elem(kv, 0, layer, h, krow + d);
    return s * scale;
}

/*
 * Verification attention + Eq. 3 statistic.
 *   q     bf16 [n_layers, batch, n_q, Hq, D]; window row j sits at position ctx_len[b]-n_q+j
 *   out   fp64 [n_layers, batch, n_q, Hq, D]
 *   lse   fp64 [n_layers, batch, n_q, Hq]   (natural log of the softmax denominator), may be NULL
 *   stats fp64 [n_layers, batch, Hkv, stat_stride]; entries [0, ctx_len[b]) written
 * Row j attends keys 0..pos_j (causal, bottom-right aligned).  The statistic sums the
 * probabilities of the last min(W, n_q) rows and of the G query heads that share a KV head.
 */
/* per_head = 0: stats [L, B, Hkv, stat_stride], the score summed over the query heads of a KV head
 * (the reading used by the hot path).  per_head = 1: stats [L, B, Hq, stat_stride], one score per
 * attention head, Eq. 3 as printed ("per-head" indices).  per_head = 2: stats [L, B, Hkv,
 * stat_stride], the LARGEST of the group's per-head scores at every key (the other way to fold the
 * group into one score per KV head; its mass is no longer G * min(W, n_q), see the pins). */
int oracle_verify_attn_ex(const oracle_kv_t *kv, const uint16_t *q, int n_q, const int32_t *ctx_len,
                          int stat_window, double *out, double *lse, double *stats,
                          int64_t stat_stride, int per_head)
{
    const int L = kv->n_layers, B = kv->batch, Hq = kv->n_q_heads, Hkv = kv->n_kv_heads;
    const int D = kv->head_dim, G = Hq / Hkv;
    const int W = stat_window > 0 ? stat_window : 16;
    const int first_stat_row = n_q - (W < n_q ? W : n_q);
    const double scale = scale_of(kv);
    if (Hq % Hkv != 0 || n_q < 1) return -1;
    for (int b = 0; b < B; ++b)
        if (ctx_len[b] < n_q) return -1;

#pragma omp parallel for collapse(3) schedule(dynamic, 1)
    for (int layer = 0; layer < L; ++layer)
        for (int b = 0; b < B; ++b)
            for (int h = 0; h < Hkv; ++h) {
                const int64_t T = ctx_len[b];
                double *p = (double *)malloc(sizeof(double) * (size_t)T);
                /* max over the group: the per-head scores are kept here and folded at the end */
                double *zg = per_head == 2 ? (double *)calloc((size_t)G * (size_t)T, sizeof(double)) : NULL;
                for (int g = 0; g < (per_head == 1 ? G : 1); ++g) {
                    double *z = per_head == 1 ? stats + (((int64_t)layer * B + b) * Hq + h * G + g) * stat_stride
                                         : stats + (((int64_t)layer * B + b) * Hkv + h) * stat_stride;
                    for (int64_t i = 0; i < T; ++i) z[i] = 0.0;
                }
                for (int j = 0; j < n_q; ++j)
                    for (int g = 0; g < G; ++g) {
                        const int qh = h * G + g;
                        double *st = per_head == 1 ? stats + (((int64_t)layer * B + b) * Hq + qh) * stat_stride
                                     : per_head == 2 ? zg + (int64_t)g * T
                                                     : stats + (((int64_t)layer * B + b) * Hkv + h) * stat_stride;
                        const int64_t pos = T - n_q + j; /* last visible key */
                        const int64_t row = (((int64_t)layer * B + b) * n_q + j) * Hq + qh;
                        const uint16_t *qrow = q + row * D;
                        double m = -INFINITY;
                        for (int64_t i = 0; i <= pos; ++i) {
                            p[i] = logit(kv, qrow, layer, b, i, h, scale);
                            if (p[i] > m) m = p[i];
                        }
                        double denom = 0.0;
                        for (int64_t i = 0; i <= pos; ++i) {
                            p[i] = exp(p[i] - m);
                            denom += p[i];
                        }
                        double *o = out + row * D;
                        for (int d = 0; d < D; ++d) o[d] = 0.0;
                        for (int64_t i = 0; i <= pos; ++i) {
                            p[i] /= denom;
                            const int64_t vrow = kv_row_offset(kv, layer, b, i, h);
                            for (int d = 0; d < D; ++d) o[d] += p[i] * kv_elem(kv, 1, layer, h, vrow + d);
                            if (j >= first_stat_row) st[i] += p[i];
                        }
                        if (lse) lse[row] = m + log(denom);
                    }
                if (zg) {
                    double *z = stats + (((int64_t)layer * B + b) * Hkv + h) * stat_stride;
                    for (int64_t i = 0; i < T; ++i) {
                        double best = zg[i];
                        for (int g = 1; g < G; ++g)
                            if (zg[(int64_t)g * T + i] > best) best = zg[(int64_t)g * T + i];
                        z[i] = best;
                    }
                    free(zg);
                }
                free(p);
            }
    return 0;
}

int oracle_verify_attn(const oracle_kv_t *kv, const uint16_t *q, int n_q, const int32_t *ctx_len,
                       int stat_window, double *out, double *lse, double *stats,
                       int64_t stat_stride)
{
    return oracle_verify_attn_ex(kv, q, n_q, ctx_len, stat_window, out, lse, stats, stat_stride, 0);
}

/* ---- Eq. 4: recall selection ------------------------------------------------------------- */

typedef struct {
    float score;
    int32_t pos;
} cand_t;

static int cand_cmp(const void *a, const void *b)
{
    const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
    if (x->score > y->score) return -1;
    if (x->score < y->score) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos); /* equal score: lower position first */
}

static int int_cmp(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

/*
 *   stats   fp32 [n_layers, batch, Hkv, stat_stride]
 *   sel_len int32 [batch]  committed length T' at which the index is built
 *   indices int32 [n_layers, batch, Hkv, k_total] ascending, padded with -1
 *   n_idx   int32 [n_layers, batch, Hkv]
 * T' <= k_total keeps every position.  Otherwise: sink = [0, k_sink),
 * recent = [T'-k_recent, T'), and the k_total-k_sink-k_recent best of the span between them
 * by (score descending, position ascending).
 */
int oracle_select_recall(const float *stats, int64_t stat_stride, int n_layers, int batch,
                         int n_kv_heads, const int32_t *sel_len, int k_sink, int k_recent,
                         int k_total, int32_t *indices, int32_t *n_idx)
{
    const int k_mid = k_total - k_sink - k_recent;
    if (k_sink < 0 || k_recent < 0 || k_mid < 0) return -1;
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
    for (int layer = 0; layer < n_layers; ++layer)
        for (int b = 0; b < batch; ++b)
            for (int h = 0; h < n_kv_heads; ++h) {
                const int64_t prob = ((int64_t)layer * batch + b) * n_kv_heads + h;
                const float *st = stats + prob * stat_stride;
                int32_t *idx = indices + prob * k_total;
                const int32_t T = sel_len[b];
                int n = 0;
                if (T <= k_total) {
                    for (int32_t i = 0; i < T; ++i) idx[n++] = i;
                } else {
                    const int32_t lo = k_sink, hi = T - k_recent; /* candidate span [lo, hi) */
                    cand_t *c = (cand_t *)malloc(sizeof(cand_t) * (size_t)(hi - lo));
                    for (int32_t i = lo; i < hi; ++i) {
                        c[i - lo].score = st[i];
                        c[i - lo].pos = i;
                    }
                    qsort(c, (size_t)(hi - lo), sizeof(cand_t), cand_cmp);
                    for (int32_t i = 0; i < k_sink; ++i) idx[n++] = i;
                    for (int32_t i = 0; i < k_mid; ++i) idx[n++] = c[i].pos;
                    for (int32_t i = T - k_recent; i < T; ++i) idx[n++] = i;
                    free(c);
                    qsort(idx, (size_t)n, sizeof(int32_t), int_cmp);
                }
                n_idx[prob] = n;
                for (int i = n; i < k_total; ++i) idx[i] = -1;
            }
    return 0;
}

/* ---- Eq. 5: sparse draft attention -------------------------------------------------------- */

/*
 *   q   bf16 [n_layers, batch, Hq, D], one drafting query per sequence
 *   key set of (layer, b, kv head h) = indices[layer,b,h,0..n_idx) followed by the dense
 *   tail [tail_start[b], cur_len[b]); softmax is renormalised over exactly that set.
 *   out fp64 [n_layers, batch, Hq, D]; lse fp64 [n_layers, batch, Hq] or NULL
 */
/* per_head = 0: indices [L, B, Hkv, k_total], one set per KV head shared by its query heads.
 * per_head = 1: indices [L, B, Hq, k_total], every attention head gathers its own set (Eq. 5 as
 * printed); K and V still come from the head's KV head. */
int oracle_sparse_draft_attn_ex(const oracle_kv_t *kv, const uint16_t *q, const int32_t *indices,
                                const int32_t *n_idx, int k_total, const int32_t *tail_start,
                                const int32_t *cur_len, double *out, double *lse, int per_head)
{
    const int L = kv->n_layers, B = kv->batch, Hq = kv->n_q_heads, Hkv = kv->n_kv_heads;
    const int D = kv->head_dim, G = Hq / Hkv;
    const double scale = scale_of(kv);
    if (Hq % Hkv != 0) return -1;
#pragma omp parallel for collapse(3) schedule(dynamic, 1)
    for (int layer = 0; layer < L; ++layer)
        for (int b = 0; b < B; ++b)
            for (int h = 0; h < Hkv; ++h) {
                const int n_tail = cur_len[b] > tail_start[b] ? cur_len[b] - tail_start[b] : 0;
                int32_t *keys = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k_total + n_tail + 1));
                double *p = (double *)malloc(sizeof(double) * (size_t)(k_total + n_tail + 1));
                for (int g = 0; g < G; ++g) {
                    const int64_t row = ((int64_t)layer * B + b) * Hq + h * G + g;
                    const int64_t prob = per_head ? row : ((int64_t)layer * B + b) * Hkv + h;
                    const int32_t *idx = indices + prob * k_total;
                    const int n_rec = n_idx[prob];
                    const int n = n_rec + n_tail;
                    for (int i = 0; i < n_rec; ++i) keys[i] = idx[i];
                    for (int i = 0; i < n_tail; ++i) keys[n_rec + i] = tail_start[b] + i;
                    const uint16_t *qrow = q + row * D;
                    double m = -INFINITY, denom = 0.0;
                    for (int i = 0; i < n; ++i) {
                        p[i] = logit(kv, qrow, layer, b, keys[i], h, scale);
                        if (p[i] > m) m = p[i];
                    }
                    for (int i = 0; i < n; ++i) {
                        p[i] = exp(p[i] - m);
                        denom += p[i];
                    }
                    double *o = out + row * D;
                    for (int d = 0; d < D; ++d) o[d] = 0.0;
                    for (int i = 0; i < n; ++i) {
                        const int64_t vrow = kv_row_offset(kv, layer, b, keys[i], h);
                        const double w = p[i] / denom;
                        for (int d = 0; d < D; ++d) o[d] += w * kv_elem(kv, 1, layer, h, vrow + d);
                    }
                    if (lse) lse[row] = n > 0 ? m + log(denom) : -INFINITY;
                }
                free(keys);
                free(p);
            }
    return 0;
}

int oracle_sparse_draft_attn(const oracle_kv_t *kv, const uint16_t *q, const int32_t *indices,
                             const int32_t *n_idx, int k_total, const int32_t *tail_start,
                             const int32_t *cur_len, double *out, double *lse)
{
    return oracle_sparse_draft_attn_ex(kv, q, indices, n_idx, k_total, tail_start, cur_len, out, lse, 0);
}
