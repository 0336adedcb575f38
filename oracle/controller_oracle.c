/*
 * CPU oracle for the entropy-guided speculation-length controller of SparseSpec-L
 * (Sec. "Entropy-Based Acceptance Prediction" and "Optimal Length Selection").
 * TEST INFRASTRUCTURE ONLY: imported by the tests, never by the product path; it
 * shares no code with the CUDA library.  Everything is the plain definition in fp64.
 *
 *   - oracle_token_entropy : Shannon entropy (nats) of softmax(logits) over the
 *     vocabulary, one value per row: the "output entropy H_i of each generated
 *     candidate token".
 *   - oracle_controller_update : Eq. "ema".  After a verification that accepted the
 *     first m of k drafted tokens: H_acc = mean entropy of tokens 1..m, H_rej = mean
 *     entropy of tokens m+1..k; each tracked mean moves by
 *     mean <- beta * mean + (1 - beta) * H_class, and only if its class is non-empty.
 *   - oracle_controller_select : Eq. "prob" and Eq. "optimal_k".
 *     p_i = exp(-|H_i - acc|) / (exp(-|H_i - acc|) + exp(-|H_i - rej|));
 *     score(k) = (1 + sum_{m=1..k} prod_{i<=m} p_i) / (k * C_d + C_v);
 *     k* = the candidate with the largest score, the smaller one on ties.
 *
 * Readings the paper leaves open (documented choices, "parity unpinned"): every
 * drafted token after the first rejection counts as rejected; a class that is empty
 * in a step leaves its mean untouched; ties go to the shorter length; entropies are
 * in nats at temperature 1.
 *
 * Pin status: entropy is pinned by closed forms (uniform, two-point, one-hot limit,
 * shift invariance) and by scipy's entropy of a library softmax; update and select by
 * closed forms (equal centres => p = 1/2 => geometric sums; far centres => p -> 1) and
 * by an independent pure-Python evaluation of the equations.
 */
#include <math.h>
#include <stdint.h>

static double bf16_to_double(uint16_t v)
{
    union {
        uint32_t u;
        float f;
    } x;
    x.u = (uint32_t)v << 16;
    return (double)x.f;
}

/* dtype: 0 = fp32 logits, 1 = bf16 logits; row r starts at logits + r * row_stride elements */
int oracle_token_entropy(const void *logits, int dtype, int n_rows, int vocab, int64_t row_stride,
                         double *entropy)
{
    if (!logits || !entropy || n_rows < 0 || vocab < 1 || (dtype != 0 && dtype != 1)) return -1;
    for (int r = 0; r < n_rows; ++r) {
        double m = -INFINITY;
        for (int v = 0; v < vocab; ++v) {
            const double z = dtype == 0 ? (double)((const float *)logits)[r * row_stride + v]
                                        : bf16_to_double(((const uint16_t *)logits)[r * row_stride + v]);
            if (z > m) m = z;
        }
        double denom = 0.0;
        for (int v = 0; v < vocab; ++v) {
            const double z = dtype == 0 ? (double)((const float *)logits)[r * row_stride + v]
                                        : bf16_to_double(((const uint16_t *)logits)[r * row_stride + v]);
            denom += exp(z - m);
        }
        double h = 0.0;
        for (int v = 0; v < vocab; ++v) {
            const double z = dtype == 0 ? (double)((const float *)logits)[r * row_stride + v]
                                        : bf16_to_double(((const uint16_t *)logits)[r * row_stride + v]);
            const double p = exp(z - m) / denom;
            if (p > 0.0) h -= p * log(p);
        }
        entropy[r] = h;
    }
    return 0;
}

/* state[0] = tracked mean entropy of accepted tokens, state[1] = of rejected tokens */
int oracle_controller_update(double *state, const double *entropy, int k, int n_accepted, double beta)
{
    if (!state || !entropy || k < 0 || n_accepted < 0 || n_accepted > k) return -1;
    if (n_accepted > 0) {
        double s = 0.0;
        for (int i = 0; i < n_accepted; ++i) s += entropy[i];
        state[0] = beta * state[0] + (1.0 - beta) * (s / n_accepted);
    }
    if (n_accepted < k) {
        double s = 0.0;
        for (int i = n_accepted; i < k; ++i) s += entropy[i];
        state[1] = beta * state[1] + (1.0 - beta) * (s / (k - n_accepted));
    }
    return 0;
}

/* cand: n_cand candidate lengths, each in 1..n; p_out (n values) and score_out (n_cand) may be NULL */
int oracle_controller_select(const double *state, const double *entropy, int n, const int32_t *cand,
                             int n_cand, double c_d, double c_v, int32_t *k_star, double *p_out,
                             double *score_out)
{
    if (!state || !entropy || !cand || !k_star || n < 1 || n_cand < 1) return -1;
    int best = -1;
    double best_score = -INFINITY;
    for (int c = 0; c < n_cand; ++c) {
        const int k = cand[c];
        if (k < 1 || k > n) return -1;
        double expected = 1.0, prefix = 1.0;
        for (int i = 0; i < k; ++i) {
            const double a = exp(-fabs(entropy[i] - state[0]));
            const double b = exp(-fabs(entropy[i] - state[1]));
            const double p = a / (a + b);
            if (p_out) p_out[i] = p;
            prefix *= p;
            expected += prefix;
        }
        const double score = expected / (k * c_d + c_v);
        if (score_out) score_out[c] = score;
        if (score > best_score || (score == best_score && k < best)) {
            best_score = score;
            best = k;
        }
    }
    if (p_out)
        for (int i = 0; i < n; ++i) {
            const double a = exp(-fabs(entropy[i] - state[0]));
            const double b = exp(-fabs(entropy[i] - state[1]));
            p_out[i] = a / (a + b);
        }
    *k_star = best;
    return 0;
}
