/*
 * CPU oracle for the verification stage's prefix acceptance (Sec. "The Draft-Verification
 * Paradigm"): the target model's logits for the k drafted tokens plus one identify the longest
 * accepted prefix x^_{n+1..n+m}; the step commits those m tokens and one corrected token.
 * TEST INFRASTRUCTURE ONLY: imported by the tests, never by the product path; shares no code
 * with the CUDA library.
 *
 * Reading (the paper names "the verification criteria" without fixing them): greedy matching.
 * Row i (0-based) of a sequence's logits is the target distribution of the token that follows
 * drafted token i (row 0 follows the last committed token).  target[i] = argmax of row i, the
 * SMALLEST index among equal maxima.  Drafted token i is accepted iff every earlier one was and
 * draft[i] == target[i]; m = number accepted (0..n_draft); the corrected token is target[m].
 * Rows after m are still reported in target[] (they are the verification pass's output) but do
 * not influence m.  A per-sequence n_draft <= k allows ragged speculation lengths in a batch.
 *
 * Pin status: argmax against a library argmax on tie-free rows and by hand-made ties; the prefix
 * rule by constructed cases (all accepted, none, first mismatch at j, a match after a mismatch
 * that must not count, ragged lengths).
 */
#include <stdint.h>

static double logit_at(const void *logits, int dtype, int64_t i)
{
    if (dtype == 0) return (double)((const float *)logits)[i];
    union {
        uint32_t u;
        float f;
    } x;
    x.u = (uint32_t)((const uint16_t *)logits)[i] << 16;
    return (double)x.f;
}

/* logits: [batch][k1][vocab] with row_stride elements between rows (rows of one sequence and of
 * consecutive sequences are equally spaced); draft: [batch][k1 - 1]; n_draft: [batch] or NULL
 * (= k1 - 1 everywhere); target: [batch][k1]; n_accepted, next_token: [batch]. */
int oracle_accept_greedy(const void *logits, int dtype, int batch, int k1, int vocab, int64_t row_stride,
                         const int32_t *draft, const int32_t *n_draft, int32_t *target,
                         int32_t *n_accepted, int32_t *next_token)
{
    if (!logits || !target || !n_accepted || !next_token || batch < 0 || k1 < 1 || vocab < 1 ||
        (dtype != 0 && dtype != 1) || (k1 > 1 && !draft))
        return -1;
    for (int b = 0; b < batch; ++b) {
        for (int i = 0; i < k1; ++i) {
            const int64_t base = ((int64_t)b * k1 + i) * row_stride;
            int best = 0;
            double best_z = logit_at(logits, dtype, base);
            for (int v = 1; v < vocab; ++v) {
                const double z = logit_at(logits, dtype, base + v);
                if (z > best_z) {
                    best_z = z;
                    best = v;
                }
            }
            target[b * k1 + i] = best;
        }
        const int nd = n_draft ? n_draft[b] : k1 - 1;
        if (nd < 0 || nd > k1 - 1) return -1;
        int m = 0;
        while (m < nd && draft[b * (k1 - 1) + m] == target[b * k1 + m]) ++m;
        n_accepted[b] = m;
        next_token[b] = target[b * k1 + m];
    }
    return 0;
}
