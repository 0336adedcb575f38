/*
 * spec_attn.h - C ABI of the B200 (sm_100a) attention hot path of SparseSpec-L
 * train-free self-speculative decoding.
 *
 * One decode iteration of the method drafts k tokens with sparse attention over a
 * recallable subset of the KV cache and then verifies them in one dense pass
 * ("Sparse Drafting Stage" / "Full Verification Stage", Sec. 3.1).  This library holds the
 * three data-parallel attention-side steps of that iteration:
 *
 *   spec_verify_attn        dense verification attention of the k+1 speculated rows over the
 *                           whole cache, with the importance score of Eq. 3 produced in the
 *                           same pass;
 *   spec_select_recall      the index set of Eq. 4 (sink + TopK over the middle span + recent);
 *   spec_sparse_draft_attn  attention over Gather(K, I), Gather(V, I) of Eq. 5, the gather
 *                           fused into the attention (the gathered copies are never
 *                           materialised), plus the dense tail of tokens drafted this round.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless it says "host".  The caller owns every buffer,
 *     including the workspace; the library allocates no device memory, never frees anything
 *     and never writes K or V (the dense cache stays resident, Sec. 3.2).
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronising.  Lengths live in device arrays.
 *   - Return value: 0 on success, a negative SPEC_ERR_* decided on the host BEFORE anything
 *     is launched.  Device-side anomalies (an out-of-range recall index, a bounded wait that
 *     ran out) set a status word at the head of the workspace and the kernel exits cleanly;
 *     read it with spec_read_status().  Workspaces must be zero-filled once after allocation;
 *     no call clears the status word, reading it does.
 *   - Positions are 0-based (the paper counts from 1).  bf16 inputs, fp32 accumulation and
 *     fp32 outputs.
 *   - GQA: query head hq reads KV head hq / (n_q_heads / n_kv_heads); the Eq. 3 score is kept
 *     per KV head, summed over the query heads that share it.
 *   - "problem" = one (layer, sequence, KV head); n_layers > 1 folds independent layers that
 *     share shapes into one launch.
 */
#ifndef SPEC_ATTN_H_
#define SPEC_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    SPEC_OK = 0,
    SPEC_ERR_INVALID_ARG = -1,         /* null pointer, negative size, inconsistent fields */
    SPEC_ERR_UNSUPPORTED_SHAPE = -2,   /* head_dim not 64/128, too many rows per KV head, ... */
    SPEC_ERR_WORKSPACE_TOO_SMALL = -3, /* workspace_bytes < spec_workspace_bytes(...) */
    SPEC_ERR_CUDA = -4,                /* a CUDA runtime/driver call failed at launch time */
    SPEC_ERR_TIMEOUT = -5,             /* status word: a bounded device-side wait ran out */
    SPEC_ERR_BAD_INDEX = -6            /* status word: a recall index, page-table entry or length was out of range */
};

/* Which entry point a workspace is sized for. */
enum { SPEC_WS_VERIFY = 0, SPEC_WS_SELECT = 1, SPEC_WS_DRAFT = 2 };

/* Verification kernel choice for spec_set_verify_impl(). */
enum {
    SPEC_VERIFY_AUTO = 0,             /* tcgen05 when the shape allows it, else generic */
    SPEC_VERIFY_GENERIC = 1,          /* plain FP32 CUDA-core kernels, every supported shape */
    SPEC_VERIFY_TCGEN05 = 2,          /* tcgen05, either variant; unsupported shapes are an error */
    SPEC_VERIFY_TCGEN05_TWOSWEEP = 3, /* K swept twice (second sweep from L2), any context length */
    SPEC_VERIFY_TCGEN05_CACHED = 4,   /* score tiles cached in tensor memory, K and V read once */
    SPEC_VERIFY_TCGEN05_CACHED_2PASS = 5, /* reported only (spec_last_verify_impl): AUTO ran the score-cache kernel
                                             on two halves of the rows because all rows did not fit the cache */
    SPEC_VERIFY_TCGEN05_CACHED_EXPANDED = 6 /* reported only: an 8-bit cache was first expanded to bf16 in the
                                               workspace (the score-cache kernel could not read its bytes itself:
                                               head_dim 64) */
};

/*
 * Dense KV cache of one or more layers (the K_{l,h}, V_{l,h} of Eq. 5), READ-ONLY.
 * Element (layer, b, pos, h, d) of K lives at
 *     k + layer*layer_stride + phys*page_stride + h*head_stride + slot*slot_stride + d
 * with page = pos / page_size, slot = pos % page_size and
 *     phys = page_table ? page_table[b*max_pages + page] : b*max_pages + page.
 * Strides are in elements; d is contiguous; every stride must be a multiple of 8 elements and
 * k, v 16-byte aligned.  A contiguous per-sequence cache is the case max_pages == 1.
 */
typedef struct {
    const void* k;                 /* bf16 */
    const void* v;                 /* bf16 */
    int64_t layer_stride, page_stride, head_stride, slot_stride;
    int32_t n_layers;              /* >= 1 */
    int32_t page_size;             /* tokens per page, >= 1 */
    const int32_t* page_table;     /* device int32 [batch, max_pages] or NULL */
    int32_t max_pages, batch, n_q_heads, n_kv_heads;
    int32_t head_dim;              /* 64 or 128 */
    int32_t n_pages;               /* physical pages in the pool (bounds page_table entries);
                                      0 means batch * max_pages */
    float sm_scale;                /* softmax scale; <= 0 means 1/sqrt(head_dim) */
    int32_t kv_dtype;              /* SPEC_KV_BF16 (0) or SPEC_KV_FP8_E4M3: k and v hold e4m3 bytes (1 sign, 4
                                      exponent bits with bias 7, 3 mantissa bits, no infinities), same
                                      addressing rule with strides in elements (= bytes), every stride a
                                      multiple of 16 */
    const float* k_scale;          /* SPEC_KV_FP8_E4M3: device fp32 [n_layers, n_kv_heads], an element's value */
    const float* v_scale;          /* is its e4m3 value times the (layer, KV head) scale; NULL means 1 */
} spec_kv_t;

/* Element type of the cache.  With SPEC_KV_FP8_E4M3 (the decode step is bound by loading the cache:
 * Sec. 1, so an 8-bit cache halves the bytes of every call) Q stays bf16 and all results are those of
 * the same attention on the dequantised values.  Served by the sparse draft attention kernel
 * (tensor cores on fp16 copies of the rows, which hold e4m3 values exactly; Q is converted to fp16:
 * exact for magnitudes in [6.1e-5, 65504], absolute error <= 3e-8 below that).  Verification at
 * head_dim 128: the tensor-core score-cache kernel streams the bytes and expands each tile to fp16 in
 * shared memory (exact), with fp16 copies of Q (same range as above) and of the probabilities (two
 * fp16 terms: relative error below 2^-21), K's scale multiplied into the softmax scale and V's into the
 * output.  At head_dim 64 the pages the contexts reach are first expanded to bf16 (exact, scales left
 * out) in the tail of the workspace and streamed by the same kernel's bf16 instances;
 * spec_workspace_bytes(SPEC_WS_VERIFY, ...) of an 8-bit cache therefore includes 4 bytes per cache
 * element of the view (K and V).  A workspace without that room (at least the size for the same view
 * as bf16), a layout whose pages or layers interleave, a per-attention-head or group-max statistic,
 * or a shape outside the score-cache kernel runs the generic FP32 kernels on the bytes instead
 * (correct, many times slower). */
enum { SPEC_KV_BF16 = 0, SPEC_KV_FP8_E4M3 = 1 };

/*
 * Full-context verification attention + importance score (Sec. 3.1 "Full Verification
 * Stage"; Eq. 3).
 *
 * Row j (0 <= j < n_q) of sequence b sits at position ctx_len[b]-n_q+j and attends keys
 * 0..that position of the whole dense cache (causal inside the window).  out = softmax(q K^T *
 * sm_scale) V.  stats[layer,b,h,i] = sum over the last min(stat_window, n_q) rows j and over
 * the query heads of KV head h of the attention probability row j gives key i (0 where
 * masked).  Probabilities use the global softmax normaliser, so each contributing row adds
 * exactly 1 to the sum of stats over i.
 *
 *   q        bf16 [n_layers, batch, n_q, n_q_heads, head_dim]
 *   n_q      k+1, 1..32, with n_q * (n_q_heads/n_kv_heads) <= 128
 *   ctx_len  int32 [batch], each n_q <= ctx_len[b] <= max_ctx_len; INCLUDES the n_q rows, whose
 *            K/V are already in the cache.  A value outside that range is clamped into it on the
 *            device and sets SPEC_ERR_BAD_INDEX in the status word (no access leaves the buffers)
 *   max_ctx_len  host upper bound of ctx_len (sizes the launch)
 *   stat_window  W of Eq. 3; 0 means 16
 *   out      fp32 [n_layers, batch, n_q, n_q_heads, head_dim]
 *   lse      fp32 [n_layers, batch, n_q, n_q_heads] (natural-log softmax denominator) or NULL
 *   stats    fp32 [n_layers, batch, n_kv_heads, stat_stride]; entries [0, ctx_len[b]) are
 *            written, the rest left untouched; stat_stride >= max_ctx_len
 *   workspace  >= spec_workspace_bytes(SPEC_WS_VERIFY, ...) bytes, 256-byte aligned, ZERO-FILLED
 *            once before its first use (cudaMemset); every call leaves it ready for the next one
 *            (no per-call memset: the kernel's last CTA puts its cross-CTA counters back to
 *            zero).  The status word is sticky until spec_read_status() returns it; after
 *            SPEC_ERR_TIMEOUT zero the workspace again.  Must not be shared by calls that may
 *            overlap on the GPU.
 */
int spec_verify_attn(const spec_kv_t* kv, const void* q, int32_t n_q, const int32_t* ctx_len,
                     int32_t max_ctx_len, int32_t stat_window, float* out, float* lse,
                     float* stats, int64_t stat_stride, void* workspace, size_t workspace_bytes,
                     void* cuda_stream);

/*
 * spec_verify_attn with option flags.  SPEC_VERIFY_ACCUMULATE_STATS: the statistic of this call
 * is ADDED to what stats[layer, b, h, 0:ctx_len[b]) already holds instead of replacing it, so that
 * the window of Eq. 3 can span the rows of several verification passes when one pass has fewer
 * than W rows (the caller keeps the running sums: zero-fill before the first pass, and subtract or
 * restart when rows leave the window; positions appended since the previous pass must hold 0).
 * Two passes over the same cache whose rows are consecutive, the second with the flag set,
 * give the statistic of one pass over all their rows (with W >= the total).  flags == 0 is
 * spec_verify_attn.  Unknown flag bits: SPEC_ERR_INVALID_ARG.
 *
 * SPEC_VERIFY_STATS_PER_QUERY_HEAD: Eq. 3 as printed, one score per attention head: stats is
 * fp32 [n_layers, batch, n_q_heads, stat_stride] and head hq's entry sums the probabilities of
 * hq's own window rows only (the default sums them over the query heads of a KV head).  The
 * per-KV-head statistic is the sum of its group's per-head statistics.  Served by the score-cache
 * tcgen05 kernel for groups of up to 8 heads whose shape fits its cache, else by the generic
 * kernels.  spec_select_recall then runs with n_kv_heads = n_q_heads, and the draft call takes
 * SPEC_DRAFT_INDICES_PER_QUERY_HEAD.
 *
 * SPEC_VERIFY_STATS_GROUP_MAX: stats keeps its per-KV-head shape, but a key's score is the LARGEST
 * of its group's per-head scores (each the Eq. 3 sum over that head's window rows) instead of their
 * sum: the other way to fold a grouped-query group into one ranking.  Each head's mass is 1 per
 * window row, so the summed form has mass G per row and this one anything between 1 and G.  Same
 * kernels and limits as SPEC_VERIFY_STATS_PER_QUERY_HEAD; the two flags exclude each other.
 *
 * SPEC_VERIFY_OUT_BF16: `out` points to bf16 elements of the same shape (the fp32 result rounded to
 * nearest even: what a bf16 output projection consumes); lse and stats stay fp32.
 */
enum { SPEC_VERIFY_ACCUMULATE_STATS = 1, SPEC_VERIFY_STATS_PER_QUERY_HEAD = 2, SPEC_VERIFY_OUT_BF16 = 4,
       SPEC_VERIFY_STATS_GROUP_MAX = 8 };
int spec_verify_attn_ex(const spec_kv_t* kv, const void* q, int32_t n_q, const int32_t* ctx_len,
                        int32_t max_ctx_len, int32_t stat_window, float* out, float* lse,
                        float* stats, int64_t stat_stride, void* workspace, size_t workspace_bytes,
                        uint32_t flags, void* cuda_stream);

/*
 * spec_verify_attn_ex that also hands the selection its first radix pass (Eq. 4 picks the largest
 * scores; the selection kernel finds the K-th largest by a radix select on the scores' fp32 bit
 * patterns, whose first pass is a histogram of the top 11 bits).  score_hist: uint32
 * [n_layers, batch, heads, 2048] (heads = n_kv_heads, or n_q_heads with
 * SPEC_VERIFY_STATS_PER_QUERY_HEAD), ZERO-FILLED once after allocation; this call ADDS, for every
 * score stats[.., i] it writes (i < ctx_len[b]), one count to bin (bit pattern >> 21) of the
 * value written.  spec_select_recall_hist consumes the counts and clears them, so a
 * verify / select pair leaves the array zero again.  The score-cache kernel counts while it writes
 * the statistic (one fire-and-forget reduction per key); every other verification path runs a short
 * sweep over the finished statistic instead.  score_hist == NULL is spec_verify_attn_ex.
 */
int spec_verify_attn_hist(const spec_kv_t* kv, const void* q, int32_t n_q, const int32_t* ctx_len,
                          int32_t max_ctx_len, int32_t stat_window, float* out, float* lse,
                          float* stats, int64_t stat_stride, void* workspace, size_t workspace_bytes,
                          uint32_t flags, uint32_t* score_hist, void* cuda_stream);

/*
 * Recall selection (Eq. 4).  For each problem with T' = sel_len[b]:
 *   T' <= k_total : indices = 0..T'-1, n = T'.
 *   otherwise     : sink [0,k_sink) U the k_mid = k_total-k_sink-k_recent positions of
 *                   [k_sink, T'-k_recent) with the largest stats (equal stats: the lower
 *                   position wins) U recent [T'-k_recent, T'); n = k_total.
 * Output ascending, padded with -1.  stats must be finite and >= 0 (they are sums of
 * probabilities), which makes the fp32 bit pattern order-isomorphic to the value; the result
 * is a pure function of the stats bits, so it is reproducible bit for bit.
 *
 *   stats     fp32 [n_layers, batch, n_kv_heads, stat_stride]
 *   sel_len   int32 [batch], committed length T' (<= stat_stride); positions >= T' are ignored
 *   indices   int32 [n_layers, batch, n_kv_heads, k_total]
 *   n_indices int32 [n_layers, batch, n_kv_heads]
 *   workspace unused at present (may be NULL, 0)
 */
int spec_select_recall(const float* stats, int64_t stat_stride, int32_t n_layers, int32_t batch,
                       int32_t n_kv_heads, const int32_t* sel_len, int32_t k_sink,
                       int32_t k_recent, int32_t k_total, int32_t* indices, int32_t* n_indices,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * spec_select_recall fed with the counts of spec_verify_attn_hist.  score_hist: uint32
 * [n_layers, batch, n_kv_heads, 2048] as that call left it; hist_len: int32 [batch], the ctx_len of
 * that call (the counts cover positions [0, hist_len[b]) of stats).  The kernel removes the
 * positions outside the candidate span from the counts, skips its own first sweep over the
 * scores, and writes zeros back to score_hist.  The result is the same, bit for bit, as
 * spec_select_recall on the same stats.  A sequence with sel_len[b] > hist_len[b] falls back to
 * the full sweep.  score_hist and hist_len are both NULL (= spec_select_recall) or both given.
 */
int spec_select_recall_hist(const float* stats, int64_t stat_stride, int32_t n_layers, int32_t batch,
                            int32_t n_kv_heads, const int32_t* sel_len, int32_t k_sink,
                            int32_t k_recent, int32_t k_total, int32_t* indices, int32_t* n_indices,
                            uint32_t* score_hist, const int32_t* hist_len, void* workspace,
                            size_t workspace_bytes, void* cuda_stream);

/*
 * Sparse draft attention (Eq. 5; Sec. 3.1 "Sparse Drafting Stage").  One query per sequence.
 * Key set of (layer, b, KV head h) = indices[layer,b,h,0..n_indices) U the dense tail
 * [tail_start[b], cur_len[b]) (tokens drafted in the current round, the query's own position
 * included); softmax is renormalised over exactly that set.  Rows are read straight from the
 * dense cache by index.
 *
 *   q          bf16 [n_layers, batch, n_q_heads, head_dim]
 *   indices    int32 [n_layers, batch, n_kv_heads, k_total], entries < tail_start[b]; unique
 *   n_indices  int32 [n_layers, batch, n_kv_heads], 0..k_total
 *   tail_start int32 [batch]; cur_len int32 [batch], cur_len - tail_start <= max_tail
 *   max_tail   host upper bound of the tail length (sizes the launch)
 *   out        fp32 [n_layers, batch, n_q_heads, head_dim]; lse fp32 [n_layers,batch,n_q_heads]
 *              or NULL
 *   workspace  >= spec_workspace_bytes(SPEC_WS_DRAFT, ...) bytes, 256-byte aligned.  It holds
 *              only the status word, which this call never clears (one launch per call, no
 *              memset): zero it once after allocation; an error stays until
 *              spec_read_status() returns it.
 * An index outside [0, cur_len[b]), or a page-table entry outside [0, n_pages), is skipped and
 * sets SPEC_ERR_BAD_INDEX in the status word; so does a cur_len[b] beyond max_pages * page_size
 * (clamped to it) and a tail longer than max_tail (the rows beyond max_tail are dropped).
 * The one device-side wait (the first CTA of a cluster waiting for the partial results of the
 * others) is bounded; if it runs out the status word gets SPEC_ERR_TIMEOUT.
 * A problem with an empty key set yields out = 0, lse = -inf.
 * Limits: n_q_heads / n_kv_heads <= 8 (SPEC_ERR_UNSUPPORTED_SHAPE otherwise; with
 * SPEC_DRAFT_INDICES_PER_QUERY_HEAD every head is its own group of one, so any ratio works);
 * n_pages * page_stride < 2^35 elements (one layer's K below 64 GiB).
 * Stream order: the call reads all of its inputs only after every earlier kernel of the stream
 * has completed, unless SPEC_DRAFT_EARLY_GATHER is given (spec_sparse_draft_attn_ex).
 */
int spec_sparse_draft_attn(const spec_kv_t* kv, const void* q, const int32_t* indices,
                           const int32_t* n_indices, int32_t k_total, const int32_t* tail_start,
                           const int32_t* cur_len, int32_t max_tail, float* out, float* lse,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Verification attention without a caller-provided workspace.  The paper has no counterpart;
 * this entry point exists for hosts that cannot allocate device memory themselves: a plugin
 * running inside a runtime that owns every device buffer and hands in only inputs and
 * outputs, or code that starts after a framework's memory pool has taken the whole GPU.
 *
 * Same arguments, results and error codes as spec_verify_attn, minus the workspace.  The
 * scratch is a fixed array inside the library image: spec_noalloc_scratch_bytes() bytes
 * (16 MiB) on every GPU that loads the library, held until the process exits.  The call
 * allocates and frees nothing.
 *   - A shape whose spec_workspace_bytes(SPEC_WS_VERIFY, ...) exceeds that size is refused with
 *     SPEC_ERR_WORKSPACE_TOO_SMALL before anything is launched.
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress, with that device current); make that first call before starting any
 *     stream capture on the device.
 *   - `cuda_stream` must belong to the device that is current at the call (the array's address is
 *     looked up for the current device).
 *   - All calls on a device share the one array, and it keeps the previous call's contents;
 *     every call re-zeroes the control words it depends on, on `cuda_stream`; the status word is
 *     kept until spec_noalloc_read_status() returns it.  Two calls that
 *     may overlap on the GPU (different streams, no ordering) race on it: serialise them.
 *   - spec_noalloc_read_status() is spec_read_status() on that array for the current device.
 */
int spec_verify_attn_noalloc(const spec_kv_t* kv, const void* q, int32_t n_q,
                             const int32_t* ctx_len, int32_t max_ctx_len, int32_t stat_window,
                             float* out, float* lse, float* stats, int64_t stat_stride,
                             void* cuda_stream);
size_t spec_noalloc_scratch_bytes(void);
int spec_noalloc_read_status(void* cuda_stream);

/*
 * Speculation-length controller (Sec. "Entropy-Based Acceptance Prediction" and "Optimal
 * Length Selection").  Every pointer except `cuda_stream` is DEVICE memory owned by the
 * caller; nothing is allocated, nothing synchronises, results stay on the device (a captured
 * graph can hold all three calls).  Arithmetic is fp32.
 *
 * spec_token_entropy: entropy[r] = Shannon entropy in nats of softmax(logits[r, 0:vocab]) at
 *   temperature 1: the H_i of each drafted token.  dtype 0 = fp32 logits, 1 = bf16 logits; row
 *   r starts `row_stride` ELEMENTS after row r - 1 (>= vocab).  One pass over the logits.
 *   Errors: SPEC_ERR_INVALID_ARG (null pointer, vocab < 1, n_rows < 0, stride < vocab, dtype).
 *
 * spec_controller_update: Eq. "ema".  entropy[0:k] are the entropies of the k tokens drafted
 *   in the step that was just verified, *n_accepted (clamped to 0..k) how many of them were
 *   accepted.  state[0] (tracked mean of accepted tokens) moves to
 *   beta * state[0] + (1 - beta) * mean(entropy[0:m]) when m > 0; state[1] (rejected tokens)
 *   likewise with entropy[m:k] when m < k.  Tokens after the first rejection count as rejected.
 *
 * spec_controller_select: Eq. "prob" and Eq. "optimal_k".  p_i = e^-|H_i - state[0]| /
 *   (e^-|H_i - state[0]| + e^-|H_i - state[1]|) for the n <= 256 entropies given;
 *   score(k) = (1 + sum_{m=1..k} prod_{i<=m} p_i) / (k * c_d + c_v) for each of the n_cand
 *   candidate lengths cand[c] in 1..n (a candidate outside that range scores -1 and never
 *   wins); *k_star = the candidate with the largest score, the smaller one on equal scores
 *   (0 if no candidate is valid).  p_out (n floats) and score_out (n_cand floats) may be NULL.
 *   Errors: SPEC_ERR_INVALID_ARG, SPEC_ERR_UNSUPPORTED_SHAPE (n > 256).
 */
int spec_token_entropy(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                       int64_t row_stride, float* entropy, void* cuda_stream);
/*
 * spec_token_argmax: token[r] = the smallest index of the largest logit of row r (greedy
 *   decoding of that row); if `entropy` is not NULL it also receives spec_token_entropy's value
 *   from the same pass over the logits (a drafting step needs both).  Same layout and errors as
 *   spec_token_entropy; n_rows <= 65535.
 *
 * spec_accept_greedy: the verification stage's prefix acceptance (Sec. "The Draft-Verification
 *   Paradigm") under greedy matching.  logits: [batch][k1][vocab], rows `row_stride` elements
 *   apart across the whole batch, row i of a sequence being the target model's output after
 *   drafted token i (row 0 after the last committed token).  draft: [batch][k1 - 1] drafted
 *   tokens; n_draft: [batch] drafted tokens actually present per sequence (clamped to
 *   0..k1 - 1), or NULL for k1 - 1 everywhere.  Outputs: target[batch][k1] = greedy token of
 *   every row; n_accepted[b] = m = length of the longest prefix with draft[b][i] == target[b][i];
 *   next_token[b] = target[b][m], the corrected token the step commits after the prefix.
 *   Integer results, bit-exact.  Two launches (row argmax, prefix scan) on `cuda_stream`.
 *   Errors: SPEC_ERR_INVALID_ARG; SPEC_ERR_UNSUPPORTED_SHAPE if batch * k1 > 65535.
 */
int spec_token_argmax(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab,
                      int64_t row_stride, int32_t* token, float* entropy, void* cuda_stream);
int spec_accept_greedy(const void* logits, int32_t dtype, int32_t batch, int32_t k1, int32_t vocab,
                       int64_t row_stride, const int32_t* draft, const int32_t* n_draft,
                       int32_t* target, int32_t* n_accepted, int32_t* next_token,
                       void* cuda_stream);
/*
 * spec_advance_lengths: the bookkeeping between two speculation rounds, on the device so that a
 * captured graph can run round after round (Sec. "The Draft-Verification Paradigm": a step commits
 * the m accepted tokens and one corrected token).  committed[b] += clamp(n_accepted[b], 0, k) + 1
 * (n_accepted == NULL: committed is left as it is); then, for the round that follows with k drafted
 * tokens, ctx_verify[b] = committed[b] + k + 1 (the ctx_len of its verification pass, rows included)
 * and cur_len[j][b] = committed[b] + j + 1 for j < k (the cur_len of its j-th drafting step, whose
 * tail starts at committed[b]).  ctx_verify and cur_len (int32 [k][batch]) may be NULL.
 * max_len > 0 is the number of tokens a sequence's cache can hold (the max_ctx_len later calls are
 * sized for): a sequence whose next round would not fit (committed + k + 1 > max_len) is held at
 * max_len - k - 1 instead and SPEC_ERR_BAD_INDEX is recorded in the status word at the head of
 * `workspace` (any workspace of this library; NULL: not recorded).  max_len == 0: no bound.
 */
int spec_advance_lengths(int32_t* committed, const int32_t* n_accepted, int32_t batch, int32_t k,
                         int32_t max_len, void* workspace, int32_t* ctx_verify, int32_t* cur_len,
                         void* cuda_stream);
int spec_controller_update(float* state, const float* entropy, int32_t k,
                           const int32_t* n_accepted, float beta, void* cuda_stream);
int spec_controller_select(const float* state, const float* entropy, int32_t n,
                           const int32_t* cand, int32_t n_cand, float c_d, float c_v,
                           int32_t* k_star, float* p_out, float* score_out, void* cuda_stream);

/*
 * spec_sparse_draft_attn with option flags.  SPEC_DRAFT_INDICES_PER_QUERY_HEAD: Eq. 5 as printed,
 * every attention head gathers its own index set: indices is int32 [n_layers, batch, n_q_heads,
 * k_total] and n_indices int32 [n_layers, batch, n_q_heads]; K and V rows still come from the
 * head's KV head (hq / group).  The gathered bytes grow by the group size.
 * SPEC_DRAFT_OUT_BF16: `out` points to bf16 elements (fp32 result rounded to nearest even).
 * SPEC_DRAFT_EARLY_GATHER: the kernel is launched so that it may start while the preceding kernel
 * of the stream is still running, and it reads indices, n_indices, tail_start, cur_len, the page
 * table and the recalled K/V rows BEFORE that kernel has finished; only q, the rows of the dense
 * tail and the outputs wait for the stream's earlier work.  Give the flag only when those
 * early-read arguments were complete before the preceding kernel of the stream STARTED: true for
 * every call of a drafting round but the first one that follows the producers of the index sets and
 * the lengths (selection, the length bookkeeping), since nothing changes them during a round.
 * Without the flag the call starts after all earlier work of the stream, like any kernel.
 * flags == 0 is spec_sparse_draft_attn.  Unknown flag bits: SPEC_ERR_INVALID_ARG.
 */
enum { SPEC_DRAFT_INDICES_PER_QUERY_HEAD = 1, SPEC_DRAFT_OUT_BF16 = 2, SPEC_DRAFT_EARLY_GATHER = 4 };
int spec_sparse_draft_attn_ex(const spec_kv_t* kv, const void* q, const int32_t* indices,
                              const int32_t* n_indices, int32_t k_total, const int32_t* tail_start,
                              const int32_t* cur_len, int32_t max_tail, float* out, float* lse,
                              void* workspace, size_t workspace_bytes, uint32_t flags,
                              void* cuda_stream);

/*
 * Bytes of workspace entry point `which` needs for this cache description.  n_q and
 * max_ctx_len matter for SPEC_WS_VERIFY, k_total (+ max_tail folded into it by the caller)
 * for SPEC_WS_DRAFT.  Returns 0 on invalid arguments.
 */
size_t spec_workspace_bytes(int which, const spec_kv_t* kv, int32_t n_q, int32_t max_ctx_len,
                            int32_t k_total);

/*
 * Synchronises `cuda_stream` and returns the status word at the head of `workspace`
 * (SPEC_OK, SPEC_ERR_TIMEOUT or SPEC_ERR_BAD_INDEX), or SPEC_ERR_CUDA if the stream reports
 * an error.  A non-zero word is reset to SPEC_OK once it has been returned.
 */
int spec_read_status(const void* workspace, void* cuda_stream);

/* Chooses the verification kernel (process-wide; SPEC_VERIFY_AUTO picks the tcgen05 kernel
 * when the shape allows it).  Returns the previous setting, or SPEC_ERR_INVALID_ARG. */
int spec_set_verify_impl(int impl);

/* Device-side waits (a CTA waiting for another CTA's partial result, for a copy, for the tensor
 * cores) give up after this many SM clocks, set SPEC_ERR_TIMEOUT in the status word and let the
 * kernel drain and return.  Default 2e9 (about a second).  Process-wide; applies to calls made
 * after it.  Returns the previous limit, or SPEC_ERR_INVALID_ARG for cycles < 1. */
int64_t spec_set_wait_limit_cycles(int64_t cycles);

/* Which kernel the last spec_verify_attn call of this process used (SPEC_VERIFY_GENERIC,
 * SPEC_VERIFY_TCGEN05_TWOSWEEP, SPEC_VERIFY_TCGEN05_CACHED, SPEC_VERIFY_TCGEN05_CACHED_2PASS or
 * SPEC_VERIFY_TCGEN05_CACHED_EXPANDED; 0 before the first call). */
int spec_last_verify_impl(void);

/*
 * How a call of this shape would be split (host-side planning only: nothing is launched, no GPU is
 * needed; without a current device the plan assumes 148 SMs).  which = SPEC_WS_VERIFY: out =
 * {kernel (0 = generic kernels, 1 = tcgen05 two-sweep, 2 = tcgen05 score-cache, 3 = score-cache on two
 * halves of the rows), KV heads per unit, CTAs per head, units, score columns N, score tiles the
 * tensor-memory cache holds, K/V tile slots, P buffers}.  which = SPEC_WS_DRAFT (k_total = budget
 * + longest tail): out = {CTAs per cluster, keys per CTA, warps per CTA, stages per warp, 0...}.
 */
int spec_describe_plan(int which, const spec_kv_t* kv, int32_t n_q, int32_t max_ctx_len,
                       int32_t k_total, int32_t out[8]);

/* Number of kernels this library has launched since load (host-side counter). */
int64_t spec_launch_count(void);

const char* spec_strerror(int code);
int spec_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SPEC_ATTN_H_ */
