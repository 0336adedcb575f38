// C-ABI entry points: argument validation on the host, then kernel launches on the caller's
// stream.  No device allocation, no synchronisation (except spec_read_status).
#include <atomic>
#include <cmath>
#include <map>
#include <mutex>
#include <utility>

#include "draft_common.cuh"
#include "spec_common.cuh"
#include "verify_sm100.cuh"

namespace spec {

static std::atomic<int64_t> g_launches{0};
static std::atomic<int> g_verify_impl{SPEC_VERIFY_AUTO};
static std::atomic<int> g_last_verify_impl{0};

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Everything remembered about a device is kept per device ordinal: one process may drive several.
constexpr int kMaxDevices = 64;

int sm_count()
{
    static std::atomic<int> cached[kMaxDevices];
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
    n = cached[dev].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

static std::atomic<long long> g_wait_limit{2000ll * 1000ll * 1000ll};  // about a second of SM clocks
long long wait_limit() { return g_wait_limit.load(std::memory_order_relaxed); }

bool draft::opt_in_smem(const void* kernel, size_t smem)
{
    static std::mutex mu;
    static std::map<std::pair<const void*, int>, size_t> configured;  // (kernel, device) -> largest size opted in
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    std::lock_guard<std::mutex> lock(mu);
    size_t& have = configured[std::make_pair(kernel, dev)];
    if (smem <= have) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    have = smem;
    return true;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Validates the cache description and converts it; returns SPEC_OK or an error.
static int make_view(const spec_kv_t* kv, KvView* out)
{
    if (!kv || !kv->k || !kv->v) return SPEC_ERR_INVALID_ARG;
    if (kv->n_layers < 1 || kv->page_size < 1 || kv->max_pages < 1 || kv->batch < 1 ||
        kv->n_q_heads < 1 || kv->n_kv_heads < 1)
        return SPEC_ERR_INVALID_ARG;
    if (kv->n_q_heads % kv->n_kv_heads != 0) return SPEC_ERR_INVALID_ARG;
    if (kv->head_dim != 64 && kv->head_dim != 128) return SPEC_ERR_UNSUPPORTED_SHAPE;
    if (!aligned16(kv->k) || !aligned16(kv->v)) return SPEC_ERR_INVALID_ARG;
    if (kv->kv_dtype != SPEC_KV_BF16 && kv->kv_dtype != SPEC_KV_FP8_E4M3) return SPEC_ERR_INVALID_ARG;
    const bool fp8 = kv->kv_dtype == SPEC_KV_FP8_E4M3;
    const int64_t strides[4] = {kv->layer_stride, kv->page_stride, kv->head_stride, kv->slot_stride};
    for (int64_t s : strides)
        if (s < 0 || s % (fp8 ? 16 : 8) != 0) return SPEC_ERR_INVALID_ARG;  // every row starts on 16 bytes
    if (kv->slot_stride < kv->head_dim) return SPEC_ERR_INVALID_ARG;
    out->fp8 = fp8 ? 1 : 0;
    out->k = fp8 ? nullptr : static_cast<const __nv_bfloat16*>(kv->k);
    out->v = fp8 ? nullptr : static_cast<const __nv_bfloat16*>(kv->v);
    out->k8 = fp8 ? static_cast<const uint8_t*>(kv->k) : nullptr;
    out->v8 = fp8 ? static_cast<const uint8_t*>(kv->v) : nullptr;
    out->k_scale = fp8 ? kv->k_scale : nullptr;
    out->v_scale = fp8 ? kv->v_scale : nullptr;
    out->layer_stride = kv->layer_stride;
    out->page_stride = kv->page_stride;
    out->head_stride = kv->head_stride;
    out->slot_stride = kv->slot_stride;
    out->page_table = kv->page_table;
    out->n_layers = kv->n_layers;
    out->page_size = kv->page_size;
    out->max_pages = kv->max_pages;
    out->batch = kv->batch;
    out->n_q_heads = kv->n_q_heads;
    out->n_kv_heads = kv->n_kv_heads;
    out->head_dim = kv->head_dim;
    if (kv->n_pages < 0) return SPEC_ERR_INVALID_ARG;
    out->n_pages = kv->n_pages > 0 ? kv->n_pages : kv->batch * kv->max_pages;
    out->scale = kv->sm_scale > 0.f ? kv->sm_scale : 1.0f / std::sqrt((float)kv->head_dim);
    set_page_divisor(out);
    return SPEC_OK;
}

// The bf16 twin of an 8-bit view: same strides, page table and scales, data pointers filled in by the caller.
static KvView bf16_twin(const KvView& kv)
{
    KvView t = kv;
    t.fp8 = 0;
    t.k8 = nullptr;
    t.v8 = nullptr;
    return t;
}

// Workspace of a verification call over an 8-bit cache: [0, base) as for any call (base = the larger of the
// generic kernels' and the tensor-core kernels' needs on the bf16 twin), then the twin's K and V.
static size_t fp8_verify_base(const KvView& kv, int n_q, int max_ctx_len)
{
    const size_t g = verify_generic_workspace(kv, n_q, max_ctx_len);
    const size_t f = verify_sm100_workspace(bf16_twin(kv), n_q, max_ctx_len);
    return ((g > f ? g : f) + 255) & ~(size_t)255;
}

static int sm100_variant(int impl)
{
    return impl == SPEC_VERIFY_TCGEN05_TWOSWEEP ? 1 : (impl == SPEC_VERIFY_TCGEN05_CACHED ? 2 : 0);
}

}  // namespace spec

using namespace spec;

extern "C" {

int spec_verify_attn(const spec_kv_t* kv, const void* q, int32_t n_q, const int32_t* ctx_len,
                     int32_t max_ctx_len, int32_t stat_window, float* out, float* lse, float* stats,
                     int64_t stat_stride, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    return spec_verify_attn_ex(kv, q, n_q, ctx_len, max_ctx_len, stat_window, out, lse, stats, stat_stride, workspace,
                               workspace_bytes, 0u, cuda_stream);
}

int spec_verify_attn_ex(const spec_kv_t* kv, const void* q, int32_t n_q, const int32_t* ctx_len,
                        int32_t max_ctx_len, int32_t stat_window, float* out, float* lse, float* stats,
                        int64_t stat_stride, void* workspace, size_t workspace_bytes, uint32_t flags,
                        void* cuda_stream)
{
    return spec_verify_attn_hist(kv, q, n_q, ctx_len, max_ctx_len, stat_window, out, lse, stats, stat_stride, workspace,
                                 workspace_bytes, flags, nullptr, cuda_stream);
}

int spec_verify_attn_hist(const spec_kv_t* kv, const void* q, int32_t n_q, const int32_t* ctx_len,
                          int32_t max_ctx_len, int32_t stat_window, float* out, float* lse, float* stats,
                          int64_t stat_stride, void* workspace, size_t workspace_bytes, uint32_t flags,
                          uint32_t* score_hist, void* cuda_stream)
{
    if (flags & ~(uint32_t)(SPEC_VERIFY_ACCUMULATE_STATS | SPEC_VERIFY_STATS_PER_QUERY_HEAD | SPEC_VERIFY_OUT_BF16 |
                            SPEC_VERIFY_STATS_GROUP_MAX))
        return SPEC_ERR_INVALID_ARG;
    if ((flags & SPEC_VERIFY_STATS_PER_QUERY_HEAD) && (flags & SPEC_VERIFY_STATS_GROUP_MAX)) return SPEC_ERR_INVALID_ARG;
    VerifyArgs a;
    const int rc = make_view(kv, &a.kv);
    if (rc != SPEC_OK) return rc;
    if (!q || !ctx_len || !out || !stats || !workspace) return SPEC_ERR_INVALID_ARG;
    if (n_q < 1 || n_q > 32 || max_ctx_len < n_q || stat_window < 0 || stat_stride < max_ctx_len)
        return SPEC_ERR_INVALID_ARG;
    if ((int64_t)kv->max_pages * kv->page_size < max_ctx_len) return SPEC_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return SPEC_ERR_INVALID_ARG;
    const int G = kv->n_q_heads / kv->n_kv_heads;
    if (n_q * G > 128) return SPEC_ERR_UNSUPPORTED_SHAPE;
    const int W = stat_window > 0 ? stat_window : 16;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.n_q = n_q;
    a.ctx_len = ctx_len;
    a.max_ctx_len = max_ctx_len;
    a.first_stat_row = n_q - (W < n_q ? W : n_q);
    a.out = out;
    a.lse = lse;
    a.stats = stats;
    a.stat_stride = stat_stride;
    a.workspace = workspace;
    a.workspace_bytes = workspace_bytes;
    a.stat_accumulate = (flags & SPEC_VERIFY_ACCUMULATE_STATS) ? 1 : 0;
    a.stat_per_head = (flags & SPEC_VERIFY_STATS_PER_QUERY_HEAD) ? 1 : 0;
    a.stat_group_max = (flags & SPEC_VERIFY_STATS_GROUP_MAX) ? 1 : 0;
    a.out_bf16 = (flags & SPEC_VERIFY_OUT_BF16) ? 1 : 0;
    a.hist = score_hist;  // the score-cache kernel counts in its statistic pass; the others get a sweep afterwards
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const long hist_probs = (long)kv->n_layers * kv->batch * (a.stat_per_head ? kv->n_q_heads : kv->n_kv_heads);
    const int hist_heads = a.stat_per_head ? kv->n_q_heads : kv->n_kv_heads;
    const int impl = g_verify_impl.load();
    // 8-bit cache: the score-cache kernel reads the bytes itself where its F8 instances apply; else the
    // cache is expanded to bf16 in the tail of the workspace (when the caller sized it with
    // spec_workspace_bytes and the layout allows) and streamed by the kernel's scaled instances; else the
    // generic kernels read the bytes
    VerifyArgs twin = a;
    bool fast_ok = !a.kv.fp8, expanded = false;
    if (a.kv.fp8 && impl != SPEC_VERIFY_GENERIC &&
        verify_sm100_can_run(a, sm100_variant(impl))) {
        fast_ok = true;
    } else if (a.kv.fp8 && impl != SPEC_VERIFY_GENERIC && kv_expand_supported(a.kv)) {
        const size_t base = fp8_verify_base(a.kv, n_q, max_ctx_len);
        const size_t elems = (size_t)kv_expand_elems(a.kv);
        if (workspace_bytes >= base + 4 * elems) {
            __nv_bfloat16* k16 = reinterpret_cast<__nv_bfloat16*>(static_cast<char*>(workspace) + base);
            twin.kv = bf16_twin(a.kv);
            twin.kv.k = k16;
            twin.kv.v = k16 + elems;
            twin.workspace_bytes = base;
            fast_ok = verify_sm100_can_run(twin, sm100_variant(impl));
            expanded = fast_ok;
            if (fast_ok) {
                const int rc1 = kv_expand_launch(a.kv, k16, k16 + elems, ctx_len, max_ctx_len,
                                                 static_cast<int*>(workspace), stream);
                if (rc1 != SPEC_OK) return rc1;
            }
        }
    }
    if (impl != SPEC_VERIFY_GENERIC && fast_ok) {
        int used = 0;
        const int rc2 = verify_sm100_launch(twin, sm100_variant(impl), stream, &used);
        if (rc2 == SPEC_OK) {
            g_last_verify_impl.store(expanded    ? SPEC_VERIFY_TCGEN05_CACHED_EXPANDED
                                     : used == 3 ? SPEC_VERIFY_TCGEN05_CACHED_2PASS
                                     : used == 2 ? SPEC_VERIFY_TCGEN05_CACHED
                                                 : SPEC_VERIFY_TCGEN05_TWOSWEEP);
            if (score_hist && used != 2)
                return score_hist_launch(stats, stat_stride, hist_probs, kv->batch, hist_heads, ctx_len, max_ctx_len,
                                         score_hist, stream);
            return SPEC_OK;
        }
        // an explicit tcgen05 request fails loudly; AUTO falls through to the generic kernels only
        // when the shape is outside the fast path
        if (impl != SPEC_VERIFY_AUTO || rc2 != SPEC_ERR_UNSUPPORTED_SHAPE) return rc2;
    }
    if (workspace_bytes < verify_generic_workspace(a.kv, n_q, max_ctx_len)) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    g_last_verify_impl.store(SPEC_VERIFY_GENERIC);
    const int rc3 = verify_generic_launch(a, stream);
    if (rc3 != SPEC_OK || !score_hist) return rc3;
    return score_hist_launch(stats, stat_stride, hist_probs, kv->batch, hist_heads, ctx_len, max_ctx_len, score_hist,
                             stream);
}

int spec_select_recall(const float* stats, int64_t stat_stride, int32_t n_layers, int32_t batch,
                       int32_t n_kv_heads, const int32_t* sel_len, int32_t k_sink, int32_t k_recent,
                       int32_t k_total, int32_t* indices, int32_t* n_indices, void* workspace,
                       size_t workspace_bytes, void* cuda_stream)
{
    return spec_select_recall_hist(stats, stat_stride, n_layers, batch, n_kv_heads, sel_len, k_sink, k_recent, k_total,
                                   indices, n_indices, nullptr, nullptr, workspace, workspace_bytes, cuda_stream);
}

int spec_select_recall_hist(const float* stats, int64_t stat_stride, int32_t n_layers, int32_t batch,
                            int32_t n_kv_heads, const int32_t* sel_len, int32_t k_sink, int32_t k_recent,
                            int32_t k_total, int32_t* indices, int32_t* n_indices, uint32_t* score_hist,
                            const int32_t* hist_len, void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    (void)workspace;
    (void)workspace_bytes;
    if ((score_hist != nullptr) != (hist_len != nullptr)) return SPEC_ERR_INVALID_ARG;
    if (!stats || !sel_len || !indices || !n_indices) return SPEC_ERR_INVALID_ARG;
    if (n_layers < 1 || batch < 1 || n_kv_heads < 1 || stat_stride < 1) return SPEC_ERR_INVALID_ARG;
    if (k_sink < 0 || k_recent < 0 || k_total < 1 || k_sink + (int64_t)k_recent > k_total)
        return SPEC_ERR_INVALID_ARG;
    return select_launch(stats, stat_stride, n_layers, batch, n_kv_heads, sel_len, k_sink, k_recent,
                         k_total, indices, n_indices, score_hist, hist_len, static_cast<cudaStream_t>(cuda_stream));
}

int spec_sparse_draft_attn(const spec_kv_t* kv, const void* q, const int32_t* indices,
                           const int32_t* n_indices, int32_t k_total, const int32_t* tail_start,
                           const int32_t* cur_len, int32_t max_tail, float* out, float* lse,
                           void* workspace, size_t workspace_bytes, void* cuda_stream)
{
    return spec_sparse_draft_attn_ex(kv, q, indices, n_indices, k_total, tail_start, cur_len, max_tail, out, lse,
                                     workspace, workspace_bytes, 0u, cuda_stream);
}

int spec_sparse_draft_attn_ex(const spec_kv_t* kv, const void* q, const int32_t* indices,
                              const int32_t* n_indices, int32_t k_total, const int32_t* tail_start,
                              const int32_t* cur_len, int32_t max_tail, float* out, float* lse,
                              void* workspace, size_t workspace_bytes, uint32_t flags, void* cuda_stream)
{
    if (flags & ~(uint32_t)(SPEC_DRAFT_INDICES_PER_QUERY_HEAD | SPEC_DRAFT_OUT_BF16 | SPEC_DRAFT_EARLY_GATHER))
        return SPEC_ERR_INVALID_ARG;
    DraftArgs a;
    const int rc = make_view(kv, &a.kv);
    if (rc != SPEC_OK) return rc;
    a.head_div = 1;
    a.out_bf16 = (flags & SPEC_DRAFT_OUT_BF16) ? 1 : 0;
    a.early_gather = (flags & SPEC_DRAFT_EARLY_GATHER) ? 1 : 0;
    a.wait_limit = wait_limit();
    if (flags & SPEC_DRAFT_INDICES_PER_QUERY_HEAD) {
        // every attention head is a problem of its own (group size 1) that reads the rows of its
        // KV head: the kernels see n_q_heads "KV heads" and divide the head index for the cache
        a.head_div = a.kv.n_q_heads / a.kv.n_kv_heads;
        a.kv.n_kv_heads = a.kv.n_q_heads;
    }
    if (!q || !indices || !n_indices || !tail_start || !cur_len || !out || !workspace)
        return SPEC_ERR_INVALID_ARG;
    if (k_total < 1 || max_tail < 0) return SPEC_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return SPEC_ERR_INVALID_ARG;
    a.q = static_cast<const __nv_bfloat16*>(q);
    a.indices = indices;
    a.n_indices = n_indices;
    a.k_total = k_total;
    a.tail_start = tail_start;
    a.cur_len = cur_len;
    a.max_tail = max_tail;
    a.out = out;
    a.lse = lse;
    a.workspace = workspace;
    a.workspace_bytes = workspace_bytes;
    if (workspace_bytes < draft_workspace(a.kv, k_total + max_tail)) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    return draft_launch(a, static_cast<cudaStream_t>(cuda_stream));
}

size_t spec_workspace_bytes(int which, const spec_kv_t* kv, int32_t n_q, int32_t max_ctx_len,
                            int32_t k_total)
{
    if (which == SPEC_WS_SELECT) return kStatusBytes;
    KvView v;
    if (make_view(kv, &v) != SPEC_OK) return 0;
    if (which == SPEC_WS_VERIFY) {
        if (n_q < 1 || n_q > 32 || max_ctx_len < n_q) return 0;
        // 8-bit cache: room for its bf16 copy behind the usual workspace (4 bytes per cache element of the view)
        if (v.fp8 && kv_expand_supported(v))
            return fp8_verify_base(v, n_q, max_ctx_len) + 4 * (size_t)kv_expand_elems(v);
        size_t g = verify_generic_workspace(v, n_q, max_ctx_len);
        size_t f = verify_sm100_workspace(v, n_q, max_ctx_len);
        return g > f ? g : f;
    }
    if (which == SPEC_WS_DRAFT) {
        if (k_total < 1) return 0;
        return draft_workspace(v, k_total);
    }
    return 0;
}

int spec_token_entropy(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab, int64_t row_stride,
                       float* entropy, void* cuda_stream)
{
    if (!logits || !entropy || n_rows < 0 || vocab < 1 || row_stride < vocab || (dtype != 0 && dtype != 1))
        return SPEC_ERR_INVALID_ARG;
    if (n_rows == 0) return SPEC_OK;
    if (n_rows > 65535) return SPEC_ERR_UNSUPPORTED_SHAPE;
    return rows_launch(logits, dtype, n_rows, vocab, row_stride, entropy, nullptr,
                       static_cast<cudaStream_t>(cuda_stream));
}

int spec_token_argmax(const void* logits, int32_t dtype, int32_t n_rows, int32_t vocab, int64_t row_stride,
                      int32_t* token, float* entropy, void* cuda_stream)
{
    if (!logits || !token || n_rows < 0 || vocab < 1 || row_stride < vocab || (dtype != 0 && dtype != 1))
        return SPEC_ERR_INVALID_ARG;
    if (n_rows == 0) return SPEC_OK;
    if (n_rows > 65535) return SPEC_ERR_UNSUPPORTED_SHAPE;
    return rows_launch(logits, dtype, n_rows, vocab, row_stride, entropy, token,
                       static_cast<cudaStream_t>(cuda_stream));
}

int spec_accept_greedy(const void* logits, int32_t dtype, int32_t batch, int32_t k1, int32_t vocab,
                       int64_t row_stride, const int32_t* draft, const int32_t* n_draft, int32_t* target,
                       int32_t* n_accepted, int32_t* next_token, void* cuda_stream)
{
    if (!logits || !target || !n_accepted || !next_token || batch < 0 || k1 < 1 || vocab < 1 ||
        row_stride < vocab || (dtype != 0 && dtype != 1) || (k1 > 1 && !draft))
        return SPEC_ERR_INVALID_ARG;
    if (batch == 0) return SPEC_OK;
    if ((int64_t)batch * k1 > 65535) return SPEC_ERR_UNSUPPORTED_SHAPE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int rc = rows_launch(logits, dtype, batch * k1, vocab, row_stride, nullptr, target, stream);
    if (rc != SPEC_OK) return rc;
    return accept_launch(target, draft, n_draft, batch, k1, n_accepted, next_token, stream);
}

int spec_advance_lengths(int32_t* committed, const int32_t* n_accepted, int32_t batch, int32_t k,
                         int32_t max_len, void* workspace, int32_t* ctx_verify, int32_t* cur_len,
                         void* cuda_stream)
{
    if (!committed || batch < 0 || k < 0 || max_len < 0) return SPEC_ERR_INVALID_ARG;
    if (batch == 0) return SPEC_OK;
    return advance_lengths_launch(committed, n_accepted, batch, k, max_len, static_cast<int*>(workspace), ctx_verify, cur_len,
                                  static_cast<cudaStream_t>(cuda_stream));
}

int spec_controller_update(float* state, const float* entropy, int32_t k, const int32_t* n_accepted, float beta,
                           void* cuda_stream)
{
    if (!state || !entropy || !n_accepted || k < 0 || !(beta >= 0.f && beta <= 1.f)) return SPEC_ERR_INVALID_ARG;
    if (k == 0) return SPEC_OK;
    return controller_update_launch(state, entropy, k, n_accepted, beta, static_cast<cudaStream_t>(cuda_stream));
}

int spec_controller_select(const float* state, const float* entropy, int32_t n, const int32_t* cand, int32_t n_cand,
                           float c_d, float c_v, int32_t* k_star, float* p_out, float* score_out, void* cuda_stream)
{
    if (!state || !entropy || !cand || !k_star || n < 1 || n_cand < 1 || !(c_d >= 0.f) || !(c_v >= 0.f) ||
        !(c_d + c_v > 0.f))
        return SPEC_ERR_INVALID_ARG;
    return controller_select_launch(state, entropy, n, cand, n_cand, c_d, c_v, k_star, p_out, score_out,
                                    static_cast<cudaStream_t>(cuda_stream));
}

int spec_read_status(const void* workspace, void* cuda_stream)
{
    if (!workspace) return SPEC_ERR_INVALID_ARG;
    int code = 0;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(&code, workspace, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return SPEC_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return SPEC_ERR_CUDA;
    if (code != 0) {  // reading an error acknowledges it
        if (cudaMemsetAsync(const_cast<void*>(workspace), 0, sizeof(int), stream) != cudaSuccess ||
            cudaStreamSynchronize(stream) != cudaSuccess)
            return SPEC_ERR_CUDA;
    }
    return code;
}

int spec_set_verify_impl(int impl)
{
    if (impl < SPEC_VERIFY_AUTO || impl > SPEC_VERIFY_TCGEN05_CACHED) return SPEC_ERR_INVALID_ARG;
    return g_verify_impl.exchange(impl);
}

int spec_last_verify_impl(void) { return g_last_verify_impl.load(); }

int spec_describe_plan(int which, const spec_kv_t* kv, int32_t n_q, int32_t max_ctx_len, int32_t k_total,
                       int32_t out[8])
{
    if (!out) return SPEC_ERR_INVALID_ARG;
    for (int i = 0; i < 8; ++i) out[i] = 0;
    KvView v;
    const int rc = make_view(kv, &v);
    if (rc != SPEC_OK) return rc;
    if (which == SPEC_WS_VERIFY) {
        if (n_q < 1 || n_q > 32 || max_ctx_len < n_q) return SPEC_ERR_INVALID_ARG;
        verify_sm100_describe(v, n_q, max_ctx_len, out);
        return SPEC_OK;
    }
    if (which == SPEC_WS_DRAFT) {
        if (k_total < 1) return SPEC_ERR_INVALID_ARG;
        StreamShape s;
        if (!stream_plan(v, v.head_dim, k_total, &s)) return SPEC_ERR_UNSUPPORTED_SHAPE;
        out[0] = s.cs;
        out[1] = s.per;
        out[2] = s.nw;
        out[3] = s.st;
        return SPEC_OK;
    }
    return SPEC_ERR_INVALID_ARG;
}

int64_t spec_set_wait_limit_cycles(int64_t cycles)
{
    if (cycles < 1) return SPEC_ERR_INVALID_ARG;
    return g_wait_limit.exchange(cycles);
}

int64_t spec_launch_count(void) { return g_launches.load(); }

const char* spec_strerror(int code)
{
    switch (code) {
        case SPEC_OK: return "ok";
        case SPEC_ERR_INVALID_ARG: return "invalid argument";
        case SPEC_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case SPEC_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case SPEC_ERR_CUDA: return "CUDA error";
        case SPEC_ERR_TIMEOUT: return "device-side wait timed out";
        case SPEC_ERR_BAD_INDEX: return "recall index, page-table entry or length out of range";
        default: return "unknown error";
    }
}

int spec_version(void) { return 100; }

}  // extern "C"
