// Shared device-side definitions of the attention kernels: cache addressing, bf16 unpacking,
// warp reductions, and the host-side launcher declarations used by spec_api.cu.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp8.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "spec_attn.h"

namespace spec {

// Device copy of the cache description (see spec_kv_t for the addressing rule).
struct KvView {
    const __nv_bfloat16* k;
    const __nv_bfloat16* v;
    int64_t layer_stride, page_stride, head_stride, slot_stride;
    const int32_t* page_table;
    int32_t n_layers, page_size, max_pages, batch, n_q_heads, n_kv_heads, head_dim, n_pages;
    float scale;  // resolved softmax scale
    // 8-bit cache (spec_kv_t::kv_dtype == SPEC_KV_FP8_E4M3): k8 / v8 hold e4m3 bytes and k / v are null;
    // an element's value is its e4m3 value times k_scale / v_scale [n_layers, n_kv_heads] (null: 1)
    int32_t fp8;
    const uint8_t* k8;
    const uint8_t* v8;
    const float* k_scale;
    const float* v_scale;
    // pos / page_size without a division: page = umulhi(pos, page_mul) >> page_sh for 0 <= pos < 2^31
    // (page_mul = ceil(2^(31 + c) / page_size), page_sh = c - 1, c = ceil(log2 page_size));
    // page_sh < 0 marks page_size == 1
    uint32_t page_mul;
    int32_t page_sh;
};

inline void set_page_divisor(KvView* kv)
{
    const uint32_t d = (uint32_t)kv->page_size;
    if (d <= 1) {
        kv->page_mul = 0;
        kv->page_sh = -1;
        return;
    }
    int c = 0;
    while ((1ull << c) < d) ++c;
    kv->page_mul = (uint32_t)(((1ull << (31 + c)) + d - 1) / d);
    kv->page_sh = c - 1;
}

__device__ __forceinline__ int page_of(const KvView& kv, int pos)
{
    return kv.page_sh < 0 ? pos : (int)(__umulhi((uint32_t)pos, kv.page_mul) >> kv.page_sh);
}

// Offset of a cache row.  A page-table entry outside [0, n_pages) is replaced by page 0 (the access stays
// inside the cache) and, when a status word is given, reported there as SPEC_ERR_BAD_INDEX.
__device__ __forceinline__ int64_t kv_row_offset(const KvView& kv, int layer, int b, int pos, int h,
                                                 int* status = nullptr)
{
    const int page = page_of(kv, pos);
    const int slot = pos - page * kv.page_size;
    int64_t phys = kv.page_table ? (int64_t)__ldg(kv.page_table + (int64_t)b * kv.max_pages + page)
                                 : (int64_t)b * kv.max_pages + page;
    if (phys < 0 || phys >= kv.n_pages) {
        if (status) atomicCAS(status, 0, SPEC_ERR_BAD_INDEX);
        phys = 0;
    }
    return layer * kv.layer_stride + phys * kv.page_stride + h * kv.head_stride +
           slot * kv.slot_stride;
}

// Two e4m3 bytes (low byte first) as two floats: exact (cvt to fp16 holds every e4m3 value).
__device__ __forceinline__ float2 e4m3x2_to_float2(uint16_t two)
{
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)two, __NV_E4M3);
    return __half22float2(*reinterpret_cast<const __half2*>(&h));
}
__device__ __forceinline__ float kv_scale_of(const float* scale, const KvView& kv, int layer, int h)
{
    return scale ? __ldg(scale + (int64_t)layer * kv.n_kv_heads + h) : 1.f;
}

// Two fp32 values as one packed bf16 pair (x in the low half), round to nearest even.
__device__ __forceinline__ uint32_t pack_bf16(float x, float y)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(x, y);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ float warp_max(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
    return x;
}
__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// The status word lives in the first int of every workspace; errors are sticky until the next
// call clears it.
__device__ __forceinline__ void set_status(int* status, int code) { atomicCAS(status, 0, code); }

constexpr int kStatusBytes = 256;  // head of every workspace: status word + padding
constexpr int kScoreBins = 2048;   // histogram of the top 11 bits of a score's fp32 pattern (first radix pass of Eq. 4)

// ---- launchers (defined in the kernel files; all enqueue on `stream`, none synchronises) ----
struct VerifyArgs {
    KvView kv;
    const __nv_bfloat16* q;
    int n_q;
    const int32_t* ctx_len;
    int max_ctx_len;
    int first_stat_row;  // window rows j >= first_stat_row feed the statistic
    float* out;
    float* lse;
    float* stats;
    int64_t stat_stride;
    void* workspace;
    size_t workspace_bytes;
    int stat_accumulate;  // add this call's statistic to what stats[] holds instead of overwriting it
    int stat_per_head;    // stats is [layers, batch, n_q_heads, stride]: one score per attention head
    int stat_group_max;   // stats is per KV head, but the group's per-head scores are folded by max instead of sum
    int out_bf16;         // `out` points to bf16 elements (round to nearest even) instead of fp32
    uint32_t* hist;       // not null: += counts of the final scores' top 11 bits, [problems][kScoreBins]
};

// Context length of sequence b as the kernels use it: a value outside [n_q, max_ctx_len] (the range the
// launch, the workspace and the score rows were sized for) is clamped into it and reported.
__device__ __forceinline__ int clamped_ctx_len(const VerifyArgs& a, int b)
{
    const int t = a.ctx_len[b];
    const int T = min(max(t, a.n_q), a.max_ctx_len);
    if (T != t) set_status(static_cast<int*>(a.workspace), SPEC_ERR_BAD_INDEX);
    return T;
}

size_t verify_generic_workspace(const KvView& kv, int n_q, int max_ctx_len);

// 8-bit cache -> bf16 copy with the same strides (kv_expand.cu): elements per tensor, whether the view's
// layout allows it, and the launch (pages up to each sequence's context only; scales are not applied)
int64_t kv_expand_elems(const KvView& kv);
bool kv_expand_supported(const KvView& kv);
int kv_expand_launch(const KvView& kv, __nv_bfloat16* k_out, __nv_bfloat16* v_out, const int32_t* ctx_len,
                     int max_ctx_len, int* status, cudaStream_t stream);
int verify_generic_launch(const VerifyArgs& a, cudaStream_t stream);

int select_launch(const float* stats, int64_t stat_stride, int n_layers, int batch, int n_kv_heads,
                  const int32_t* sel_len, int k_sink, int k_recent, int k_total, int32_t* indices,
                  int32_t* n_indices, uint32_t* hist, const int32_t* hist_len, cudaStream_t stream);
// counts the top 11 bits of stats[prob][0 : len[b]) into hist[prob][kScoreBins] (kernels that do not fuse it)
int score_hist_launch(const float* stats, int64_t stat_stride, long probs, int batch, int heads, const int32_t* len,
                      int max_len, uint32_t* hist, cudaStream_t stream);

struct DraftArgs {
    KvView kv;
    const __nv_bfloat16* q;
    const int32_t* indices;
    const int32_t* n_indices;
    int k_total;
    const int32_t* tail_start;
    const int32_t* cur_len;
    int max_tail;
    float* out;
    float* lse;
    void* workspace;
    size_t workspace_bytes;
    int head_div;  // K/V of problem head h are read from cache head h / head_div (1 unless every
                   // attention head carries its own index set)
    int out_bf16;  // `out` points to bf16 elements (round to nearest even) instead of fp32
    int early_gather;      // the caller promised that the index sets, lengths and recalled rows were complete
                           // before the preceding kernel of the stream started: they are read before this
                           // kernel's dependency on that kernel is resolved
    long long wait_limit;  // SM clocks after which a device-side wait gives up (SPEC_ERR_TIMEOUT)
};
size_t draft_workspace(const KvView& kv, int k_total_plus_tail);
int draft_launch(const DraftArgs& a, cudaStream_t stream);

int rows_launch(const void* logits, int dtype, int n_rows, int vocab, int64_t row_stride, float* entropy,
                int32_t* token, cudaStream_t stream);
int accept_launch(const int32_t* target, const int32_t* draft, const int32_t* n_draft, int batch, int k1,
                  int32_t* n_accepted, int32_t* next_token, cudaStream_t stream);
int advance_lengths_launch(int32_t* committed, const int32_t* n_accepted, int batch, int k, int max_len, int* status, int32_t* ctx_verify,
                           int32_t* cur_len, cudaStream_t stream);
int controller_update_launch(float* state, const float* entropy, int k, const int32_t* n_accepted, float beta,
                             cudaStream_t stream);
int controller_select_launch(const float* state, const float* entropy, int n, const int32_t* cand, int n_cand,
                             float c_d, float c_v, int32_t* k_star, float* p_out, float* score_out,
                             cudaStream_t stream);

void count_launch(int n = 1);
int sm_count();            // of the current device
long long wait_limit();    // SM clocks a device-side wait may take (spec_set_wait_limit_cycles)

}  // namespace spec
