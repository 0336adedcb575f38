// Expands an 8-bit (e4m3) KV cache into a bf16 copy with the same strides, page by page, so that the
// tensor-core verification kernel can stream it.  Every e4m3 value is a bf16 value, so the copy is
// exact; the per-(layer, KV head) scales are NOT applied here (a scaled value need not be a bf16
// value): the verification kernel folds K's scale into the softmax scale and V's into the output.
// Only the pages a sequence's context reaches are expanded.
#include "spec_common.cuh"

namespace spec {

namespace {

// One CTA per (block of kRows rows of a logical page, sequence, layer and K-or-V).  A page is
// n_kv_heads x page_size rows of head_dim bytes; a thread expands 16 bytes at a time.
constexpr int kRows = 256;

__global__ void __launch_bounds__(256)
expand_pages_kernel(KvView kv, __nv_bfloat16* __restrict__ k_out, __nv_bfloat16* __restrict__ v_out,
                    const int32_t* __restrict__ ctx_len, int max_ctx_len, int* status)
{
    const int rows_per_page = kv.n_kv_heads * kv.page_size;
    const int blocks_per_page = (rows_per_page + kRows - 1) / kRows;
    const int page = blockIdx.x / blocks_per_page, b = blockIdx.y;
    const int row0 = (blockIdx.x - page * blocks_per_page) * kRows;
    const int layer = blockIdx.z >> 1;
    const bool is_v = blockIdx.z & 1;
    const int T = min(max(__ldg(ctx_len + b), 0), max_ctx_len);  // (the verification kernel reports a bad length)
    if ((int64_t)page * kv.page_size >= T) return;
    int64_t phys = kv.page_table ? (int64_t)__ldg(kv.page_table + (int64_t)b * kv.max_pages + page)
                                 : (int64_t)b * kv.max_pages + page;
    if (phys < 0 || phys >= kv.n_pages) {  // same rule as kv_row_offset: reported, page 0 stands in
        if (threadIdx.x == 0) atomicCAS(status, 0, SPEC_ERR_BAD_INDEX);
        phys = 0;
    }
    const int64_t base = layer * kv.layer_stride + phys * kv.page_stride;
    const uint8_t* src = (is_v ? kv.v8 : kv.k8) + base;
    __nv_bfloat16* dst = (is_v ? v_out : k_out) + base;
    const int pieces = kv.head_dim >> 4;  // 16-byte pieces per row
    const int n = min(kRows, rows_per_page - row0) * pieces;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int piece = i % pieces;
        const int row = row0 + i / pieces;
        const int slot = row % kv.page_size, h = row / kv.page_size;
        if ((int64_t)page * kv.page_size + slot >= T) continue;  // beyond the context: never read
        const int64_t off = h * kv.head_stride + slot * kv.slot_stride + piece * 16;
        const uint4 in = *reinterpret_cast<const uint4*>(src + off);
        const uint32_t w[4] = {in.x, in.y, in.z, in.w};
        uint32_t o[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 lo = e4m3x2_to_float2((uint16_t)(w[j] & 0xffffu));
            const float2 hi = e4m3x2_to_float2((uint16_t)(w[j] >> 16));
            o[2 * j] = pack_bf16(lo.x, lo.y);
            o[2 * j + 1] = pack_bf16(hi.x, hi.y);
        }
        uint4* out = reinterpret_cast<uint4*>(dst + off);
        out[0] = make_uint4(o[0], o[1], o[2], o[3]);
        out[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

}  // namespace

// Elements of one expanded tensor (K or V): the span the view's strides cover.
int64_t kv_expand_elems(const KvView& kv)
{
    return (int64_t)(kv.n_layers - 1) * kv.layer_stride + (int64_t)kv.n_pages * kv.page_stride;
}

// True if pages and layers of the view do not interleave, i.e. a page's rows lie inside its own
// page_stride and a layer's pages inside its layer_stride (what every cache of this library's inputs does).
bool kv_expand_supported(const KvView& kv)
{
    const int64_t page_extent =
        (int64_t)(kv.n_kv_heads - 1) * kv.head_stride + (int64_t)(kv.page_size - 1) * kv.slot_stride + kv.head_dim;
    if (page_extent > kv.page_stride) return false;
    if (kv.n_layers > 1 && (int64_t)kv.n_pages * kv.page_stride > kv.layer_stride) return false;
    return kv.fp8 != 0;
}

int kv_expand_launch(const KvView& kv, __nv_bfloat16* k_out, __nv_bfloat16* v_out, const int32_t* ctx_len,
                     int max_ctx_len, int* status, cudaStream_t stream)
{
    const int pages = (max_ctx_len + kv.page_size - 1) / kv.page_size;
    const int64_t blocks = (int64_t)pages * ((kv.n_kv_heads * kv.page_size + kRows - 1) / kRows);
    if (pages < 1 || blocks > 0x7fffffff || kv.batch > 65535 || kv.n_layers * 2 > 65535) return SPEC_ERR_UNSUPPORTED_SHAPE;
    expand_pages_kernel<<<dim3((unsigned)blocks, (unsigned)kv.batch, (unsigned)kv.n_layers * 2), 256, 0, stream>>>(
        kv, k_out, v_out, ctx_len, max_ctx_len, status);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

}  // namespace spec
