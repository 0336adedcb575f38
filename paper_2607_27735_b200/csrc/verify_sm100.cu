// Host side of the sm_100a verification path: shape checks, the work plan (how KV heads are
// grouped into units and split over the CTAs), TMA tensor maps, and the choice between the
// score-cache kernel (K and V read once) and the two-sweep kernel (any context length).
#include <cstdlib>

#include "sm100_common.cuh"
#include "verify_sm100.cuh"

namespace spec {

using namespace sm100;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

struct Plan {
    bool cached;
    int HG, cph, n_units, N, n_slots, p_bufs, box_rows, boxes, n_cache, n_raw;
    size_t smem_bytes;
    size_t ctr_off, ctr_bytes, ml_off, o_off, total;
};

int box_rows_for(int page_size)
{
    if (page_size >= kTile) return (page_size % kTile == 0) ? kTile : 0;
    if (page_size >= 8 && kTile % page_size == 0) return page_size;
    return 0;
}

// variant: 0 = prefer the score-cache kernel, 1 = two-sweep only, 2 = score-cache only
bool make_plan(const KvView& kv, int n_q, int max_ctx_len, int variant, Plan* pl)
{
    const int G = kv.n_q_heads / kv.n_kv_heads, R = n_q * G;
    pl->n_raw = 0;
    // an 8-bit cache is read by the score-cache kernel only (its F8 instances), at head_dim 128
    if (kv.fp8 && (variant == 1 || kv.head_dim != kD)) return false;
    // head_dim 64 runs on the score-cache kernel only (one 64-wide half per tile, V padded with zero rows)
    if (!(kv.head_dim == kD || (kv.head_dim == 64 && variant != 1)) || R > 128 || G > 256 || n_q > 256) return false;
    const int box_rows = box_rows_for(kv.page_size);
    if (box_rows == 0) return false;
    const int nsm = sm_count();
    const int N = (R + 15) / 16 * 16;
    const int nb = (max_ctx_len + kTile - 1) / kTile;
    const long lb = (long)kv.n_layers * kv.batch;
    int n_cache = (kTmemCols - 2 * N) / N;
    if (n_cache > 32) n_cache = 32;

    int best_hg = 0;
    bool cached = false;
    if (variant != 1) {  // score-cache kernel: a CTA's share of a head must fit the TMEM cache
        double best = -1.0;
        for (int hg = 1; hg <= kv.n_kv_heads; ++hg) {
            if (kv.n_kv_heads % hg) continue;
            const int cph = nsm / hg;
            if (cph < 1) continue;
            const int tpc = (nb + cph - 1) / cph;
            if (tpc > n_cache) continue;
            const double score = (double)nb * hg / ((double)nsm * tpc) + 0.001 * hg;
            if (score > best) {
                best = score;
                best_hg = hg;
            }
        }
        cached = best_hg != 0;
    }
    if (!cached) {
        if (variant == 2 || kv.head_dim != kD || kv.fp8) return false;
        double best = -1.0;
        for (int hg = 1; hg <= kv.n_kv_heads; ++hg) {
            if (kv.n_kv_heads % hg) continue;
            const int cph = nsm / hg;
            if (cph < 1) continue;
            const int tpc = (nb + cph - 1) / cph;
            double score = (double)nb * hg / ((double)nsm * tpc);  // fraction of CTA-tile slots doing work
            const double k_mib = (double)hg * max_ctx_len * 256.0 / (1 << 20);
            if (k_mib > 40.0) score -= 0.3;                         // the unit's K must stay L2-resident
            if (lb * (kv.n_kv_heads / hg) < 2) score -= 0.1;        // a single unit cannot be pipelined
            score += 0.001 * hg;                                    // ties: fewer partials per head
            if (score > best) {
                best = score;
                best_hg = hg;
            }
        }
        if (best_hg == 0) return false;
    }
    pl->cached = cached;
    pl->n_cache = n_cache;
    pl->HG = best_hg;
    pl->cph = nsm / best_hg;
    pl->n_units = (int)(lb * (kv.n_kv_heads / best_hg));
    pl->N = N;
    pl->box_rows = box_rows;
    pl->boxes = kTile / box_rows;
    const size_t cap = 227 * 1024;
    size_t fixed = 0;
    int slots = 0;
    if (cached) {
        // one Q buffer, two P buffers ([hi | lo] rows, 8-row blocks: 2N * 256 B each), 12.25 KB of
        // barriers and small arrays; the rest is the K/V tile ring
        pl->p_bufs = 2;
        pl->n_raw = kv.fp8 ? 3 : 0;  // 8-bit cache: three raw stages of 16 KB in front of the slots
        fixed = 1024 /*alignment slack*/ + (size_t)N * 256 + 2 * (size_t)(2 * N * 256) + 12544 + (size_t)pl->n_raw * 16384;
        slots = fixed < cap ? (int)((cap - fixed) / kSlotBytes) : 0;
        if (slots > 8) slots = 8;
        // more P buffers (up to four) where they cost no K/V slot: the P V product of a tile then has two tiles
        // of softmax work to hide behind
        while (slots >= 4 && pl->p_bufs < 4 && fixed + (size_t)(2 * N * 256) + (size_t)slots * kSlotBytes <= cap) {
            ++pl->p_bufs;
            fixed += (size_t)(2 * N * 256);
        }
        if (slots < 4) {
            pl->p_bufs = 1;
            fixed -= (size_t)(2 * N * 256);
            slots = fixed < cap ? (int)((cap - fixed) / kSlotBytes) : 0;
        }
        if (kv.fp8) {
            // 8-bit cache: the raw stages already hold whole tiles in flight, so three operand slots do;
            // P buffers first (the P V product of a tile hides behind the next tiles' softmax work)
            slots = 0;
            for (int pb = 3; pb >= 1 && slots < 3; --pb) {
                for (int nr = 3; nr >= 2 && slots < 3; --nr) {
                    fixed = 1024 + (size_t)N * 256 + (size_t)pb * (2 * N * 256) + 12544 + (size_t)nr * 16384;
                    slots = fixed < cap ? (int)((cap - fixed) / kSlotBytes) : 0;
                    if (slots > 8) slots = 8;
                    pl->p_bufs = pb;
                    pl->n_raw = nr;
                }
            }
        }
    } else {
        const size_t p_bytes = (size_t)((2 * N + 63) / 64) * 16384;
        for (int pb = 2; pb >= 1; --pb) {  // two P buffers if that still leaves a 4-deep K/V ring
            fixed = 1024 /*alignment slack*/ + 2 * (size_t)N * 256 + pb * p_bytes + 12544;
            slots = fixed < cap ? (int)((cap - fixed) / kSlotBytes) : 0;
            pl->p_bufs = pb;
            if (slots >= 4) break;
        }
    }
    if (slots > 8) slots = 8;
    if (slots < 3) return false;
    pl->n_slots = slots;
    pl->smem_bytes = fixed + (size_t)slots * kSlotBytes;
    size_t off = kStatusBytes;
    pl->ctr_off = off;
    pl->ctr_bytes = ((size_t)2 * pl->n_units * pl->HG + 1) * sizeof(int);
    off += pl->ctr_bytes;
    off = (off + 255) & ~(size_t)255;
    pl->ml_off = off;
    off += (size_t)kRing * pl->HG * pl->cph * R * sizeof(float2);
    off = (off + 255) & ~(size_t)255;
    pl->o_off = off;
    off += (size_t)kRing * pl->HG * pl->cph * R * kD * sizeof(float);
    pl->total = (off + 255) & ~(size_t)255;
    return true;
}

bool encode_kv_map(CUtensorMap* map, const void* base, const KvView& kv, int n_pages, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[5] = {(cuuint64_t)kv.head_dim, (cuuint64_t)kv.page_size, (cuuint64_t)kv.n_kv_heads,
                                (cuuint64_t)n_pages, (cuuint64_t)kv.n_layers};
    const cuuint64_t strides[4] = {(cuuint64_t)kv.slot_stride * 2, (cuuint64_t)kv.head_stride * 2,
                                   (cuuint64_t)kv.page_stride * 2, (cuuint64_t)kv.layer_stride * 2};
    const cuuint32_t box[5] = {64, (cuuint32_t)box_rows, 1, 1, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    // a stride of 0 is legal only for extent-1 dimensions; give those any multiple of 16
    cuuint64_t st[4];
    for (int i = 0; i < 4; ++i) st[i] = strides[i] ? strides[i] : 16;
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(base), dims, st, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// 8-bit cache: a box is box_rows whole rows of 128 bytes, unswizzled (the softmax warps expand it)
bool encode_kv_map_u8(CUtensorMap* map, const void* base, const KvView& kv, int n_pages, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[5] = {(cuuint64_t)kv.head_dim, (cuuint64_t)kv.page_size, (cuuint64_t)kv.n_kv_heads,
                                (cuuint64_t)n_pages, (cuuint64_t)kv.n_layers};
    const cuuint64_t strides[4] = {(cuuint64_t)kv.slot_stride, (cuuint64_t)kv.head_stride, (cuuint64_t)kv.page_stride,
                                   (cuuint64_t)kv.layer_stride};
    const cuuint32_t box[5] = {128, (cuuint32_t)box_rows, 1, 1, 1};
    const cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    cuuint64_t st[4];
    for (int i = 0; i < 4; ++i) st[i] = strides[i] ? strides[i] : 16;
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 5, const_cast<void*>(base), dims, st, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool encode_q_map(CUtensorMap* map, const void* q, const KvView& kv, int n_q, int G)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)kv.head_dim, (cuuint64_t)kv.n_q_heads,
                                (cuuint64_t)kv.n_layers * kv.batch * n_q};
    const cuuint64_t strides[2] = {(cuuint64_t)kv.head_dim * 2, (cuuint64_t)kv.n_q_heads * kv.head_dim * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)n_q};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// ---- rows in two passes ----------------------------------------------------------------------
// A single (layer, sequence) whose n_q * G rows do not fit the score cache at its context length
// (many speculated rows at a very long context) is verified as two calls of the score-cache kernel:
// rows [0, nA) against the context shortened by the nB rows that follow them, then rows [nA, n_q)
// against the whole context.  Both are ordinary causal verifications of the same cache; their
// statistics add up (the window rule is applied to each part's own rows).  K and V are read
// twice, which still beats the two-sweep kernel at these shapes.
struct SplitPlan {
    int nA, nB;
    size_t main_bytes, ctx_off, stat_off, total;
    int64_t stat_stride;
};

bool make_split_plan(const KvView& kv, int n_q, int max_ctx_len, SplitPlan* sp)
{
    if (kv.n_layers * kv.batch != 1 || n_q < 2) return false;
    Plan full;
    if (make_plan(kv, n_q, max_ctx_len, 2, &full)) return false;  // fits in one pass
    sp->nA = (n_q + 1) / 2;
    sp->nB = n_q - sp->nA;
    Plan pa, pb;
    if (!make_plan(kv, sp->nA, max_ctx_len, 2, &pa) || !make_plan(kv, sp->nB, max_ctx_len, 2, &pb)) return false;
    sp->main_bytes = pa.total > pb.total ? pa.total : pb.total;
    sp->ctx_off = sp->main_bytes;
    sp->stat_off = sp->ctx_off + 256;
    sp->stat_stride = ((int64_t)max_ctx_len + 63) / 64 * 64;
    sp->total = sp->stat_off + (size_t)kv.n_kv_heads * sp->stat_stride * sizeof(float);
    sp->total = (sp->total + 255) & ~(size_t)255;
    return true;
}

__global__ void shorten_ctx_kernel(const int32_t* ctx_len, int by, int32_t* out) { out[0] = ctx_len[0] - by; }

// stats <- (first part's value where it wrote one) + second part's value
__global__ void add_stats_kernel(float* stats, int64_t stat_stride, const float* second, int64_t second_stride,
                                 const int32_t* ctx_len, int max_ctx_len, int nB, int n_kv_heads, int accumulate)
{
    const int T = min(max(ctx_len[0], 0), max_ctx_len);  // the two verification kernels report a length out of range
    for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < (int64_t)n_kv_heads * T;
         i += (int64_t)gridDim.x * blockDim.x) {
        const int h = (int)(i / T), key = (int)(i - (int64_t)h * T);
        const float first = (key < T - nB || accumulate) ? stats[h * stat_stride + key] : 0.f;  // the first part wrote keys < T - nB
        stats[h * stat_stride + key] = first + second[h * second_stride + key];
    }
}

}  // namespace

bool verify_sm100_supported(const KvView& kv, int n_q, int variant)
{
    Plan pl;
    if (!make_plan(kv, n_q, kTile, variant == 2 ? 0 : variant, &pl)) return false;
    return kv.slot_stride >= kv.head_dim;
}

void verify_sm100_describe(const KvView& kv, int n_q, int max_ctx_len, int32_t out[8])
{
    for (int i = 0; i < 8; ++i) out[i] = 0;
    Plan pl;
    SplitPlan sp;
    int kind = 0;
    if (make_split_plan(kv, n_q, max_ctx_len, &sp) && make_plan(kv, sp.nA, max_ctx_len, 2, &pl)) kind = 3;
    else if (make_plan(kv, n_q, max_ctx_len, 0, &pl)) kind = pl.cached ? 2 : 1;
    if (!kind || kv.slot_stride < kv.head_dim) return;
    const int v[8] = {kind, pl.HG, pl.cph, pl.n_units, pl.N, pl.n_cache, pl.n_slots, pl.p_bufs};
    for (int i = 0; i < 8; ++i) out[i] = v[i];
}

size_t verify_sm100_workspace(const KvView& kv, int n_q, int max_ctx_len)
{
    // the same bytes serve either variant: take the larger of the two plans
    size_t best = 0;
    for (int variant = 1; variant <= 2; ++variant) {
        Plan pl;
        if (make_plan(kv, n_q, max_ctx_len, variant, &pl) && pl.total > best) best = pl.total;
    }
    SplitPlan sp;
    if (make_split_plan(kv, n_q, max_ctx_len, &sp) && sp.total > best) best = sp.total;
    return best;
}

// Whether verify_sm100_launch would accept these arguments (same decisions, nothing launched).
bool verify_sm100_can_run(const VerifyArgs& a, int variant)
{
    const bool scaled = a.kv.k_scale || a.kv.v_scale || a.kv.fp8;
    if (scaled && (a.stat_per_head || a.stat_group_max)) return false;  // no such instance of the kernel
    if (a.stat_per_head || a.stat_group_max) {
        const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
        Plan pl;
        if (variant == 1 || G > 8 || !make_plan(a.kv, a.n_q, a.max_ctx_len, 2, &pl)) return false;
        variant = 2;
    }
    SplitPlan sp;
    if (variant == 0 && make_split_plan(a.kv, a.n_q, a.max_ctx_len, &sp)) return a.workspace_bytes >= sp.total;
    Plan pl;
    if (!make_plan(a.kv, a.n_q, a.max_ctx_len, variant, &pl)) return false;
    if ((a.kv.k_scale || a.kv.v_scale) && !pl.cached) return false;
    return a.workspace_bytes >= pl.total;
}

int verify_sm100_launch(const VerifyArgs& a, int variant, cudaStream_t stream, int* used_variant)
{
    if ((a.kv.k_scale || a.kv.v_scale || a.kv.fp8) && (a.stat_per_head || a.stat_group_max))
        return SPEC_ERR_UNSUPPORTED_SHAPE;
    if (a.stat_per_head || a.stat_group_max) {
        // only the score-cache kernel keeps one score per attention head, for groups of up to 8;
        // everything else goes to the generic kernels
        const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
        Plan pl;
        if (variant == 1 || G > 8 || !make_plan(a.kv, a.n_q, a.max_ctx_len, 2, &pl))
            return SPEC_ERR_UNSUPPORTED_SHAPE;
        variant = 2;
    }
    SplitPlan sp;
    if (variant == 0 && make_split_plan(a.kv, a.n_q, a.max_ctx_len, &sp)) {
        if (a.workspace_bytes < sp.total) return SPEC_ERR_WORKSPACE_TOO_SMALL;
        char* ws = static_cast<char*>(a.workspace);
        int32_t* ctx_a = reinterpret_cast<int32_t*>(ws + sp.ctx_off);
        float* second = reinterpret_cast<float*>(ws + sp.stat_off);
        const int64_t row_elems = (int64_t)a.kv.n_q_heads * a.kv.head_dim;
        shorten_ctx_kernel<<<1, 1, 0, stream>>>(a.ctx_len, sp.nB, ctx_a);
        count_launch(1);
        VerifyArgs pa = a;  // rows [0, nA): the context ends where the other rows begin
        pa.n_q = sp.nA;
        pa.ctx_len = ctx_a;
        pa.first_stat_row = a.first_stat_row < sp.nA ? a.first_stat_row : sp.nA;
        pa.workspace_bytes = sp.main_bytes;
        pa.hist = nullptr;  // the histogram is of the summed statistic: counted after the closing add
        int rc = verify_sm100_launch(pa, 2, stream, nullptr);
        if (rc != SPEC_OK) return rc;
        VerifyArgs pb = a;  // rows [nA, n_q) against the whole context; their statistic goes to scratch
        pb.n_q = sp.nB;
        pb.q = a.q + sp.nA * row_elems;
        pb.out = a.out_bf16 ? reinterpret_cast<float*>(reinterpret_cast<__nv_bfloat16*>(a.out) + sp.nA * row_elems)
                            : a.out + sp.nA * row_elems;
        pb.lse = a.lse ? a.lse + (int64_t)sp.nA * a.kv.n_q_heads : nullptr;
        pb.first_stat_row = a.first_stat_row > sp.nA ? a.first_stat_row - sp.nA : 0;
        pb.stats = second;
        pb.stat_stride = sp.stat_stride;
        pb.stat_accumulate = 0;
        pb.hist = nullptr;
        pb.workspace_bytes = sp.main_bytes;
        rc = verify_sm100_launch(pb, 2, stream, nullptr);
        if (rc != SPEC_OK) return rc;
        add_stats_kernel<<<sm_count(), 256, 0, stream>>>(a.stats, a.stat_stride, second, sp.stat_stride, a.ctx_len, a.max_ctx_len, sp.nB,
                                                         a.kv.n_kv_heads, a.stat_accumulate);
        count_launch(1);
        if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
        if (used_variant) *used_variant = 3;
        return SPEC_OK;
    }
    Plan pl;
    if (!make_plan(a.kv, a.n_q, a.max_ctx_len, variant, &pl)) return SPEC_ERR_UNSUPPORTED_SHAPE;
    // per-(layer, KV head) scales (an 8-bit cache expanded to bf16): only the score-cache kernel applies them
    if ((a.kv.k_scale || a.kv.v_scale) && !pl.cached) return SPEC_ERR_UNSUPPORTED_SHAPE;
    if (a.workspace_bytes < pl.total) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const int n_pages = a.kv.n_pages;
    CUtensorMap tk, tv, tq;
    if (a.kv.fp8) {
        if (!encode_kv_map_u8(&tk, a.kv.k8, a.kv, n_pages, pl.box_rows) ||
            !encode_kv_map_u8(&tv, a.kv.v8, a.kv, n_pages, pl.box_rows))
            return SPEC_ERR_CUDA;
    } else if (!encode_kv_map(&tk, a.kv.k, a.kv, n_pages, pl.box_rows) ||
               !encode_kv_map(&tv, a.kv.v, a.kv, n_pages, pl.box_rows)) {
        return SPEC_ERR_CUDA;
    }
    if (!encode_q_map(&tq, a.q, a.kv, a.n_q, G)) return SPEC_ERR_CUDA;
    char* ws = static_cast<char*>(a.workspace);
    FastParams fp;
    fp.a = a;
    fp.HG = pl.HG;
    fp.NHG = a.kv.n_kv_heads / pl.HG;
    fp.cph = pl.cph;
    set_divisor(&fp, 0, a.kv.batch * fp.NHG);
    set_divisor(&fp, 1, fp.NHG);
    set_divisor(&fp, 2, fp.cph);
    set_divisor(&fp, 3, a.kv.n_q_heads / a.kv.n_kv_heads);
    fp.n_units = pl.n_units;
    fp.N = pl.N;
    fp.R = a.n_q * G;
    fp.G = G;
    fp.D = a.kv.head_dim;
    fp.n_slots = pl.n_slots;
    fp.n_raw = pl.n_raw;
    fp.p_bufs = pl.p_bufs;
    fp.box_rows = pl.box_rows;
    fp.boxes = pl.boxes;
    fp.scale_log2 = a.kv.scale * 1.4426950408889634f;
    fp.counters = reinterpret_cast<int*>(ws + pl.ctr_off);
    fp.ml_part = reinterpret_cast<float2*>(ws + pl.ml_off);
    fp.o_part = reinterpret_cast<float*>(ws + pl.o_off);
    fp.status = reinterpret_cast<int*>(ws);
    fp.n_pages = n_pages;
    fp.n_cache = pl.n_cache;
    fp.wait_limit = wait_limit();
    // no memset: the workspace arrives zeroed and the kernel's last CTA re-zeroes the counters
    if (used_variant) *used_variant = pl.cached ? 2 : 1;
    const int grid = pl.cph * pl.HG;
    return pl.cached ? launch_cached(tk, tv, tq, fp, grid, pl.smem_bytes, stream)
                     : launch_twosweep(tk, tv, tq, fp, grid, pl.smem_bytes, stream);
}

}  // namespace spec
