// Generic verification attention + Eq. 3 statistic: plain FP32 CUDA-core kernels for every
// supported shape (head_dim 64/128, any page size, any alignment).  The tcgen05 kernel in
// verify_sm100.cu is the fast path; this one is the reference-shaped fallback for shapes it
// does not take.
//
// The statistic of Eq. 3 sums softmax PROBABILITIES, so each key's contribution needs the
// row's global normaliser.  Four launches: (1) per-split running (max, sum) of every row,
// (2) combine into the row LSE, (3) second sweep that forms P = exp(s - LSE) directly, writes
// the column sums and accumulates P V per split, (4) sum of the split partials in a fixed order.
#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kTK = 128;       // keys per tile
constexpr int kSP = kTK + 4;   // row pitch of the score tile in shared memory (floats)
constexpr int kThreads = 256;
constexpr int kMaxRows = 128;  // rows per KV head: n_q * group

struct Layout {
    int n_splits;
    size_t ml_off, lse_off, opart_off, total;
};

Layout make_layout(const KvView& kv, int n_q, int max_ctx_len)
{
    Layout lo;
    const int R = n_q * (kv.n_q_heads / kv.n_kv_heads);
    const long probs = (long)kv.n_layers * kv.batch * kv.n_kv_heads;
    const int tiles = (max_ctx_len + kTK - 1) / kTK;
    long want = (4L * 148 + probs - 1) / probs;
    if (want > 64) want = 64;
    if (want > tiles) want = tiles;
    if (want < 1) want = 1;
    lo.n_splits = (int)want;
    size_t off = kStatusBytes;
    lo.ml_off = off;
    off += (size_t)probs * lo.n_splits * R * sizeof(float2);
    off = (off + 255) & ~(size_t)255;
    lo.lse_off = off;
    off += (size_t)probs * R * sizeof(float);
    off = (off + 255) & ~(size_t)255;
    lo.opart_off = off;
    off += (size_t)probs * lo.n_splits * R * kv.head_dim * sizeof(float);
    lo.total = (off + 255) & ~(size_t)255;
    return lo;
}

// Scores of one tile of keys against all R rows of the KV head, into shared memory.
// Masked entries (beyond the row's causal limit or beyond the context) become -inf.
template <int D>
__device__ __forceinline__ void score_tile(const KvView& kv, int layer, int b, int h,
                                           const float* __restrict__ Qs, float* __restrict__ S,
                                           int R, int G, int n_q, int T, int key0, int* status)
{
    const int key_l = threadIdx.x % kTK;
    const int rg = threadIdx.x / kTK;  // 0 or 1
    const int key = key0 + key_l;
    const bool valid = key < T;
    const uint4* krow = nullptr;
    const uint2* krow8 = nullptr;
    const float scale = kv.scale * (kv.fp8 ? kv_scale_of(kv.k_scale, kv, layer, h) : 1.f);
    if (valid) {
        const int64_t off = kv_row_offset(kv, layer, b, key, h, status);
        if (kv.fp8) krow8 = reinterpret_cast<const uint2*>(kv.k8 + off);
        else krow = reinterpret_cast<const uint4*>(kv.k + off);
    }
    for (int r0 = rg * 4; r0 < R; r0 += 8) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        if (valid) {
#pragma unroll 4
            for (int c = 0; c < D / 8; ++c) {
                float kf[8];
                if (kv.fp8) {  // eight e4m3 bytes; the head's scale joins the softmax scale
                    const uint2 kk = __ldg(krow8 + c);
                    const float2 a0 = e4m3x2_to_float2((uint16_t)kk.x), a1 = e4m3x2_to_float2((uint16_t)(kk.x >> 16));
                    const float2 a2 = e4m3x2_to_float2((uint16_t)kk.y), a3 = e4m3x2_to_float2((uint16_t)(kk.y >> 16));
                    kf[0] = a0.x; kf[1] = a0.y; kf[2] = a1.x; kf[3] = a1.y;
                    kf[4] = a2.x; kf[5] = a2.y; kf[6] = a3.x; kf[7] = a3.y;
                } else {
                    const uint4 kk = __ldg(krow + c);
                    kf[0] = bf16_lo(kk.x); kf[1] = bf16_hi(kk.x); kf[2] = bf16_lo(kk.y); kf[3] = bf16_hi(kk.y);
                    kf[4] = bf16_lo(kk.z); kf[5] = bf16_hi(kk.z); kf[6] = bf16_lo(kk.w); kf[7] = bf16_hi(kk.w);
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    if (r0 + i < R) {
                        const float4* qp = reinterpret_cast<const float4*>(Qs + (r0 + i) * D + c * 8);
                        const float4 q0 = qp[0], q1 = qp[1];
                        acc[i] += q0.x * kf[0] + q0.y * kf[1] + q0.z * kf[2] + q0.w * kf[3] +
                                  q1.x * kf[4] + q1.y * kf[5] + q1.z * kf[6] + q1.w * kf[7];
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = r0 + i;
            if (r < R) {
                const int pos = T - n_q + r / G;  // last key row r may see
                S[r * kSP + key_l] = (valid && key <= pos) ? acc[i] * scale : -INFINITY;
            }
        }
    }
}

template <int D>
__device__ __forceinline__ void load_q(const VerifyArgs& a, int layer, int b, int h, int R, int G,
                                       float* Qs)
{
    const int Hq = a.kv.n_q_heads;
    for (int idx = threadIdx.x; idx < R * D; idx += kThreads) {
        const int r = idx / D, d = idx - r * D;
        const int j = r / G, g = r - j * G;
        const int64_t row = (((int64_t)layer * a.kv.batch + b) * a.n_q + j) * Hq + h * G + g;
        Qs[idx] = __bfloat162float(a.q[row * D + d]);
    }
}

__device__ __forceinline__ void split_range(int T, int n_splits, int split, int& t0, int& t1)
{
    const int tiles = (T + kTK - 1) / kTK;
    const int per = (tiles + n_splits - 1) / n_splits;
    t0 = split * per;
    t1 = min(tiles, t0 + per);
}

template <int D>
__global__ void __launch_bounds__(kThreads)
verify_lse_partial_kernel(VerifyArgs a, int n_splits, float2* __restrict__ ml_part)
{
    extern __shared__ __align__(16) float smem[];
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads, R = a.n_q * G;
    float* Qs = smem;
    float* S = Qs + R * D;
    float* m_run = S + R * kSP;
    float* l_run = m_run + R;
    const int split = blockIdx.x, h = blockIdx.y;
    const int layer = blockIdx.z / a.kv.batch, b = blockIdx.z % a.kv.batch;
    const int T = clamped_ctx_len(a, b);
    int t0, t1;
    split_range(T, n_splits, split, t0, t1);
    load_q<D>(a, layer, b, h, R, G, Qs);
    for (int r = threadIdx.x; r < R; r += kThreads) {
        m_run[r] = -INFINITY;
        l_run[r] = 0.f;
    }
    __syncthreads();
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    for (int t = t0; t < t1; ++t) {
        score_tile<D>(a.kv, layer, b, h, Qs, S, R, G, a.n_q, T, t * kTK, static_cast<int*>(a.workspace));
        __syncthreads();
        for (int r = warp; r < R; r += kThreads / 32) {
            float v[kTK / 32];
            float mt = -INFINITY;
#pragma unroll
            for (int i = 0; i < kTK / 32; ++i) {
                v[i] = S[r * kSP + lane + 32 * i];
                mt = fmaxf(mt, v[i]);
            }
            mt = warp_max(mt);
            if (mt > -INFINITY) {
                const float m_old = m_run[r];
                const float m_new = fmaxf(m_old, mt);
                float s = 0.f;
#pragma unroll
                for (int i = 0; i < kTK / 32; ++i) s += expf(v[i] - m_new);
                s = warp_sum(s);
                if (lane == 0) {
                    l_run[r] = l_run[r] * expf(m_old - m_new) + s;
                    m_run[r] = m_new;
                }
            }
        }
        __syncthreads();
    }
    const int64_t prob = (int64_t)blockIdx.z * a.kv.n_kv_heads + h;
    for (int r = threadIdx.x; r < R; r += kThreads)
        ml_part[(prob * n_splits + split) * R + r] = make_float2(m_run[r], l_run[r]);
}

__global__ void verify_lse_combine_kernel(VerifyArgs a, int n_splits,
                                          const float2* __restrict__ ml_part,
                                          float* __restrict__ lse_ws)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads, R = a.n_q * G;
    const int64_t prob = blockIdx.x;
    const int r = threadIdx.x;
    if (r >= R) return;
    float M = -INFINITY;
    for (int s = 0; s < n_splits; ++s) M = fmaxf(M, ml_part[(prob * n_splits + s) * R + r].x);
    float Lsum = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float2 ml = ml_part[(prob * n_splits + s) * R + r];
        if (ml.y > 0.f) Lsum += ml.y * expf(ml.x - M);
    }
    const float lse = M + logf(Lsum);
    lse_ws[prob * R + r] = lse;
    if (a.lse) {
        const int h = prob % a.kv.n_kv_heads;
        const int64_t lb = prob / a.kv.n_kv_heads;
        const int j = r / G, g = r - j * G;
        a.lse[(lb * a.n_q + j) * a.kv.n_q_heads + h * G + g] = lse;
    }
}

template <int D, int RPT>
__global__ void __launch_bounds__(kThreads)
verify_main_kernel(VerifyArgs a, int n_splits, const float* __restrict__ lse_ws,
                   float* __restrict__ opart)
{
    extern __shared__ __align__(16) float smem[];
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads, R = a.n_q * G;
    float* Qs = smem;
    float* S = Qs + R * D;
    float* lse_s = S + R * kSP;
    const int split = blockIdx.x, h = blockIdx.y;
    const int layer = blockIdx.z / a.kv.batch, b = blockIdx.z % a.kv.batch;
    const int64_t prob = (int64_t)blockIdx.z * a.kv.n_kv_heads + h;
    const int T = clamped_ctx_len(a, b);
    int t0, t1;
    split_range(T, n_splits, split, t0, t1);
    load_q<D>(a, layer, b, h, R, G, Qs);
    for (int r = threadIdx.x; r < R; r += kThreads) lse_s[r] = lse_ws[prob * R + r];
    __syncthreads();

    constexpr int NG = kThreads / (D / 2);  // row groups in the PV step
    const int dp = threadIdx.x % (D / 2), rg = threadIdx.x / (D / 2);
    float acc[RPT][2];
#pragma unroll
    for (int i = 0; i < RPT; ++i) acc[i][0] = acc[i][1] = 0.f;
    const int stat_r0 = a.first_stat_row * G;
    const float v_scale = a.kv.fp8 ? kv_scale_of(a.kv.v_scale, a.kv, layer, h) : 1.f;

    for (int t = t0; t < t1; ++t) {
        const int key0 = t * kTK;
        score_tile<D>(a.kv, layer, b, h, Qs, S, R, G, a.n_q, T, key0, static_cast<int*>(a.workspace));
        __syncthreads();
        for (int idx = threadIdx.x; idx < R * kTK; idx += kThreads) {
            const int r = idx / kTK, kl = idx - r * kTK;
            const float s = S[r * kSP + kl];
            S[r * kSP + kl] = (s == -INFINITY) ? 0.f : expf(s - lse_s[r]);
        }
        __syncthreads();
        if (threadIdx.x < kTK && key0 + threadIdx.x < T) {
            if (a.stat_group_max) {  // per KV head, the largest of the group's per-head scores
                float best = 0.f;
                for (int g = 0; g < G; ++g) {
                    float cs = 0.f;
                    for (int r = stat_r0 + g; r < R; r += G) cs += S[r * kSP + threadIdx.x];
                    best = g == 0 ? cs : fmaxf(best, cs);
                }
                float* dst = a.stats + prob * a.stat_stride + key0 + threadIdx.x;
                *dst = a.stat_accumulate ? *dst + best : best;
            } else if (a.stat_per_head) {  // one score per attention head: rows j * G + g with the same g
                for (int g = 0; g < G; ++g) {
                    float cs = 0.f;
                    for (int r = stat_r0 + g; r < R; r += G) cs += S[r * kSP + threadIdx.x];
                    float* dst = a.stats + (prob * G + g) * a.stat_stride + key0 + threadIdx.x;
                    *dst = a.stat_accumulate ? *dst + cs : cs;
                }
            } else {
                float cs = 0.f;
                for (int r = stat_r0; r < R; ++r) cs += S[r * kSP + threadIdx.x];
                float* dst = a.stats + prob * a.stat_stride + key0 + threadIdx.x;
                *dst = a.stat_accumulate ? *dst + cs : cs;
            }
        }
        const int nk = min(kTK, T - key0);
        for (int kl = 0; kl < nk; kl += 4) {
            float v0[4], v1[4];
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                if (kl + kk < nk) {
                    const int64_t voff = kv_row_offset(a.kv, layer, b, key0 + kl + kk, h, static_cast<int*>(a.workspace));
                    if (a.kv.fp8) {
                        const float2 vv = e4m3x2_to_float2(__ldg(reinterpret_cast<const uint16_t*>(a.kv.v8 + voff) + dp));
                        v0[kk] = vv.x * v_scale;
                        v1[kk] = vv.y * v_scale;
                    } else {
                        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(a.kv.v + voff) + dp);
                        v0[kk] = bf16_lo(w);
                        v1[kk] = bf16_hi(w);
                    }
                } else {
                    v0[kk] = v1[kk] = 0.f;
                }
            }
#pragma unroll
            for (int i = 0; i < RPT; ++i) {
                const int r = rg + i * NG;
                if (r < R) {
                    const float4 p = *reinterpret_cast<const float4*>(S + r * kSP + kl);
                    acc[i][0] += p.x * v0[0] + p.y * v0[1] + p.z * v0[2] + p.w * v0[3];
                    acc[i][1] += p.x * v1[0] + p.y * v1[1] + p.z * v1[2] + p.w * v1[3];
                }
            }
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < RPT; ++i) {
        const int r = rg + i * NG;
        if (r < R) {
            float2* dst = reinterpret_cast<float2*>(opart + ((prob * n_splits + split) * R + r) * D) + dp;
            *dst = make_float2(acc[i][0], acc[i][1]);
        }
    }
}

__global__ void verify_out_combine_kernel(VerifyArgs a, int n_splits, const float* __restrict__ opart)
{
    const int D = a.kv.head_dim, G = a.kv.n_q_heads / a.kv.n_kv_heads, R = a.n_q * G;
    const int64_t prob = blockIdx.x / R;
    const int r = blockIdx.x % R;
    const int d = threadIdx.x;
    float s = 0.f;
    for (int sp = 0; sp < n_splits; ++sp) s += opart[((prob * n_splits + sp) * R + r) * D + d];
    const int h = prob % a.kv.n_kv_heads;
    const int64_t lb = prob / a.kv.n_kv_heads;
    const int j = r / G, g = r - j * G;
    const int64_t o = ((lb * a.n_q + j) * a.kv.n_q_heads + h * G + g) * D + d;
    if (a.out_bf16) reinterpret_cast<__nv_bfloat16*>(a.out)[o] = __float2bfloat16_rn(s);
    else a.out[o] = s;
}

template <int D>
int launch_d(const VerifyArgs& a, const Layout& lo, cudaStream_t stream)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads, R = a.n_q * G;
    char* ws = static_cast<char*>(a.workspace);
    float2* ml = reinterpret_cast<float2*>(ws + lo.ml_off);
    float* lse_ws = reinterpret_cast<float*>(ws + lo.lse_off);
    float* opart = reinterpret_cast<float*>(ws + lo.opart_off);
    const dim3 grid(lo.n_splits, a.kv.n_kv_heads, a.kv.n_layers * a.kv.batch);
    const long probs = (long)a.kv.n_layers * a.kv.batch * a.kv.n_kv_heads;
    const size_t smem1 = (size_t)(R * D + R * kSP + 2 * R) * sizeof(float);
    const size_t smem3 = (size_t)(R * D + R * kSP + R) * sizeof(float);

    if (cudaFuncSetAttribute(verify_lse_partial_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem1) != cudaSuccess)
        return SPEC_ERR_CUDA;
    verify_lse_partial_kernel<D><<<grid, kThreads, smem1, stream>>>(a, lo.n_splits, ml);
    verify_lse_combine_kernel<<<(unsigned)probs, kMaxRows, 0, stream>>>(a, lo.n_splits, ml, lse_ws);

    constexpr int NG = kThreads / (D / 2);
    const int rpt = (R + NG - 1) / NG;
#define SPEC_LAUNCH_MAIN(RPT)                                                                     \
    do {                                                                                          \
        if (cudaFuncSetAttribute(verify_main_kernel<D, RPT>,                                      \
                                 cudaFuncAttributeMaxDynamicSharedMemorySize,                     \
                                 (int)smem3) != cudaSuccess)                                      \
            return SPEC_ERR_CUDA;                                                                 \
        verify_main_kernel<D, RPT><<<grid, kThreads, smem3, stream>>>(a, lo.n_splits, lse_ws,    \
                                                                       opart);                    \
    } while (0)
    if (rpt <= 2) SPEC_LAUNCH_MAIN(2);
    else if (rpt <= 4) SPEC_LAUNCH_MAIN(4);
    else if (rpt <= 8) SPEC_LAUNCH_MAIN(8);
    else if (rpt <= 16) SPEC_LAUNCH_MAIN(16);
    else SPEC_LAUNCH_MAIN(32);
#undef SPEC_LAUNCH_MAIN
    verify_out_combine_kernel<<<(unsigned)(probs * R), D, 0, stream>>>(a, lo.n_splits, opart);
    count_launch(4);
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

}  // namespace

size_t verify_generic_workspace(const KvView& kv, int n_q, int max_ctx_len)
{
    return make_layout(kv, n_q, max_ctx_len).total;
}

int verify_generic_launch(const VerifyArgs& a, cudaStream_t stream)
{
    const int R = a.n_q * (a.kv.n_q_heads / a.kv.n_kv_heads);
    if (R > kMaxRows) return SPEC_ERR_UNSUPPORTED_SHAPE;
    const Layout lo = make_layout(a.kv, a.n_q, a.max_ctx_len);
    if (a.workspace_bytes < lo.total) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    if (a.kv.head_dim == 128) return launch_d<128>(a, lo, stream);
    if (a.kv.head_dim == 64) return launch_d<64>(a, lo, stream);
    return SPEC_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace spec
