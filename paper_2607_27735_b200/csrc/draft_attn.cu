// Sparse draft attention of Eq. 5: one query per sequence attends the recalled rows
// Gather(K, I), Gather(V, I) plus the dense tail of tokens drafted this round.  The gather is
// fused: 16-byte cp.async copies pull the indexed 2*D-byte rows straight from the dense cache
// into shared memory; nothing gathered is written back to global memory.
//
// Split-KV: the key list of a problem is cut into n_splits contiguous ranges, one CTA each,
// every CTA producing an un-normalised partial (running max, sum, P V); a small second kernel
// merges the partials in a fixed order (deterministic).
#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kTK = 64;        // keys per tile
constexpr int kThreads = 128;
constexpr int kMaxGroup = 8;   // query heads per KV head
constexpr int kRPT = 4;        // accumulator rows per thread in the PV step

struct Layout {
    int n_splits;
    size_t part_off, total;
};

Layout make_layout(const KvView& kv, int n_keys_max)
{
    Layout lo;
    const int G = kv.n_q_heads / kv.n_kv_heads;
    const long probs = (long)kv.n_layers * kv.batch * kv.n_kv_heads;
    const int tiles = n_keys_max > 0 ? (n_keys_max + kTK - 1) / kTK : 1;
    long want = (2L * 148 + probs - 1) / probs;
    if (want > tiles) want = tiles;
    if (want < 1) want = 1;
    lo.n_splits = (int)want;
    lo.part_off = kStatusBytes;
    lo.total = lo.part_off + (size_t)probs * lo.n_splits * G * (kv.head_dim + 2) * sizeof(float);
    lo.total = (lo.total + 255) & ~(size_t)255;
    return lo;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc)
{
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

template <int D>
__global__ void __launch_bounds__(kThreads)
draft_partial_kernel(DraftArgs a, int n_splits, float* __restrict__ part, int* __restrict__ status)
{
    constexpr int PITCH = D + 8;  // bf16 elements per shared row: 16 B of padding spreads the banks
    constexpr int CH = D / 8;     // 16-byte chunks per row
    __shared__ __align__(16) __nv_bfloat16 Ks[kTK * PITCH];
    __shared__ __align__(16) __nv_bfloat16 Vs[kTK * PITCH];
    __shared__ __align__(16) float Qs[kMaxGroup * D];
    __shared__ float S[kMaxGroup * kTK];
    __shared__ int keypos[kTK];
    __shared__ float m_run[kMaxGroup], l_run[kMaxGroup], alpha_s[kMaxGroup];

    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const int split = blockIdx.x, h = blockIdx.y;
    const int layer = blockIdx.z / a.kv.batch, b = blockIdx.z % a.kv.batch;
    const int64_t prob = (int64_t)blockIdx.z * a.kv.n_kv_heads + h;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const int n_rec = min(max(a.n_indices[prob], 0), a.k_total);
    const int ts = a.tail_start[b], cl = a.cur_len[b];
    const int n_tail = min(max(cl - ts, 0), a.max_tail);
    const int n = n_rec + n_tail;
    const int tiles = (n + kTK - 1) / kTK;
    const int per = (tiles + n_splits - 1) / n_splits * kTK;
    const int k0 = split * per;
    const int k1 = min(n, k0 + per);
    const int32_t* idx = a.indices + prob * a.k_total;

    for (int i = tid; i < G * D; i += kThreads) {
        const int g = i / D, d = i - g * D;
        const int64_t row = ((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + g;
        Qs[i] = __bfloat162float(a.q[row * D + d]);
    }
    if (tid < kMaxGroup) {
        m_run[tid] = -INFINITY;
        l_run[tid] = 0.f;
    }
    constexpr int NG = kThreads / (D / 2);
    const int dp = tid % (D / 2), rg = tid / (D / 2);
    float acc[kRPT][2];
#pragma unroll
    for (int i = 0; i < kRPT; ++i) acc[i][0] = acc[i][1] = 0.f;
    __syncthreads();

    for (int base = k0; base < k1; base += kTK) {
        const int nk = min(kTK, k1 - base);
        if (tid < kTK) {
            int pos = -1;
            if (tid < nk) {
                const int e = base + tid;
                pos = e < n_rec ? __ldg(idx + e) : ts + (e - n_rec);
                if (pos < 0 || pos >= cl) {
                    set_status(status, SPEC_ERR_BAD_INDEX);
                    pos = -1;
                }
            }
            keypos[tid] = pos;
        }
        __syncthreads();
        for (int c = tid; c < kTK * CH; c += kThreads) {
            const int row = c / CH, ch = c - row * CH;
            const int pos = keypos[row];
            if (pos >= 0) {
                const int64_t off = kv_row_offset(a.kv, layer, b, pos, h) + ch * 8;
                cp_async16(Ks + row * PITCH + ch * 8, a.kv.k + off);
                cp_async16(Vs + row * PITCH + ch * 8, a.kv.v + off);
            } else {
                *reinterpret_cast<uint4*>(Ks + row * PITCH + ch * 8) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(Vs + row * PITCH + ch * 8) = make_uint4(0, 0, 0, 0);
            }
        }
        cp_async_wait_all();
        __syncthreads();
        {  // scores: thread = (key, half of the rows)
            const int key = tid % kTK, part_id = tid / kTK;
            const bool ok = keypos[key] >= 0;
            for (int g = part_id; g < G; g += kThreads / kTK) {
                float dot = 0.f;
                const uint4* kr = reinterpret_cast<const uint4*>(Ks + key * PITCH);
                const float4* qr = reinterpret_cast<const float4*>(Qs + g * D);
#pragma unroll 4
                for (int c = 0; c < CH; ++c) {
                    const uint4 kk = kr[c];
                    const float4 q0 = qr[2 * c], q1 = qr[2 * c + 1];
                    dot += q0.x * bf16_lo(kk.x) + q0.y * bf16_hi(kk.x) + q0.z * bf16_lo(kk.y) +
                           q0.w * bf16_hi(kk.y) + q1.x * bf16_lo(kk.z) + q1.y * bf16_hi(kk.z) +
                           q1.z * bf16_lo(kk.w) + q1.w * bf16_hi(kk.w);
                }
                S[g * kTK + key] = ok ? dot * a.kv.scale : -INFINITY;
            }
        }
        __syncthreads();
        for (int g = warp; g < G; g += kThreads / 32) {  // online softmax, one warp per row
            const float v0 = S[g * kTK + lane], v1 = S[g * kTK + lane + 32];
            const float mt = warp_max(fmaxf(v0, v1));
            const float m_old = m_run[g];
            const float m_new = fmaxf(m_old, mt);
            float alpha = 1.f, p0 = 0.f, p1 = 0.f;
            if (m_new > -INFINITY) {
                alpha = expf(m_old - m_new);
                p0 = expf(v0 - m_new);
                p1 = expf(v1 - m_new);
            }
            S[g * kTK + lane] = p0;
            S[g * kTK + lane + 32] = p1;
            const float s = warp_sum(p0 + p1);
            if (lane == 0) {
                l_run[g] = l_run[g] * alpha + s;
                m_run[g] = m_new;
                alpha_s[g] = alpha;
            }
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kRPT; ++i) {
            const int r = rg + i * NG;
            if (r < G) {
                const float al = alpha_s[r];
                acc[i][0] *= al;
                acc[i][1] *= al;
            }
        }
        for (int key = 0; key < nk; ++key) {
            const uint32_t w = *reinterpret_cast<const uint32_t*>(Vs + key * PITCH + 2 * dp);
            const float v0 = bf16_lo(w), v1 = bf16_hi(w);
#pragma unroll
            for (int i = 0; i < kRPT; ++i) {
                const int r = rg + i * NG;
                if (r < G) {
                    const float p = S[r * kTK + key];
                    acc[i][0] += p * v0;
                    acc[i][1] += p * v1;
                }
            }
        }
        __syncthreads();
    }
    float* dst = part + (prob * n_splits + split) * (int64_t)G * (D + 2);
#pragma unroll
    for (int i = 0; i < kRPT; ++i) {
        const int r = rg + i * NG;
        if (r < G) *(reinterpret_cast<float2*>(dst + r * D) + dp) = make_float2(acc[i][0], acc[i][1]);
    }
    if (tid < G) {
        dst[G * D + tid] = m_run[tid];
        dst[G * D + G + tid] = l_run[tid];
    }
}

__global__ void draft_combine_kernel(DraftArgs a, int n_splits, const float* __restrict__ part)
{
    const int D = a.kv.head_dim, G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const int64_t prob = blockIdx.x;
    const int d = threadIdx.x;
    const int h = prob % a.kv.n_kv_heads;
    const int64_t lb = prob / a.kv.n_kv_heads;
    const int64_t stride = (int64_t)G * (D + 2);
    for (int g = 0; g < G; ++g) {
        float M = -INFINITY;
        for (int s = 0; s < n_splits; ++s) M = fmaxf(M, part[(prob * n_splits + s) * stride + G * D + g]);
        float Lsum = 0.f, o = 0.f;
        if (M > -INFINITY) {
            for (int s = 0; s < n_splits; ++s) {
                const float* p = part + (prob * n_splits + s) * stride;
                const float l = p[G * D + G + g];
                if (l > 0.f) {
                    const float w = expf(p[G * D + g] - M);
                    Lsum += l * w;
                    o += p[g * D + d] * w;
                }
            }
        }
        const int64_t row = lb * a.kv.n_q_heads + h * G + g;
        a.out[row * D + d] = Lsum > 0.f ? o / Lsum : 0.f;
        if (a.lse && d == 0) a.lse[row] = Lsum > 0.f ? M + logf(Lsum) : -INFINITY;
    }
}

}  // namespace

size_t draft_workspace(const KvView& kv, int n_keys_max) { return make_layout(kv, n_keys_max).total; }

int draft_launch(const DraftArgs& a, cudaStream_t stream)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    if (G > kMaxGroup) return SPEC_ERR_UNSUPPORTED_SHAPE;
    const Layout lo = make_layout(a.kv, a.k_total + a.max_tail);
    if (a.workspace_bytes < lo.total) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    char* ws = static_cast<char*>(a.workspace);
    float* part = reinterpret_cast<float*>(ws + lo.part_off);
    int* status = reinterpret_cast<int*>(ws);
    const dim3 grid(lo.n_splits, a.kv.n_kv_heads, a.kv.n_layers * a.kv.batch);
    const long probs = (long)a.kv.n_layers * a.kv.batch * a.kv.n_kv_heads;
    if (a.kv.head_dim == 128)
        draft_partial_kernel<128><<<grid, kThreads, 0, stream>>>(a, lo.n_splits, part, status);
    else if (a.kv.head_dim == 64)
        draft_partial_kernel<64><<<grid, kThreads, 0, stream>>>(a, lo.n_splits, part, status);
    else
        return SPEC_ERR_UNSUPPORTED_SHAPE;
    draft_combine_kernel<<<(unsigned)probs, a.kv.head_dim, 0, stream>>>(a, lo.n_splits, part);
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

}  // namespace spec
