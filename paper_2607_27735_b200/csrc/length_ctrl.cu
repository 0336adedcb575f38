// Entropy-guided speculation-length controller (Sec. "Entropy-Based Acceptance Prediction" and
// "Optimal Length Selection"): the entropy of each drafted token's output distribution, the two
// tracked class means (Eq. "ema"), the soft acceptance probabilities (Eq. "prob") and the length
// that maximises the expected tokens per unit cost (Eq. "optimal_k").
//
// The entropy is the only part with real data behind it: one pass over rows x vocabulary logits
// (HBM-bound; 256 KB per row at a 128K vocabulary in bf16).  A row is split over a thread-block
// cluster when there are few rows, so that a single drafted token still uses several SMs; every
// thread keeps a running (max, sum e^(z-max), sum e^(z-max) z) and H = max + ln S - T / S.
// The two controller steps are a handful of scalars: one warp each, results stay in device
// memory so that a captured graph can branch on them without a host round trip.
#include <cooperative_groups.h>

#include <cstdlib>

#include "spec_common.cuh"

namespace cg = cooperative_groups;

namespace spec {

namespace {

constexpr int kEntThreads = 512;
constexpr int kMaxDrafted = 256;  // drafted tokens the controller looks at in one call

struct Mst {  // running maximum, sum of e^(z - m), sum of e^(z - m) * z
    float m, s, t;
};

__device__ __forceinline__ Mst merge(const Mst& a, const Mst& b)
{
    const float m = fmaxf(a.m, b.m);
    const float fa = __expf(a.m - m), fb = __expf(b.m - m);
    return Mst{m, a.s * fa + b.s * fb, a.t * fa + b.t * fb};
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr int kUnroll = 4;  // 16-byte loads a thread keeps in flight
constexpr float kNegInf = -__builtin_huge_valf();

struct Arg {  // largest logit seen and the smallest index that holds it
    float v;
    int i;
};

__device__ __forceinline__ Arg merge(const Arg& a, const Arg& b)
{
    return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// eight logits z (group maximum cm) starting at vocabulary index v0
template <bool ENT, bool ARG>
__device__ __forceinline__ void fold8(Mst& acc, Arg& arg, const float (&z)[8], float cm, int v0)
{
    if (ARG && cm > arg.v) {  // rare after the first groups: the running maximum seldom moves
        int first = 7;
#pragma unroll
        for (int i = 6; i >= 0; --i) first = z[i] == cm ? i : first;
        arg = Arg{cm, v0 + first};
    }
    if (ENT) {
        const float mn = fmaxf(acc.m, cm), mb = mn * kLog2e;
        const float f = ex2(fmaf(acc.m, kLog2e, -mb));
        float s = acc.s * f, t = acc.t * f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float e = ex2(fmaf(z[i], kLog2e, -mb));
            s += e;
            t = fmaf(e, z[i], t);
        }
        acc = Mst{mn, s, t};
    }
}

template <bool ENT, bool ARG>
__device__ __forceinline__ void fold1(Mst& acc, Arg& arg, float z, int v)
{
    if (ARG && z > arg.v) arg = Arg{z, v};
    if (ENT) {
        const float mn = fmaxf(acc.m, z), mb = mn * kLog2e;
        const float f = ex2(fmaf(acc.m, kLog2e, -mb)), e = ex2(fmaf(z, kLog2e, -mb));
        acc = Mst{mn, fmaf(acc.s, f, e), fmaf(acc.t, f, e * z)};
    }
}

__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

template <bool ENT, bool ARG>
__device__ __forceinline__ void fold_words(Mst& acc, Arg& arg, const uint4& w, int v0)  // eight bf16 logits
{
    const uint32_t mx = bf16x2_max(bf16x2_max(w.x, w.y), bf16x2_max(w.z, w.w));
    const float z[8] = {bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y),
                        bf16_lo(w.z), bf16_hi(w.z), bf16_lo(w.w), bf16_hi(w.w)};
    fold8<ENT, ARG>(acc, arg, z, fmaxf(bf16_lo(mx), bf16_hi(mx)), v0);
}

template <bool ENT, bool ARG>
__device__ __forceinline__ void fold_words(Mst& acc, Arg& arg, const float4& a, const float4& b, int v0)  // eight fp32
{
    const float z[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    fold8<ENT, ARG>(acc, arg, z,
                    fmaxf(fmaxf(fmaxf(a.x, a.y), fmaxf(a.z, a.w)), fmaxf(fmaxf(b.x, b.y), fmaxf(b.z, b.w))), v0);
}

template <int DT>
__device__ __forceinline__ float load_logit(const void* base, int v)
{
    return DT == 1 ? __bfloat162float(static_cast<const __nv_bfloat16*>(base)[v]) : static_cast<const float*>(base)[v];
}

// One cluster (gridDim.x CTAs) per row.  DT = 0: fp32 logits, 1: bf16 logits.  ENT: entropy[row];
// ARG: token[row] = the smallest index of the largest logit.
template <int DT, bool ENT, bool ARG>
__global__ void __launch_bounds__(kEntThreads) row_kernel(const void* __restrict__ logits, int vocab, int64_t row_stride,
                                                          float* __restrict__ entropy, int32_t* __restrict__ token)
{
    cg::cluster_group cluster = cg::this_cluster();
    __shared__ Mst warp_part[kEntThreads / 32];
    __shared__ Arg warp_arg[kEntThreads / 32];
    __shared__ Mst cta_part;
    __shared__ Arg cta_arg;
    const int CS = gridDim.x, rank = blockIdx.x, row = blockIdx.y;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const char* base = static_cast<const char*>(logits) + (int64_t)row * row_stride * (DT == 1 ? 2 : 4);
    Mst acc{-3.0e38f, 0.f, 0.f};
    Arg arg{kNegInf, 0x7fffffff};
    if ((reinterpret_cast<uintptr_t>(base) & 15) == 0) {
        // whole groups of 8 logits, a contiguous share per CTA; the ragged end goes to the last CTA
        const int groups = vocab / 8;
        const int g_per = (groups + CS - 1) / CS;
        const int g0 = min(groups, rank * g_per), g1 = min(groups, g0 + g_per);
        for (int g = g0 + tid; g < g1; g += kUnroll * kEntThreads) {
            if (DT == 1) {
                uint4 w[kUnroll];
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (g + j * kEntThreads < g1)
                        w[j] = __ldg(reinterpret_cast<const uint4*>(base) + g + j * kEntThreads);
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (g + j * kEntThreads < g1) fold_words<ENT, ARG>(acc, arg, w[j], (g + j * kEntThreads) * 8);
            } else {
                float4 w[kUnroll][2];
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (g + j * kEntThreads < g1) {
                        w[j][0] = __ldg(reinterpret_cast<const float4*>(base) + 2 * (g + j * kEntThreads));
                        w[j][1] = __ldg(reinterpret_cast<const float4*>(base) + 2 * (g + j * kEntThreads) + 1);
                    }
#pragma unroll
                for (int j = 0; j < kUnroll; ++j)
                    if (g + j * kEntThreads < g1)
                        fold_words<ENT, ARG>(acc, arg, w[j][0], w[j][1], (g + j * kEntThreads) * 8);
            }
        }
        if (rank == CS - 1 && groups * 8 + tid < vocab)
            fold1<ENT, ARG>(acc, arg, load_logit<DT>(base, groups * 8 + tid), groups * 8 + tid);
    } else {
        // a row that does not start on a 16-byte boundary: element by element
        const int per = (vocab + CS - 1) / CS;
        const int v0 = min(vocab, rank * per), v1 = min(vocab, v0 + per);
        for (int v = v0 + tid; v < v1; v += kEntThreads) fold1<ENT, ARG>(acc, arg, load_logit<DT>(base, v), v);
    }
    // warp, CTA, cluster: merged in a fixed order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        if (ENT) {
            Mst other{__shfl_xor_sync(0xffffffffu, acc.m, o), __shfl_xor_sync(0xffffffffu, acc.s, o),
                      __shfl_xor_sync(0xffffffffu, acc.t, o)};
            acc = merge(acc, other);
        }
        if (ARG) {
            Arg other{__shfl_xor_sync(0xffffffffu, arg.v, o), __shfl_xor_sync(0xffffffffu, arg.i, o)};
            arg = merge(arg, other);
        }
    }
    if (lane == 0) {
        warp_part[warp] = acc;
        warp_arg[warp] = arg;
    }
    __syncthreads();
    if (tid == 0) {
        Mst a = warp_part[0];
        Arg g = warp_arg[0];
        for (int w = 1; w < kEntThreads / 32; ++w) {
            if (ENT) a = merge(a, warp_part[w]);
            if (ARG) g = merge(g, warp_arg[w]);
        }
        cta_part = a;
        cta_arg = g;
    }
    if (CS > 1) cluster.sync(); else __syncthreads();
    if (rank == 0 && tid == 0) {
        Mst a = cta_part;
        Arg g = cta_arg;
        for (int c = 1; c < CS; ++c) {
            if (ENT) a = merge(a, *cluster.map_shared_rank(&cta_part, c));
            if (ARG) g = merge(g, *cluster.map_shared_rank(&cta_arg, c));
        }
        if (ENT) entropy[row] = a.s > 0.f ? a.m + __logf(a.s) - a.t / a.s : 0.f;
        if (ARG) token[row] = g.i == 0x7fffffff ? 0 : g.i;
    }
    if (CS > 1) cluster.sync();  // nobody leaves while its partial may still be read
}

// Greedy prefix acceptance: drafted token i of a sequence is accepted iff every earlier one was and
// it equals the target's token for that position; one thread per sequence.
__global__ void accept_kernel(const int32_t* __restrict__ target, const int32_t* __restrict__ draft,
                              const int32_t* __restrict__ n_draft, int batch, int k1,
                              int32_t* __restrict__ n_accepted, int32_t* __restrict__ next_token)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int nd = n_draft ? min(max(n_draft[b], 0), k1 - 1) : k1 - 1;
    int m = 0;
    while (m < nd && draft[b * (k1 - 1) + m] == target[b * k1 + m]) ++m;
    n_accepted[b] = m;
    next_token[b] = target[b * k1 + m];
}

// Eq. "ema": state[0] <- beta state[0] + (1 - beta) mean(H_1..H_m), state[1] likewise with H_{m+1}..H_k
__global__ void controller_update_kernel(float* state, const float* __restrict__ entropy, int k,
                                         const int32_t* __restrict__ n_accepted, float beta)
{
    const int lane = threadIdx.x;
    const int m = min(max(*n_accepted, 0), k);
    float sa = 0.f, sr = 0.f;
    for (int i = lane; i < k; i += 32) {
        const float h = entropy[i];
        if (i < m) sa += h; else sr += h;
    }
    sa = warp_sum(sa);
    sr = warp_sum(sr);
    if (lane == 0) {
        if (m > 0) state[0] = beta * state[0] + (1.f - beta) * (sa / m);
        if (m < k) state[1] = beta * state[1] + (1.f - beta) * (sr / (k - m));
    }
}

// Eq. "prob" and Eq. "optimal_k"; ties go to the smaller candidate
__global__ void controller_select_kernel(const float* __restrict__ state, const float* __restrict__ entropy, int n,
                                         const int32_t* __restrict__ cand, int n_cand, float c_d, float c_v,
                                         int32_t* k_star, float* p_out, float* score_out)
{
    __shared__ float expected[kMaxDrafted];  // 1 + sum_{m <= k} prod_{i <= m} p_i at k = index + 1
    const int lane = threadIdx.x;
    const float acc_c = state[0], rej_c = state[1];
    for (int i = lane; i < n; i += 32) {
        const float a = __expf(-fabsf(entropy[i] - acc_c)), b = __expf(-fabsf(entropy[i] - rej_c));
        const float p = a / (a + b);
        expected[i] = p;
        if (p_out) p_out[i] = p;
    }
    __syncwarp();
    if (lane == 0) {
        float prefix = 1.f, e = 1.f;
        for (int i = 0; i < n; ++i) {
            prefix *= expected[i];
            e += prefix;
            expected[i] = e;
        }
        int best = 0;
        float best_score = -1.f;
        for (int c = 0; c < n_cand; ++c) {
            const int k = cand[c];
            float score = -1.f;  // a candidate outside 1..n never wins
            if (k >= 1 && k <= n) score = expected[k - 1] / (k * c_d + c_v);
            if (score_out) score_out[c] = score;
            if (score >= 0.f && (score > best_score || (score == best_score && k < best))) {
                best_score = score;
                best = k;
            }
        }
        *k_star = best;
    }
}

// Lengths of the next round, on the device: committed += accepted + 1 (the corrected token), the
// verification context of a round with k drafted tokens, and the draft step lengths.
__global__ void advance_lengths_kernel(int32_t* __restrict__ committed, const int32_t* __restrict__ n_accepted,
                                       int batch, int k, int32_t* __restrict__ ctx_verify,
                                       int32_t* __restrict__ cur_len, int max_len, int* __restrict__ status)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    int t = committed[b] + (n_accepted ? min(max(n_accepted[b], 0), k) + 1 : 0);
    if (max_len > 0 && t + k + 1 > max_len) {  // the next round would leave the cache: hold the sequence and say so
        t = max(max_len - k - 1, 0);
        if (status) atomicCAS(status, 0, SPEC_ERR_BAD_INDEX);
    }
    committed[b] = t;
    if (ctx_verify) ctx_verify[b] = t + k + 1;
    if (cur_len)
        for (int j = 0; j < k; ++j) cur_len[j * batch + b] = t + j + 1;
}

}  // namespace

template <int DT, bool ENT, bool ARG>
static cudaError_t launch_rows(const cudaLaunchConfig_t& cfg, const void* logits, int vocab, int64_t row_stride,
                               float* entropy, int32_t* token)
{
    return cudaLaunchKernelEx(&cfg, row_kernel<DT, ENT, ARG>, logits, vocab, row_stride, entropy, token);
}

// entropy and/or token may be null (not both)
int rows_launch(const void* logits, int dtype, int n_rows, int vocab, int64_t row_stride, float* entropy,
                int32_t* token, cudaStream_t stream)
{
    // A row is worth splitting only while the rows alone leave SMs idle: one SM needs about 4 us
    // for the 128K exponentials of a row (16 per clock), but a cluster costs a few hundred
    // nanoseconds of barriers, which shows once every SM has two CTAs anyway.  No CTA without a
    // full sweep of its threads.
    int cs = 8;
    while (cs > 1 && (long)n_rows * cs > 2L * sm_count()) cs /= 2;
    while (cs > 1 && vocab < cs * 8 * kEntThreads) cs /= 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(cs, n_rows);
    cfg.blockDim = dim3(kEntThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err;
    if (entropy && token)
        err = dtype == 1 ? launch_rows<1, true, true>(cfg, logits, vocab, row_stride, entropy, token)
                         : launch_rows<0, true, true>(cfg, logits, vocab, row_stride, entropy, token);
    else if (entropy)
        err = dtype == 1 ? launch_rows<1, true, false>(cfg, logits, vocab, row_stride, entropy, token)
                         : launch_rows<0, true, false>(cfg, logits, vocab, row_stride, entropy, token);
    else
        err = dtype == 1 ? launch_rows<1, false, true>(cfg, logits, vocab, row_stride, entropy, token)
                         : launch_rows<0, false, true>(cfg, logits, vocab, row_stride, entropy, token);
    if (err != cudaSuccess) {
        cudaGetLastError();
        return SPEC_ERR_CUDA;
    }
    count_launch(1);
    return SPEC_OK;
}

int accept_launch(const int32_t* target, const int32_t* draft, const int32_t* n_draft, int batch, int k1,
                  int32_t* n_accepted, int32_t* next_token, cudaStream_t stream)
{
    accept_kernel<<<(batch + 127) / 128, 128, 0, stream>>>(target, draft, n_draft, batch, k1, n_accepted, next_token);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    count_launch(1);
    return SPEC_OK;
}

int advance_lengths_launch(int32_t* committed, const int32_t* n_accepted, int batch, int k, int max_len, int* status, int32_t* ctx_verify,
                           int32_t* cur_len, cudaStream_t stream)
{
    advance_lengths_kernel<<<(batch + 127) / 128, 128, 0, stream>>>(committed, n_accepted, batch, k, ctx_verify, cur_len, max_len, status);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    count_launch(1);
    return SPEC_OK;
}

int controller_update_launch(float* state, const float* entropy, int k, const int32_t* n_accepted, float beta,
                             cudaStream_t stream)
{
    controller_update_kernel<<<1, 32, 0, stream>>>(state, entropy, k, n_accepted, beta);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    count_launch(1);
    return SPEC_OK;
}

int controller_select_launch(const float* state, const float* entropy, int n, const int32_t* cand, int n_cand,
                             float c_d, float c_v, int32_t* k_star, float* p_out, float* score_out,
                             cudaStream_t stream)
{
    if (n > kMaxDrafted) return SPEC_ERR_UNSUPPORTED_SHAPE;
    controller_select_kernel<<<1, 32, 0, stream>>>(state, entropy, n, cand, n_cand, c_d, c_v, k_star, p_out, score_out);
    if (cudaGetLastError() != cudaSuccess) return SPEC_ERR_CUDA;
    count_launch(1);
    return SPEC_OK;
}

}  // namespace spec
