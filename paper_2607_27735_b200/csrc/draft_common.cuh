// Pieces shared by the sparse draft attention kernels: PTX wrappers (cp.async, ldmatrix,
// distributed-shared-memory stores counted on an mbarrier), the bounded wait of a cluster's first
// CTA for the other CTAs' partial results, the rank-ordered merge, and per-device launch set-up.
#pragma once

#include "spec_common.cuh"

namespace spec {

// Split of a call of the streaming kernel (see draft_stream.cu).
struct StreamShape {
    int cs;   // CTAs per cluster; one cluster per (layer, sequence, KV head)
    int per;  // keys per CTA, a multiple of 16
    int nw;   // warps per CTA
    int st;   // shared-memory stages per warp
};
bool stream_plan(const KvView& kv, int head_dim, int n_keys_max, StreamShape* out);
int draft_stream_launch(const DraftArgs& a, const StreamShape& shp, cudaStream_t stream);

namespace draft {

constexpr int kMaxGroup = 8;    // query heads per KV head
constexpr int kMaxCluster = 8;  // portable cluster size
constexpr float kNegBig = -1.0e30f;  // "minus infinity" that stays finite under subtraction
constexpr size_t kSmemLimit = 227 * 1024;

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// 16 bytes global -> shared; src_bytes = 0 writes zeros instead (masked rows)
__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc, uint32_t src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_addr(smem_dst)), "l"(gsrc), "r"(src_bytes)
                 : "memory");
}
// asks L2 for `bytes` (a multiple of 16, from a 16-byte aligned address); nothing waits for it
__device__ __forceinline__ void prefetch_l2(const void* gsrc, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(gsrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
// Stores into the shared memory of another CTA of the cluster; the bytes are counted on that CTA's
// mbarrier when they have landed (no fence, no cluster barrier needed on either side).
// Two neighbouring floats (the address a multiple of 8):
__device__ __forceinline__ void st_async_f32x2(uint32_t remote_addr, float v0, float v1, uint32_t remote_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];"
                 ::"r"(remote_addr), "r"(__float_as_uint(v0)), "r"(__float_as_uint(v1)), "r"(remote_bar) : "memory");
}
// and for four (the address a multiple of 16)
__device__ __forceinline__ void st_async_f32x4(uint32_t remote_addr, float4 v, uint32_t remote_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
                 ::"r"(remote_addr), "r"(__float_as_uint(v.x)), "r"(__float_as_uint(v.y)), "r"(__float_as_uint(v.z)),
                   "r"(__float_as_uint(v.w)), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(p)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_addr(p)));
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// The first CTA of a cluster waits until every byte the others deposit has landed.  Bounded: after
// `limit` SM clocks the status word gets SPEC_ERR_TIMEOUT and the CTA goes on with what it has.
__device__ __forceinline__ void wait_deposits(uint32_t bar, long long limit, int* status)
{
    if (mbar_try_wait(bar, 0)) return;
    const long long t_start = clock64();
    while (!mbar_try_wait(bar, 0)) {
        if (clock64() - t_start > limit) {
            set_status(status, SPEC_ERR_TIMEOUT);
            break;
        }
    }
}

// Merge of the cluster's partial results in the first CTA, in rank order (deterministic), and the
// store of the normalised output rows.  comb: [cs][G * (D + 2)] = O rows [G][D], then (maximum, sum) per head.
template <int D, int NT>
__device__ __forceinline__ void merge_and_store(const DraftArgs& a, const float* comb, int CS, int G, int layer, int b,
                                                int h, int tid)
{
    const int PS = G * (D + 2);
    for (int i = tid; i < G * (D / 2); i += NT) {
        const int r = i / (D / 2), dp = i - r * (D / 2);
        float2 ml[kMaxCluster], oc[kMaxCluster];
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) {  // every load is in flight before the first is used
            if (c < CS) {
                const float* pc = comb + c * PS;
                ml[c] = *(reinterpret_cast<const float2*>(pc + G * D) + r);
                oc[c] = *(reinterpret_cast<const float2*>(pc + r * D) + dp);
            }
        }
        float M = kNegBig;
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c)
            if (c < CS) M = fmaxf(M, ml[c].x);
        float Lsum = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) {
            if (c < CS && ml[c].y > 0.f) {
                const float wgt = ex2f(ml[c].x - M);
                Lsum += ml[c].y * wgt;
                o0 += oc[c].x * wgt;
                o1 += oc[c].y * wgt;
            }
        }
        const int64_t row = ((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + r;
        const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
        if (a.out_bf16)
            *(reinterpret_cast<uint32_t*>(reinterpret_cast<__nv_bfloat16*>(a.out) + row * D) + dp) = pack_bf16(o0 * inv, o1 * inv);
        else
            *(reinterpret_cast<float2*>(a.out + row * D) + dp) = make_float2(o0 * inv, o1 * inv);
        if (a.lse && dp == 0) a.lse[row] = Lsum > 0.f ? (M + log2f(Lsum)) * 0.69314718055994530942f : -INFINITY;
    }
}

// Opts a kernel into `smem` bytes of dynamic shared memory on the current device (the attribute
// is per device and per function: remembered for each pair, up to 64 devices).
bool opt_in_smem(const void* kernel, size_t smem);

}  // namespace draft
}  // namespace spec
