// Sparse draft attention of Eq. 5: one query per sequence attends the recalled rows
// Gather(K, I), Gather(V, I) plus the dense tail of tokens drafted this round.  The gather is
// fused: one bulk asynchronous copy (cp.async.bulk, completion on an mbarrier) per indexed
// 2*D-byte row pulls K and V straight from the dense cache into shared memory (two 144-key
// tiles in flight per CTA); nothing gathered is written back to global memory.
//
// The call is latency-bound (a few thousand recalled keys per head), so the kernel is built to
// be short rather than wide:
//   - every warp is an independent flash-decoding worker on 16 keys of each tile: q K^T and
//     P V run on the tensor cores (mma.sync m16n8k16, the G <= 8 query rows of the GQA group
//     padded to 16; P split into bf16 hi + lo parts), its running (max, sum, O) stay in
//     registers, and no block-wide barrier is needed inside a tile;
//   - the warps of a CTA are merged once through shared memory, the CTAs of a problem (a
//     thread-block cluster that splits the key list) once through distributed shared memory:
//     each deposits its partial in the first CTA of the cluster, which merges them in rank
//     order (deterministic) after one cluster barrier.
// One launch per call, no global scratch, no second kernel.
#include <cooperative_groups.h>

#include "spec_common.cuh"

namespace cg = cooperative_groups;

namespace spec {

namespace {

constexpr int kTK = 144;       // keys per tile: nine 16-key chunks dealt to the 8 warps
constexpr int kStages = 2;     // two tiles (288 keys) can be in flight per CTA
constexpr int kThreads = 256;
constexpr int kMaxGroup = 8;   // query heads per KV head
constexpr int kMaxCluster = 8;  // portable cluster size (16 was measured slower: one cluster per GPC)
constexpr long long kTimeoutCycles = 2000ll * 1000ll * 1000ll;  // bound of the copy wait: about a second

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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
// one row of the cache -> shared memory (16-byte aligned on both sides, size a multiple of 16)
__device__ __forceinline__ void bulk_copy_row(void* smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(smem_dst)), "l"(gsrc), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p)
{
    const uint32_t a = (uint32_t)__cvta_generic_to_shared(p);
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(a));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2f(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

template <int D>
struct SmemLayout {
    static constexpr int PITCH = D + 8;  // bf16 elements per shared row: 16 B of padding spreads the banks
    static constexpr int kv_tile = kTK * PITCH * 2;  // bytes of one K (or V) tile
    static constexpr int off_k = 0;
    static constexpr int off_v = kStages * kv_tile;
    static constexpr int off_q = 2 * kStages * kv_tile;              // bf16 [16][PITCH], rows >= G zero
    static constexpr int off_pos = off_q + 16 * PITCH * 2;           // int [kStages][kTK]
    static constexpr int off_bar = off_pos + kStages * kTK * 4;      // mbarrier [kStages]
    static constexpr int off_wml = off_bar + 64;                     // float2 [8 warps][kMaxGroup]
    static constexpr int off_wo = off_k;  // float [8 warps][kMaxGroup][D]: reuses the K tiles once the loop is over
    static constexpr int off_comb = off_wml + 8 * kMaxGroup * 8;     // float [kMaxCluster][kMaxGroup][D + 2]
    static constexpr int total = off_comb + kMaxCluster * kMaxGroup * (D + 2) * 4;
    static_assert(8 * kMaxGroup * D * 4 <= kStages * kv_tile, "warp partials must fit in the K tiles");
    static_assert(PITCH * 2 % 16 == 0, "bulk copies need 16-byte aligned rows");
    static_assert(total <= 227 * 1024, "shared memory budget");
};

template <int D>
__global__ void __launch_bounds__(kThreads)
draft_cluster_kernel(DraftArgs a, int* __restrict__ status)
{
    using SL = SmemLayout<D>;
    constexpr int PITCH = SL::PITCH;
    constexpr int CH = D / 8;    // 16-byte chunks per row
    constexpr int NT = D / 8;    // 8-wide output tiles of the P V product
    constexpr float kLog2e = 1.4426950408889634f;
    extern __shared__ __align__(16) uint8_t smem[];
    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem + SL::off_k);
    __nv_bfloat16* Vs = reinterpret_cast<__nv_bfloat16*>(smem + SL::off_v);
    __nv_bfloat16* Qs = reinterpret_cast<__nv_bfloat16*>(smem + SL::off_q);
    int* keypos = reinterpret_cast<int*>(smem + SL::off_pos);
    float2* wml = reinterpret_cast<float2*>(smem + SL::off_wml);
    float* wo = reinterpret_cast<float*>(smem + SL::off_wo);
    float* comb = reinterpret_cast<float*>(smem + SL::off_comb);

#ifdef SPEC_TRACE
#define DSTAMP(i) do { if (threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) reinterpret_cast<long long*>(status)[8 + (i)] = clock64(); } while (0)
#else
#define DSTAMP(i) do { } while (0)
#endif
    DSTAMP(0);
    cg::cluster_group cluster = cg::this_cluster();
    const int CS = gridDim.x;              // the cluster spans the x dimension
    const int rank = blockIdx.x;
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const int h = blockIdx.y;
    const int layer = blockIdx.z / a.kv.batch, b = blockIdx.z % a.kv.batch;
    const int64_t prob = (int64_t)blockIdx.z * a.kv.n_kv_heads + h;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // Programmatic dependent launch: the next kernel in the stream may start its own prologue
    // (index loads, gather of recalled rows) while this one is still computing.  Everything this
    // kernel reads before griddep_wait() below is immutable during a drafting round (indices,
    // lengths, recalled rows of the dense cache); Q, the dense tail and the outputs come after.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    bool dep_waited = false;
    auto griddep_wait = [&]() {
        if (!dep_waited) {
            asm volatile("griddepcontrol.wait;" ::: "memory");
            dep_waited = true;
        }
    };
    const uint32_t bar0 = smem_addr(smem + SL::off_bar);
    if (tid == 0) {
        for (int i = 0; i < kStages; ++i) mbar_init(bar0 + 8 * i, kTK);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const int32_t* idx = a.indices + prob * a.k_total;
    // the index of this thread's row in the first tile is fetched before the list length is
    // known (the tail of the array holds -1 padding, never read past k_total)
    const int per_guess = ((a.k_total + a.max_tail + CS - 1) / CS + 15) & ~15;
    int idx_pre = -1;
    if (tid < kTK && rank * per_guess + tid < a.k_total) idx_pre = __ldg(idx + rank * per_guess + tid);
    const int n_rec = min(max(__ldg(a.n_indices + prob), 0), a.k_total);
    const int ts = __ldg(a.tail_start + b), cl = __ldg(a.cur_len + b);
    const int n_tail = min(max(cl - ts, 0), a.max_tail);
    const int n = n_rec + n_tail;
    // contiguous shares in multiples of the 16-key chunk; the share size depends only on host-side
    // bounds, so every CTA of the cluster agrees on it without exchanging anything
    const int per = per_guess;
    const int k0 = min(n, rank * per);
    const int k1 = min(n, k0 + per);
    const int n_tiles = (k1 - k0 + kTK - 1) / kTK;
    __syncthreads();  // barriers initialised

    // one thread per row: position, then one bulk copy each for the K row and the V row; every
    // copy of the tile is in flight before anything waits
    auto issue_tile = [&](int tile) {
        const int buf = tile % kStages;
        const int base = k0 + tile * kTK;
        const int nk = min(kTK, k1 - base);
        if (base + nk > n_rec) griddep_wait();  // the tile reaches into the tail drafted this round
        if (tid >= kTK) return;
        const uint32_t bar = bar0 + 8 * buf;
        int pos = -1;
        if (tid < nk) {
            const int e = base + tid;
            pos = e < n_rec ? (tile == 0 ? idx_pre : __ldg(idx + e)) : ts + (e - n_rec);
            if (pos < 0 || pos >= cl) {
                set_status(status, SPEC_ERR_BAD_INDEX);
                pos = -1;
            }
        }
        keypos[buf * kTK + tid] = pos;
        __nv_bfloat16* kr = Ks + (buf * kTK + tid) * PITCH;
        __nv_bfloat16* vr = Vs + (buf * kTK + tid) * PITCH;
        if (pos >= 0) {
            const int64_t off = kv_row_offset(a.kv, layer, b, pos, h);
            mbar_arrive_expect_tx(bar, 2 * D * 2);
            bulk_copy_row(kr, a.kv.k + off, D * 2, bar);
            bulk_copy_row(vr, a.kv.v + off, D * 2, bar);
        } else {  // masked rows must still be finite: they meet P = 0 in the P V product
#pragma unroll
            for (int ch = 0; ch < CH; ++ch) {
                *reinterpret_cast<uint4*>(kr + ch * 8) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(vr + ch * 8) = make_uint4(0, 0, 0, 0);
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // a later bulk copy reuses the row
            mbar_arrive(bar);
        }
    };

    int issued = 0;
    for (; issued < min(n_tiles, kStages); ++issued) issue_tile(issued);

    DSTAMP(1);
    griddep_wait();
    DSTAMP(2);
    // Q of the group -> bf16 [16][PITCH] in shared memory (rows >= G zero), then A fragments
    for (int i = tid; i < 16 * CH; i += kThreads) {
        const int g = i / CH, ch = i - g * CH;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (g < G) {
            const int64_t row = ((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + g;
            val = __ldg(reinterpret_cast<const uint4*>(a.q + row * D) + ch);
        }
        *reinterpret_cast<uint4*>(Qs + g * PITCH + ch * 8) = val;
    }
    __syncthreads();
    uint32_t qa[D / 16][4];
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks)
        ldmatrix_x4(qa[ks], Qs + ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + ks * 16 + (lane >> 4) * 8);

    DSTAMP(3);
    // per-warp flash-decoding state: the thread owns row g = lane / 4 (and the padding row g + 8)
    const int g_row = lane >> 2, quad = lane & 3;
    const float sc = a.kv.scale * kLog2e;
    float m_run = -INFINITY, l_run = 0.f;
    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f;

    for (int tile = 0; tile < n_tiles; ++tile) {
        const int buf = tile % kStages;
        {  // the tile's rows have landed (bounded wait: a stall ends in a status code)
            const uint32_t bar = bar0 + 8 * buf, parity = (tile / kStages) & 1;
            const long long t0 = clock64();
            while (!mbar_try_wait(bar, parity)) {
                if (clock64() - t0 > kTimeoutCycles) {
                    set_status(status, SPEC_ERR_TIMEOUT);
                    break;
                }
            }
        }
        const int nk = min(kTK, k1 - (k0 + tile * kTK));
        for (int ck = warp * 16; ck < nk; ck += 8 * 16) {  // this warp's 16-key chunks of the tile
            const int* kp = keypos + buf * kTK;
            const __nv_bfloat16* kb = Ks + (buf * kTK + ck) * PITCH;
            const __nv_bfloat16* vb = Vs + (buf * kTK + ck) * PITCH;
            // ---- S = q K^T for 16 keys: two 8-key output tiles ----
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
                uint32_t kf[4];
                ldmatrix_x4(kf, kb + ((lane & 7) + (lane >> 4) * 8) * PITCH + ks * 16 + ((lane >> 3) & 1) * 8);
                mma_bf16(s0, qa[ks], kf[0], kf[1]);
                mma_bf16(s1, qa[ks], kf[2], kf[3]);
            }
            // the thread's keys: ck + 2*quad + {0,1} (tile 0) and + 8 (tile 1); rows g_row (real) only
            const int kA = ck + 2 * quad;
            float v0 = kp[kA] >= 0 ? s0[0] * sc : -INFINITY;
            float v1 = kp[kA + 1] >= 0 ? s0[1] * sc : -INFINITY;
            float v2 = kp[kA + 8] >= 0 ? s1[0] * sc : -INFINITY;
            float v3 = kp[kA + 9] >= 0 ? s1[1] * sc : -INFINITY;
            float mt = fmaxf(fmaxf(v0, v1), fmaxf(v2, v3));
            mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 1));
            mt = fmaxf(mt, __shfl_xor_sync(0xffffffffu, mt, 2));
            const float m_new = fmaxf(m_run, mt);
            float alpha = 1.f, p0 = 0.f, p1 = 0.f, p2 = 0.f, p3 = 0.f;
            if (m_new > -INFINITY) {
                alpha = ex2f(m_run - m_new);
                p0 = ex2f(v0 - m_new);
                p1 = ex2f(v1 - m_new);
                p2 = ex2f(v2 - m_new);
                p3 = ex2f(v3 - m_new);
            }
            m_run = m_new;
            l_run = l_run * alpha + (p0 + p1) + (p2 + p3);
            // ---- P (hi + lo bf16) as the A operand of P V; padding rows (g_row + 8) are zero ----
            uint32_t ph[4], pl[4];
            ph[0] = pack_bf16x2(p0, p1);
            ph[2] = pack_bf16x2(p2, p3);
            ph[1] = ph[3] = 0u;
            pl[0] = pack_bf16x2(p0 - __uint_as_float(ph[0] << 16), p1 - __uint_as_float(ph[0] & 0xffff0000u));
            pl[2] = pack_bf16x2(p2 - __uint_as_float(ph[2] << 16), p3 - __uint_as_float(ph[2] & 0xffff0000u));
            pl[1] = pl[3] = 0u;
#pragma unroll
            for (int nt = 0; nt < NT; nt += 2) {
                uint32_t vf[4];
                ldmatrix_x4_trans(vf, vb + ((lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + nt * 8 + (lane >> 4) * 8);
                o[nt][0] *= alpha;
                o[nt][1] *= alpha;
                o[nt + 1][0] *= alpha;
                o[nt + 1][1] *= alpha;
                mma_bf16(o[nt], ph, vf[0], vf[1]);
                mma_bf16(o[nt], pl, vf[0], vf[1]);
                mma_bf16(o[nt + 1], ph, vf[2], vf[3]);
                mma_bf16(o[nt + 1], pl, vf[2], vf[3]);
            }
        }
        __syncthreads();  // the tile's buffer is free again
        if (issued < n_tiles) {
            issue_tile(issued);
            ++issued;
        }
    }

    DSTAMP(4);
    // ---- merge the 8 warps of the CTA ----
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
    l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
    if (g_row < G) {
        if (quad == 0) wml[warp * kMaxGroup + g_row] = make_float2(m_run, l_run);
        float* dst = wo + (warp * kMaxGroup + g_row) * D + 2 * quad;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) *reinterpret_cast<float2*>(dst + nt * 8) = make_float2(o[nt][0], o[nt][1]);
    }
    __syncthreads();
    float* comb0 = CS > 1 ? cluster.map_shared_rank(comb, 0) : comb;
    float* mine = comb0 + rank * (kMaxGroup * (D + 2));
    for (int i = tid; i < G * (D / 2); i += kThreads) {
        const int r = i / (D / 2), dp = i - r * (D / 2);
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 8; ++w) M = fmaxf(M, wml[w * kMaxGroup + r].x);
        float Lsum = 0.f, o0 = 0.f, o1 = 0.f;
        if (M > -INFINITY) {
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                const float2 ml = wml[w * kMaxGroup + r];
                if (ml.y > 0.f) {
                    const float wgt = ex2f(ml.x - M);
                    const float2 ov = *(reinterpret_cast<const float2*>(wo + (w * kMaxGroup + r) * D) + dp);
                    Lsum += ml.y * wgt;
                    o0 += ov.x * wgt;
                    o1 += ov.y * wgt;
                }
            }
        }
        *(reinterpret_cast<float2*>(mine + r * D) + dp) = make_float2(o0, o1);
        if (dp == 0) {
            mine[kMaxGroup * D + r] = M;
            mine[kMaxGroup * D + kMaxGroup + r] = Lsum;
        }
    }
    // ---- merge the CTAs of the cluster in its first CTA ----
    DSTAMP(5);
    if (CS > 1) cluster.sync(); else __syncthreads();
    DSTAMP(6);
    if (rank != 0) return;
    for (int i = tid; i < G * (D / 2); i += kThreads) {
        const int r = i / (D / 2), dp = i - r * (D / 2);
        float M = -INFINITY;
        for (int c = 0; c < CS; ++c) M = fmaxf(M, comb[c * (kMaxGroup * (D + 2)) + kMaxGroup * D + r]);
        float Lsum = 0.f, o0 = 0.f, o1 = 0.f;
        if (M > -INFINITY) {
            for (int c = 0; c < CS; ++c) {
                const float* pc = comb + c * (kMaxGroup * (D + 2));
                const float lc = pc[kMaxGroup * D + kMaxGroup + r];
                if (lc > 0.f) {
                    const float wgt = ex2f(pc[kMaxGroup * D + r] - M);
                    const float2 ov = *(reinterpret_cast<const float2*>(pc + r * D) + dp);
                    Lsum += lc * wgt;
                    o0 += ov.x * wgt;
                    o1 += ov.y * wgt;
                }
            }
        }
        const int64_t row = ((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + r;
        const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
        *(reinterpret_cast<float2*>(a.out + row * D) + dp) = make_float2(o0 * inv, o1 * inv);
        if (a.lse && dp == 0) a.lse[row] = Lsum > 0.f ? (M + log2f(Lsum)) * 0.69314718055994530942f : -INFINITY;
    }
    DSTAMP(7);
}

int pick_cluster(const KvView& kv, int n_keys_max)
{
    // enough CTAs to cover the SMs, at most about one tile of work each
    const long probs = (long)kv.n_layers * kv.batch * kv.n_kv_heads;
    const int tiles = n_keys_max > 0 ? (n_keys_max + kTK - 1) / kTK : 1;
    int cs = 1;
    while (cs < kMaxCluster && probs * cs < sm_count() && cs < tiles) cs *= 2;
    return cs;
}

template <int D>
int launch_d(const DraftArgs& a, int cs, cudaStream_t stream)
{
    auto kern = draft_cluster_kernel<D>;
    const size_t smem = SmemLayout<D>::total;
    static bool configured = false;  // per template instance
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return SPEC_ERR_CUDA;
        // clusters of 16 are outside the portable range: opt in (a refusal just keeps them at 8)
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
            cudaGetLastError();
        configured = true;
    }
    for (; cs >= 1; cs /= 2) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(cs, a.kv.n_kv_heads, a.kv.n_layers * a.kv.batch);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = cs;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see the kernel's prologue
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        if (cudaLaunchKernelEx(&cfg, kern, a, static_cast<int*>(a.workspace)) == cudaSuccess) {
            count_launch(1);
            return SPEC_OK;
        }
        cudaGetLastError();
        if (cs <= 8) break;  // a portable size that still fails is a real error
    }
    return SPEC_ERR_CUDA;
}

}  // namespace

size_t draft_workspace(const KvView&, int) { return kStatusBytes; }

int draft_launch(const DraftArgs& a, cudaStream_t stream)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    if (G > kMaxGroup) return SPEC_ERR_UNSUPPORTED_SHAPE;
    if (a.workspace_bytes < kStatusBytes) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    const int cs = pick_cluster(a.kv, a.k_total + a.max_tail);
    if (a.kv.head_dim == 128) return launch_d<128>(a, cs, stream);
    if (a.kv.head_dim == 64) return launch_d<64>(a, cs, stream);
    return SPEC_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace spec
