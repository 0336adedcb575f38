// Shared device-side pieces of the sm_100a verification kernels: PTX wrappers for mbarrier,
// TMA (cp.async.bulk.tensor, never multicast), tcgen05 (alloc / mma / commit / ld / fences),
// UMMA shared-memory descriptors, bounded waits, and the work decomposition.
#pragma once

#include <cuda.h>

#include "spec_common.cuh"

namespace spec {
namespace sm100 {

constexpr int kTile = 128;            // keys per tile = UMMA M
constexpr int kD = 128;               // head_dim the tiles are laid out for (head_dim 64 uses the lower half)
constexpr int kSlotBytes = 32768;     // one K or V tile: 2 halves x 128 rows x 128 B (SW128)
constexpr int kThreads = 384;
constexpr int kRing = 4;              // partial buffers are recycled every kRing units
constexpr uint64_t kEvictFirst = 0x12F0000000000000ull;
constexpr uint64_t kEvictLast = 0x14F0000000000000ull;
constexpr int kTmemCols = 512;
constexpr int kColS0 = 0, kColS1 = 128, kColO = 256;

struct FastParams {
    VerifyArgs a;
    int HG, NHG, cph, n_units, N, R, G;
    int n_slots, p_bufs;
    int n_raw;                        // 8-bit cache read directly: raw 16 KB stages in front of the operand slots (else 0)
    int D;                            // head_dim: 128, or 64 (score-cache kernel only)
    int box_rows, boxes;              // TMA boxes per 64-wide half of a tile
    float scale_log2;
    int* counters;                    // [2][n_units * HG]: P1 partials done, O partials done; then one
                                      // "CTAs finished" word.  All zero between calls.
    float2* ml_part;                  // [kRing][HG][cph][R]
    float* o_part;                    // [kRing][HG][cph][R][kD] (columns >= head_dim unused)
    int* status;
    int n_pages;
    int n_cache;                      // S tiles the TMEM cache holds (cached variant)
    int q_bufs;                       // Q buffers in shared memory (cached variant: 1)
    long long wait_limit;             // SM clocks after which a device-side wait gives up
    // divisions of get_seg() as multiply-high + shift (x / d = umulhi(x, mul) >> sh for 0 <= x < 2^31;
    // sh < 0 marks d == 1): by units per layer, by head groups per sequence, by CTAs per head, by the
    // group size G
    uint32_t div_mul[4];
    int32_t div_sh[4];
};

// Host side: magic numbers of an exact division by d >= 1 (see FastParams::div_mul).
inline void set_divisor(FastParams* p, int which, int d)
{
    if (d <= 1) {
        p->div_mul[which] = 0;
        p->div_sh[which] = -1;
        return;
    }
    int c = 0;
    while ((1ull << c) < (unsigned)d) ++c;
    p->div_mul[which] = (uint32_t)(((1ull << (31 + c)) + d - 1) / d);
    p->div_sh[which] = c - 1;
}
__device__ __forceinline__ int fast_div(const FastParams& p, int which, int x)
{
    return p.div_sh[which] < 0 ? x : (int)(__umulhi((uint32_t)x, p.div_mul[which]) >> p.div_sh[which]);
}

// ---------------------------------------------------------------------------------------------
// PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint64_t globaltimer()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
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
// Non-blocking probe (try_wait may suspend the thread for a while; a scheduler loop must not).
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* v)
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const uint32_t* v)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ int ld_acquire(const int* p)
{
    int v;
    asm volatile("ld.acquire.gpu.global.b32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1,
                                            int c2, int c3, int c4, uint64_t hint)
{
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%3, %4, %5, %6, %7}], [%2], %8;"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "l"(hint) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes"
        " [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}

// K-major operand, 128-byte swizzle: rows of 128 B, 8-row groups 1024 B apart.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// MN-major operand without swizzle: 8x8 core matrices of 128 contiguous bytes, K groups 128 B
// apart (leading offset), 8-row MN blocks 2048 B apart (stride offset).
__device__ __forceinline__ uint64_t desc_mnmajor_nosw(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (8ull << 16) | (128ull << 32) | (1ull << 46);
}
// MN-major operand, 128-byte swizzle: 64-element MN blocks 16 KiB apart (leading offset),
// 8-row K groups 1024 B apart (stride offset).
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFF) | (1024ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

// ---------------------------------------------------------------------------------------------


struct Ctl {
    volatile int* abort_flag;  // shared
    int* status;               // global status word (+ diagnostics in the following ints)
    long long limit;           // SM clocks a wait may take
};

static __device__ __noinline__ void report_timeout(const Ctl& c, int where)
{
    if (atomicCAS(c.status, 0, SPEC_ERR_TIMEOUT) == 0) {
        c.status[1] = where;
        c.status[2] = blockIdx.x;
        c.status[3] = threadIdx.x;
    }
    *c.abort_flag = 1;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const Ctl& c, int where)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 63u) == 0) {
            if (*c.abort_flag) return false;
            if (clock64() - t0 > c.limit) {
                report_timeout(c, where);
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ bool counter_wait(const int* ctr, int target, const Ctl& c, int where)
{
    if (ld_acquire(ctr) >= target) return true;
    const long long t0 = clock64();
    uint32_t spins = 0;
    while (ld_acquire(ctr) < target) {
        __nanosleep(32);
        if ((++spins & 63u) == 0) {
            if (*c.abort_flag) return false;
            if (clock64() - t0 > c.limit) {
                report_timeout(c, where);
                return false;
            }
        }
    }
    return true;
}

// Barrier among the warps of one role, built on an mbarrier so that the wait is bounded like
// every other wait (a hardware named barrier could not be abandoned after a timeout).
__device__ __forceinline__ bool group_sync(uint32_t bar, uint32_t& n, const Ctl& c, int where)
{
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bar);
    const bool ok = mbar_wait(bar, n & 1, c, where);
    ++n;
    return ok;
}

struct Seg {
    int layer, b, h, T, t0, t1;
    int64_t prob;
};

__device__ __forceinline__ Seg get_seg(const FastParams& p, int unit, int head_local, int rank)
{
    Seg s;
    const int per_layer = p.a.kv.batch * p.NHG;
    s.layer = fast_div(p, 0, unit);
    const int rem = unit - s.layer * per_layer;
    s.b = fast_div(p, 1, rem);
    s.h = (rem - s.b * p.NHG) * p.HG + head_local;
    // a length outside [n_q, max_ctx_len] is clamped (the launch, the score cache and the output rows
    // were sized for that range); the TMA producer warp reports it (check_len)
    s.T = min(max(p.a.ctx_len[s.b], p.a.n_q), p.a.max_ctx_len);
    const int nb = (s.T + kTile - 1) / kTile;
    s.t0 = fast_div(p, 2, rank * nb);        // rank < SMs, nb < 2^20: the products stay far below 2^31
    s.t1 = fast_div(p, 2, (rank + 1) * nb);
    s.prob = ((int64_t)s.layer * p.a.kv.batch + s.b) * p.a.kv.n_kv_heads + s.h;
    return s;
}

__device__ __forceinline__ void check_len(const FastParams& p, const Seg& s)
{
    if (p.a.ctx_len[s.b] != s.T) set_status(p.status, SPEC_ERR_BAD_INDEX);
}

// launchers of the two kernel variants (host)
int launch_twosweep(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const FastParams& fp,
                    int grid, size_t smem_bytes, cudaStream_t stream);
int launch_cached(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const FastParams& fp,
                  int grid, size_t smem_bytes, cudaStream_t stream);

// End of kernel: the last CTA to get here puts the cross-CTA counters back to zero, so the next
// call on this workspace needs no memset (a memset node between two kernels of a CUDA graph
// costs more than the whole prologue of this kernel).  Call after the CTA's last use of them.
__device__ __forceinline__ void reset_counters_if_last(const FastParams& p, int* smem_flag)
{
    const int n = 2 * p.n_units * p.HG;
    if (threadIdx.x == 0) {
        __threadfence();
        *smem_flag = atomicAdd(p.counters + n, 1) == (int)gridDim.x - 1;
    }
    __syncthreads();
    if (*smem_flag) {
        for (int i = threadIdx.x; i <= n; i += blockDim.x) p.counters[i] = 0;
    }
}

template <int NH>
__device__ __forceinline__ void load_cols(uint32_t taddr, uint32_t* v)
{
#pragma unroll
    for (int c = 0; c < NH; c += 8) tmem_ld8(taddr + c, v + c);
    tc_wait_ld();
}

}  // namespace sm100
}  // namespace spec
