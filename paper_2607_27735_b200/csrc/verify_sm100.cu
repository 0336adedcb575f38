// Verification attention + Eq. 3 statistic for sm_100a: one persistent, warp-specialised kernel
// built on TMA (cp.async.bulk.tensor, no multicast), tcgen05.mma with TMEM accumulators and
// mbarrier pipelines.
//
// Why two sweeps.  Eq. 3 sums softmax PROBABILITIES over the window rows, so a key's
// contribution exp(s - LSE_row) needs every row's global normaliser; rows have different
// normalisers, so a per-key partial sum cannot be fixed up afterwards.  Per "unit" (a group of
// KV heads of one (layer, sequence)) the kernel therefore runs
//   P1: stream K, S^T = K Q^T on the tensor cores, per-row running (max, sum) -> row LSE;
//   P2: stream K again (now an L2 hit: the unit is sized to stay L2-resident) and V,
//       P = exp2(S - LSE) exactly normalised, column sums -> stats, O^T += V^T P^T on the
//       tensor cores with P split into bf16 hi + lo parts (keeps the 2e-3 bar when one key
//       takes most of the mass).
// Units are software-pipelined: every CTA works through  P1(u), P2(u-1)  per round, so the
// wait for the other CTAs' P1 partials of unit u-1 is covered by a whole stage of work, and
// HBM sees K once and V once.
//
// Layout of a tile in TMEM: keys on the 128 lanes, the R = n_q * group query rows on the
// columns (S^T), so one thread owns one key: the statistic is a thread-local sum, and the
// row max/sum of P1 is thread-local state reduced once per segment.
//
// Roles (384 threads): warp 0 TMA producer, warp 1 tcgen05.mma issuer (+ TMEM alloc), warps
// 2..9 two softmax warpgroups that split the columns, warps 10..11 combine the P1 partials
// into the LSE and reduce the per-CTA O partials (fixed order: deterministic).
//
// All CTAs must be co-resident (they wait on each other's partials): the grid never exceeds
// the SM count at one CTA per SM and the launch is cooperative.  Every wait is bounded; on
// expiry the kernel records SPEC_ERR_TIMEOUT in the status word and drains.
#include <cuda.h>

#include "verify_sm100.cuh"

namespace spec {

namespace {

constexpr int kTile = 128;            // keys per tile = UMMA M
constexpr int kD = 128;               // head_dim of the fast path
constexpr int kSlotBytes = 32768;     // one K or V tile: 2 halves x 128 rows x 128 B (SW128)
constexpr int kThreads = 384;
constexpr int kRing = 4;              // partial buffers are recycled every kRing units
constexpr long long kTimeoutCycles = 2000ll * 1000ll * 1000ll;  // about a second of SM clocks
constexpr uint64_t kEvictFirst = 0x12F0000000000000ull;
constexpr uint64_t kEvictLast = 0x14F0000000000000ull;
constexpr int kTmemCols = 512;
constexpr int kColS0 = 0, kColS1 = 128, kColO = 256;

struct FastParams {
    VerifyArgs a;
    int HG, NHG, cph, n_units, N, R, G;
    int n_slots, p_bufs;
    int box_rows, boxes;              // TMA boxes per 64-wide half of a tile
    float scale_log2;
    int* counters;                    // [2][n_units * HG]: P1 partials done, O partials done
    float2* ml_part;                  // [kRing][HG][cph][R]
    float* o_part;                    // [kRing][HG][cph][R][kD]
    int* status;
    int n_pages;
    long long* trace;
};

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
// MN-major operand without swizzle (the P^T tile): 8x8 core matrices of 128 contiguous bytes,
// K groups 128 B apart (leading offset), 8-row MN blocks 2048 B apart (stride offset).
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

#ifdef SPEC_TRACE
// Development aid (not compiled by default): per-CTA, per-role clock64 stamps in the workspace.
#define TRACE(role, slot) do { if (p.trace && (threadIdx.x & 31) == 0 && trace_n[role] < 60) \
    p.trace[((int64_t)blockIdx.x * 4 + (role)) * 64 + trace_n[role]++] = ((long long)(slot) << 48) | (clock64() & 0xffffffffffffll); } while (0)
#else
#define TRACE(role, slot) do { } while (0)
#endif

struct Ctl {
    volatile int* abort_flag;  // shared
    int* status;               // global status word (+ diagnostics in the following ints)
};

__device__ __noinline__ void report_timeout(const Ctl& c, int where)
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
            if (clock64() - t0 > kTimeoutCycles) {
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
            if (clock64() - t0 > kTimeoutCycles) {
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
    s.layer = unit / per_layer;
    const int rem = unit - s.layer * per_layer;
    s.b = rem / p.NHG;
    s.h = (rem - s.b * p.NHG) * p.HG + head_local;
    s.T = p.a.ctx_len[s.b];
    const int nb = (s.T + kTile - 1) / kTile;
    s.t0 = (int)((int64_t)rank * nb / p.cph);
    s.t1 = (int)((int64_t)(rank + 1) * nb / p.cph);
    s.prob = ((int64_t)s.layer * p.a.kv.batch + s.b) * p.a.kv.n_kv_heads + s.h;
    return s;
}

struct Smem {
    // dynamic shared memory carve-up (all offsets from a 1024-byte aligned base)
    uint32_t slots, q, p, bars, lse, stat_tmp, red, misc;
};

struct Bars {  // mbarrier addresses (shared space)
    uint32_t slot_full, slot_empty, q_full, q_empty, s_full, s_empty, p_full, p_empty, o_full, o_empty,
        lse_full, lse_empty, sm_sync, aux_sync, stat_full;
};

// ---------------------------------------------------------------------------------------------
// softmax warpgroups

template <int NH>
__device__ __forceinline__ void load_cols(uint32_t taddr, uint32_t* v)
{
#pragma unroll
    for (int c = 0; c < NH; c += 8) tmem_ld8(taddr + c, v + c);
    tc_wait_ld();
}

template <int NH>
__global__ void __launch_bounds__(kThreads, 1)
verify_sm100_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const __grid_constant__ CUtensorMap tm_q, const FastParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));  // generic pointer to the aligned base

    const int N = p.N, R = p.R, G = p.G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head_local = blockIdx.x / p.cph, rank = blockIdx.x % p.cph;
    const int q_bytes = N * 256;      // one Q buffer: 2 halves x N rows x 128 B
    const int p_bytes = N * 256;      // one P part (hi or lo): 2 key halves x N rows x 128 B

    const uint32_t s_slots = sbase;
    const uint32_t s_q = s_slots + p.n_slots * kSlotBytes;
    const uint32_t s_p = s_q + 2 * q_bytes;
    const uint32_t s_misc = s_p + p.p_bufs * 2 * p_bytes;
    uint8_t* misc = sgen + (s_misc - sbase);
    // misc: barriers (8 B each), then small arrays
    uint64_t* bar_mem = reinterpret_cast<uint64_t*>(misc);
    Bars B;
    {
        uint32_t o = s_misc;
        B.slot_full = o; o += 8 * 8;
        B.slot_empty = o; o += 8 * 8;
        B.q_full = o; o += 16;
        B.q_empty = o; o += 16;
        B.s_full = o; o += 16;
        B.s_empty = o; o += 16;
        B.p_full = o; o += 16;
        B.p_empty = o; o += 16;
        B.o_full = o; o += 8;
        B.o_empty = o; o += 8;
        B.lse_full = o; o += 16;
        B.lse_empty = o; o += 16;
        B.sm_sync = o; o += 8;
        B.aux_sync = o; o += 8;
        B.stat_full = o; o += 32;
    }
    (void)bar_mem;
    float* lse_s = reinterpret_cast<float*>(misc + 512);                 // [2][128]
    float* stat_tmp = reinterpret_cast<float*>(misc + 512 + 1024);       // [4][128]
    float2* red = reinterpret_cast<float2*>(misc + 512 + 3072);          // [8 warps][64] (m, l)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 512 + 3072 + 8 * 64 * 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    Ctl ctl{abort_flag, p.status};
#ifdef SPEC_TRACE
    int trace_n[4] = {0, 0, 0, 0};
#endif

    if (threadIdx.x == 0) {
        for (int i = 0; i < p.n_slots; ++i) {
            mbar_init(B.slot_full + 8 * i, 1);
            mbar_init(B.slot_empty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(B.q_full + 8 * i, 1);
            mbar_init(B.q_empty + 8 * i, 1);
            mbar_init(B.s_full + 8 * i, 1);
            mbar_init(B.s_empty + 8 * i, 8);
            mbar_init(B.p_full + 8 * i, 8);
            mbar_init(B.p_empty + 8 * i, 1);
            mbar_init(B.lse_full + 8 * i, 1);
            mbar_init(B.lse_empty + 8 * i, 8);
        }
        mbar_init(B.o_full, 1);
        mbar_init(B.o_empty, 8);
        mbar_init(B.sm_sync, 8);
        mbar_init(B.aux_sync, 2);
        for (int i = 0; i < 4; ++i) mbar_init(B.stat_full + 8 * i, 4);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // zero the Q buffers once: rows R..N-1 are padding the TMA never writes
    for (int i = threadIdx.x; i < 2 * q_bytes / 16; i += kThreads)
        *reinterpret_cast<uint4*>(sgen + (s_q - sbase) + 16 * i) = make_uint4(0, 0, 0, 0);
    fence_proxy_async();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int U = p.n_units;

    if (warp == 0) {
        // =========================== TMA producer ===========================
        uint32_t slot_idx = 0, qn = 0;
        const int boxes = p.boxes, box_rows = p.box_rows;
        const uint32_t box_bytes = box_rows * 128;
        bool ok = true;
        auto load_tile = [&](const CUtensorMap* map, const Seg& sg, int tile, uint64_t hint) -> bool {
            const uint32_t s = slot_idx % p.n_slots, ph = (slot_idx / p.n_slots) & 1;
            ++slot_idx;
            if (!mbar_wait(B.slot_empty + 8 * s, ph ^ 1, ctl, 1)) return false;
            // boxes of this tile that hold at least one key < T (pages past the context may not exist)
            const int key0 = tile * kTile;
            const int n_box = min(boxes, (sg.T - key0 + box_rows - 1) / box_rows);
            if (lane == 0) mbar_expect_tx(B.slot_full + 8 * s, 2u * n_box * box_bytes);
            __syncwarp();
            for (int i = lane; i < 2 * n_box; i += 32) {
                const int half = i / n_box, bx = i - half * n_box;
                const int pos = key0 + bx * box_rows;
                const int page = pos / p.a.kv.page_size, slot_in_page = pos - page * p.a.kv.page_size;
                int phys = p.a.kv.page_table ? __ldg(p.a.kv.page_table + (int64_t)sg.b * p.a.kv.max_pages + page)
                                             : sg.b * p.a.kv.max_pages + page;
                if (phys < 0 || phys >= p.n_pages) {
                    set_status(p.status, SPEC_ERR_BAD_INDEX);
                    phys = 0;
                }
                const uint32_t dst = s_slots + s * kSlotBytes + half * 16384 + bx * box_bytes;
                tma_load_5d(dst, map, B.slot_full + 8 * s, half * 64, slot_in_page, sg.h, phys, sg.layer, hint);
            }
            __syncwarp();
            return true;
        };
        for (int round = 0; round <= U && ok; ++round) {
            TRACE(0, 1);
            if (round < U) {
                const Seg sg = get_seg(p, round, head_local, rank);
                if (sg.t1 > sg.t0) {
                    const uint32_t qb = qn & 1, qph = (qn >> 1) & 1;
                    ++qn;
                    ok = mbar_wait(B.q_empty + 8 * qb, qph ^ 1, ctl, 2);
                    if (!ok) break;
                    if (lane == 0) {
                        mbar_expect_tx(B.q_full + 8 * qb, 2u * R * 128);
                        const int row0 = (sg.layer * p.a.kv.batch + sg.b) * p.a.n_q;
                        tma_load_3d(s_q + qb * q_bytes, &tm_q, B.q_full + 8 * qb, 0, sg.h * G, row0);
                        tma_load_3d(s_q + qb * q_bytes + N * 128, &tm_q, B.q_full + 8 * qb, 64, sg.h * G, row0);
                    }
                    __syncwarp();
                    for (int t = sg.t0; t < sg.t1 && ok; ++t) ok = load_tile(&tm_k, sg, t, kEvictLast);
                }
            }
            TRACE(0, 2);
            if (round >= 1 && ok) {
                const Seg sg = get_seg(p, round - 1, head_local, rank);
                for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                    ok = load_tile(&tm_k, sg, t, kEvictFirst);
                    if (ok) ok = load_tile(&tm_v, sg, t, kEvictFirst);
                }
            }
        }
        if (!ok) {  // let copies in flight land before the CTA's shared memory is released
            const uint64_t t0 = globaltimer();
            while (globaltimer() - t0 < 200000ull) __nanosleep(1000);
        }
    } else if (warp == 1) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            const uint32_t idesc_qk = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | ((128u >> 4) << 24);
            const uint32_t idesc_pv = idesc_qk | (1u << 15) | (1u << 16);  // A = V^T and B = P^T, both MN-major
            uint32_t slot_idx = 0, qn = 0, qk_idx = 0, pv_idx = 0, o_phase = 0;
            bool ok = true;
            // pending PV (issued one task late so the next QK^T overlaps the softmax)
            bool pend = false, pend_first = false, pend_last = false;
            uint32_t pend_slot = 0, pend_slot_ph = 0;
            auto issue_pv = [&]() -> bool {
                const uint32_t pb = pv_idx % p.p_bufs, pph = (pv_idx / p.p_bufs) & 1;
                ++pv_idx;
                if (!mbar_wait(B.slot_full + 8 * pend_slot, pend_slot_ph, ctl, 10)) return false;
                if (!mbar_wait(B.p_full + 8 * pb, pph, ctl, 11)) return false;
                if (pend_first) {
                    if (!mbar_wait(B.o_empty, o_phase ^ 1, ctl, 12)) return false;
                }
                tc_fence_after();
                const uint32_t v_addr = s_slots + pend_slot * kSlotBytes;
                const uint32_t d_o = tmem_base + kColO;
#pragma unroll 1
                for (int part = 0; part < 2; ++part) {
                    const uint32_t p_addr = s_p + (pb * 2 + part) * p_bytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint64_t a = desc_mnmajor(v_addr + ks * 2048);
                        const uint64_t b = desc_mnmajor_nosw(p_addr + ks * 256);
                        tc_mma(d_o, a, b, idesc_pv, (pend_first && part == 0 && ks == 0) ? 0u : 1u);
                    }
                }
                tc_commit(B.slot_empty + 8 * pend_slot);
                tc_commit(B.p_empty + 8 * pb);
                if (pend_last) {
                    tc_commit(B.o_full);
                    o_phase ^= 1;
                }
                pend = false;
                return true;
            };
            auto issue_qk = [&](uint32_t qb) -> bool {
                const uint32_t s = slot_idx % p.n_slots, sph = (slot_idx / p.n_slots) & 1;
                ++slot_idx;
                const uint32_t sb = qk_idx & 1, sbph = (qk_idx >> 1) & 1;
                ++qk_idx;
                if (!mbar_wait(B.slot_full + 8 * s, sph, ctl, 13)) return false;
                if (!mbar_wait(B.s_empty + 8 * sb, sbph ^ 1, ctl, 14)) return false;
                tc_fence_after();
                const uint32_t k_addr = s_slots + s * kSlotBytes;
                const uint32_t q_addr = s_q + qb * q_bytes;
                const uint32_t d_s = tmem_base + (sb ? kColS1 : kColS0);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t a = desc_kmajor(k_addr + (ks >> 2) * 16384 + (ks & 3) * 32);
                    const uint64_t b = desc_kmajor(q_addr + (ks >> 2) * (N * 128) + (ks & 3) * 32);
                    tc_mma(d_s, a, b, idesc_qk, ks ? 1u : 0u);
                }
                tc_commit(B.s_full + 8 * sb);
                tc_commit(B.slot_empty + 8 * s);
                return true;
            };
            uint32_t prev_qb = 0;
            bool prev_nonempty = false;
            for (int round = 0; round <= U && ok; ++round) {
                uint32_t cur_qb = 0;
                bool cur_nonempty = false;
                if (round < U) {
                    const Seg sg = get_seg(p, round, head_local, rank);
                    if (sg.t1 > sg.t0) {
                        cur_nonempty = true;
                        cur_qb = qn & 1;
                        const uint32_t qph = (qn >> 1) & 1;
                        ++qn;
                        ok = mbar_wait(B.q_full + 8 * cur_qb, qph, ctl, 15);
                        for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                            ok = issue_qk(cur_qb);
                            if (ok && pend) ok = issue_pv();
                        }
                    }
                }
                if (round >= 1 && ok && prev_nonempty) {
                    const Seg sg = get_seg(p, round - 1, head_local, rank);
                    for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                        ok = issue_qk(prev_qb);
                        if (!ok) break;
                        if (t == sg.t1 - 1) tc_commit(B.q_empty + 8 * prev_qb);  // last use of this Q buffer
                        if (pend) ok = issue_pv();
                        if (!ok) break;
                        pend = true;
                        pend_first = (t == sg.t0);
                        pend_last = (t == sg.t1 - 1);
                        pend_slot = slot_idx % p.n_slots;
                        pend_slot_ph = (slot_idx / p.n_slots) & 1;
                        ++slot_idx;  // the V slot of this tile
                    }
                }
                prev_qb = cur_qb;
                prev_nonempty = cur_nonempty;
            }
            if (ok && pend) ok = issue_pv();
        }
        __syncwarp();
    } else if (warp < 10) {
        // =========================== softmax warpgroups ===========================
        const int sw = warp - 2;                 // 0..7
        const int wg = sw >> 2;                  // column half
        const int quarter = warp & 3;            // TMEM lane quarter this warp may touch
        const int key_l = quarter * 32 + lane;   // key within the tile (P1/P2) or d (epilogue)
        const int c0 = wg * NH;                  // first column of this warpgroup
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int stat_r0 = p.a.first_stat_row * G;
        const float cs = p.scale_log2;
        constexpr float kNegBig = -1.0e30f;      // finite stand-in for -inf: keeps ex2 arguments NaN-free
        uint32_t qk_idx = 0, pv_idx = 0, slot_idx = 0, lse_n = 0, o_phase = 0, sync_n = 0, stat_n = 0;
        bool ok = true;
        int prev_lse_idx = 0;
        bool prev_nonempty = false;
        for (int round = 0; round <= U && ok; ++round) {
            bool cur_nonempty = false;
            if (warp == 2) TRACE(2, 1);
            if (round < U) {
                // ------------------------------ P1 ------------------------------
                const Seg sg = get_seg(p, round, head_local, rank);
                float m[NH], l[NH];
#pragma unroll
                for (int i = 0; i < NH; ++i) {
                    m[i] = kNegBig;
                    l[i] = 0.f;
                }
                cur_nonempty = sg.t1 > sg.t0;
                for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                    const uint32_t sb = qk_idx & 1, sbph = (qk_idx >> 1) & 1;
                    ++qk_idx;
                    ++slot_idx;
                    ok = mbar_wait(B.s_full + 8 * sb, sbph, ctl, 20);
                    if (!ok) break;
                    tc_fence_after();
                    uint32_t v[NH];
                    load_cols<NH>(t_lane + (sb ? kColS1 : kColS0) + c0, v);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(B.s_empty + 8 * sb);
                    float sc[NH];
#pragma unroll
                    for (int i = 0; i < NH; ++i) sc[i] = __uint_as_float(v[i]) * cs;
                    if (t * kTile + kTile > sg.T - p.a.n_q + 1) {
                        // tile holds keys some window rows may not see (or keys beyond the context)
                        const int key = t * kTile + key_l;
                        int j = c0 / G, gg = c0 - j * G;
#pragma unroll
                        for (int i = 0; i < NH; ++i) {
                            if (key > sg.T - p.a.n_q + j) sc[i] = kNegBig;
                            if (++gg == G) {
                                gg = 0;
                                ++j;
                            }
                        }
                    }
                    // running max is refreshed only when some lane's score beats it by 2^8: one
                    // warp-uniform branch per tile, one ex2 per element otherwise
                    bool need = false;
#pragma unroll
                    for (int i = 0; i < NH; ++i) need |= sc[i] > m[i] + 8.f;
                    if (__any_sync(0xffffffffu, need)) {
#pragma unroll
                        for (int i = 0; i < NH; ++i) {
                            const float mn = fmaxf(m[i], sc[i]);
                            l[i] *= ex2(m[i] - mn);
                            m[i] = mn;
                        }
                    }
#pragma unroll
                    for (int i = 0; i < NH; ++i) l[i] += ex2(sc[i] - m[i]);
                }
                if (!ok) break;
                if (warp == 2) TRACE(2, 2);
                // reduce (m, l) over the 32 key lanes of this warp, then over the 4 warps via smem
#pragma unroll
                for (int i = 0; i < NH; ++i) {
                    float M = m[i];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
                    float L = l[i] * ex2(m[i] - M);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
                    if (lane == 0) red[sw * 64 + i] = make_float2(M, L);
                }
                ok = group_sync(B.sm_sync, sync_n, ctl, 26);
                if (!ok) break;
                {
                    const int tid = threadIdx.x - 64;  // 0..255
                    const int wgi = tid >> 7, ci = tid & 127;
                    if (ci < NH && wgi * NH + ci < R) {
                        float M = kNegBig;
#pragma unroll
                        for (int w = 0; w < 4; ++w) M = fmaxf(M, red[(wgi * 4 + w) * 64 + ci].x);
                        float L = 0.f;
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            const float2 ml = red[(wgi * 4 + w) * 64 + ci];
                            L += ml.y * ex2(ml.x - M);
                        }
                        const int64_t base = (((int64_t)(round % kRing) * p.HG + head_local) * p.cph + rank) * R;
                        p.ml_part[base + wgi * NH + ci] = make_float2(M, cur_nonempty ? L : 0.f);
                    }
                }
                ok = group_sync(B.sm_sync, sync_n, ctl, 27);
                if (!ok) break;
                if (threadIdx.x == 64) {
                    __threadfence();
                    atomicAdd(p.counters + round * p.HG + head_local, 1);
                }
            }
            if (warp == 2) TRACE(2, 3);
            if (round >= 1 && ok) {
                // ------------------------------ P2 ------------------------------
                const Seg sg = get_seg(p, round - 1, head_local, rank);
                const int64_t obase = (((int64_t)((round - 1) % kRing) * p.HG + head_local) * p.cph + rank) * R * kD;
                if (prev_nonempty) {
                    const uint32_t lb = prev_lse_idx & 1, lph = (prev_lse_idx >> 1) & 1;
                    ok = mbar_wait(B.lse_full + 8 * lb, lph, ctl, 21);
                    if (!ok) break;
                    const float4* lse4 = reinterpret_cast<const float4*>(lse_s + lb * 128 + c0);
                    if (warp == 2) TRACE(2, 4);
                    for (int t = sg.t0; t < sg.t1 && ok; ++t) {
                        const uint32_t sb = qk_idx & 1, sbph = (qk_idx >> 1) & 1;
                        ++qk_idx;
                        ++slot_idx;                       // K slot
                        const uint32_t vs = slot_idx % p.n_slots, vsph = (slot_idx / p.n_slots) & 1;
                        ++slot_idx;                       // V slot
                        const uint32_t pb = pv_idx % p.p_bufs, pph = (pv_idx / p.p_bufs) & 1;
                        ++pv_idx;
                        ok = mbar_wait(B.s_full + 8 * sb, sbph, ctl, 22);
                        if (!ok) break;
                        tc_fence_after();
                        uint32_t v[NH];
                        load_cols<NH>(t_lane + (sb ? kColS1 : kColS0) + c0, v);
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(B.s_empty + 8 * sb);
                        const int key = t * kTile + key_l;
                        float pr[NH];
#pragma unroll
                        for (int i = 0; i < NH; i += 4) {
                            const float4 ls = lse4[i >> 2];
                            pr[i + 0] = ex2(fmaf(__uint_as_float(v[i + 0]), cs, -ls.x));
                            pr[i + 1] = ex2(fmaf(__uint_as_float(v[i + 1]), cs, -ls.y));
                            pr[i + 2] = ex2(fmaf(__uint_as_float(v[i + 2]), cs, -ls.z));
                            pr[i + 3] = ex2(fmaf(__uint_as_float(v[i + 3]), cs, -ls.w));
                        }
                        if (t * kTile + kTile > sg.T - p.a.n_q + 1) {
                            int j = c0 / G, gg = c0 - j * G;
#pragma unroll
                            for (int i = 0; i < NH; ++i) {
                                if (key > sg.T - p.a.n_q + j) pr[i] = 0.f;  // select, so NaN-safe
                                if (++gg == G) {
                                    gg = 0;
                                    ++j;
                                }
                            }
                        }
                        float st = 0.f;
#pragma unroll
                        for (int i = 0; i < NH; ++i) st += (c0 + i >= stat_r0) ? pr[i] : 0.f;
                        ok = mbar_wait(B.p_empty + 8 * pb, pph ^ 1, ctl, 23);
                        if (!ok) break;
                        // P^T as the B operand, rows contiguous (8 rows = one 16-byte vector per key):
                        // vector (row block nb, key k) at nb*2048 + (k/8)*128 + (k%8)*16
                        uint8_t* p_hi = sgen + (s_p - sbase) + (pb * 2 + 0) * p_bytes + (wg * (NH / 8)) * 2048 +
                                        (key_l >> 3) * 128 + (key_l & 7) * 16;
                        uint8_t* p_lo = p_hi + p_bytes;
#pragma unroll
                        for (int nb = 0; nb < NH / 8; ++nb) {
                            uint32_t hi[4], lo[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float a = pr[nb * 8 + 2 * q], b = pr[nb * 8 + 2 * q + 1];
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(hi[q]) : "f"(b), "f"(a));
                                const float ra = a - __uint_as_float(hi[q] << 16);
                                const float rb = b - __uint_as_float(hi[q] & 0xffff0000u);
                                asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(lo[q]) : "f"(rb), "f"(ra));
                            }
                            *reinterpret_cast<uint4*>(p_hi + nb * 2048) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                            *reinterpret_cast<uint4*>(p_lo + nb * 2048) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                        }
                        if (t * kTile + kTile > sg.T) {
                            // ragged last tile: V rows at or beyond T may hold anything; zero them
                            // in shared memory so that 0 * garbage never reaches the accumulator
                            ok = mbar_wait(B.slot_full + 8 * vs, vsph, ctl, 24);
                            if (!ok) break;
                            if (key >= sg.T) {
                                uint8_t* vrow = sgen + (s_slots - sbase) + vs * kSlotBytes + wg * 16384 + key_l * 128;
#pragma unroll
                                for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(vrow + 16 * c) = make_uint4(0, 0, 0, 0);
                            }
                        }
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(B.p_full + 8 * pb);
                        // column-split statistic: warpgroup 1 hands its partial sum to warpgroup 0
                        // (4 buffers / barriers: warpgroup 1 can run at most two tiles ahead)
                        const uint32_t sq = stat_n & 3, sqph = (stat_n >> 2) & 1;
                        ++stat_n;
                        if (wg == 1) {
                            stat_tmp[sq * 128 + key_l] = st;
                            __syncwarp();
                            if (lane == 0) mbar_arrive(B.stat_full + 8 * sq);
                        } else {
                            ok = mbar_wait(B.stat_full + 8 * sq, sqph, ctl, 28);
                            if (!ok) break;
                            if (key < sg.T) p.a.stats[sg.prob * p.a.stat_stride + key] = st + stat_tmp[sq * 128 + key_l];
                        }
                    }
                    if (!ok) break;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(B.lse_empty + 8 * lb);
                    if (warp == 2) TRACE(2, 5);
                    // ---- epilogue: O^T (d on lanes, rows on columns) -> partial [r][d] ----
                    ok = mbar_wait(B.o_full, o_phase, ctl, 25);
                    if (!ok) break;
                    o_phase ^= 1;
                    tc_fence_after();
                    uint32_t v[NH];
                    load_cols<NH>(t_lane + kColO + c0, v);
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(B.o_empty);
#pragma unroll
                    for (int i = 0; i < NH; ++i) {
                        const int r = c0 + i;
                        if (r < R) p.o_part[obase + (int64_t)r * kD + key_l] = __uint_as_float(v[i]);
                    }
                } else {
                    // empty segment: contribute zeros
                    for (int i = threadIdx.x - 64; i < R * kD; i += 256) p.o_part[obase + i] = 0.f;
                }
                ok = group_sync(B.sm_sync, sync_n, ctl, 29);
                if (!ok) break;
                if (threadIdx.x == 64) {
                    __threadfence();
                    atomicAdd(p.counters + U * p.HG + (round - 1) * p.HG + head_local, 1);
                }
            }
            if (cur_nonempty) prev_lse_idx = lse_n++;
            prev_nonempty = cur_nonempty;
            if (warp == 2) TRACE(2, 6);
        }
    } else {
        // =========================== aux warps: LSE combine, O reduction ===========================
        const int tid = threadIdx.x - 320;  // 0..63
        uint32_t lse_n = 0, sync_n = 0;
        bool ok = true;
        auto reduce_unit = [&](int unit) -> bool {
            if (!counter_wait(p.counters + U * p.HG + unit * p.HG + head_local, p.cph, ctl, 30)) return false;
            __threadfence();
            const Seg sg = get_seg(p, unit, head_local, rank);
            const int E4 = R * kD / 4;
            const int lo = (int)((int64_t)rank * E4 / p.cph), hi = (int)((int64_t)(rank + 1) * E4 / p.cph);
            const float4* src = reinterpret_cast<const float4*>(
                p.o_part + ((int64_t)(unit % kRing) * p.HG + head_local) * p.cph * R * kD);
            for (int e = lo + tid; e < hi; e += 64) {
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int k0 = 0; k0 < p.cph; k0 += 8) {  // batches of 8 independent loads
                    float4 x[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        x[u] = (k0 + u < p.cph) ? __ldcg(src + (int64_t)(k0 + u) * E4 + e)
                                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        acc.x += x[u].x;
                        acc.y += x[u].y;
                        acc.z += x[u].z;
                        acc.w += x[u].w;
                    }
                }
                const int r = e / (kD / 4), d4 = e - r * (kD / 4);
                const int j = r / G, g = r - j * G;
                const int64_t row = (((int64_t)sg.layer * p.a.kv.batch + sg.b) * p.a.n_q + j) * p.a.kv.n_q_heads + sg.h * G + g;
                reinterpret_cast<float4*>(p.a.out + row * kD)[d4] = acc;
            }
            return true;
        };
        for (int round = 1; round <= U + 1 && ok; ++round) {
            if (round <= U) {
                // LSE of unit round-1, needed by the P2 stage of this round
                const int unit = round - 1;
                const Seg sg = get_seg(p, unit, head_local, rank);
                if (sg.t1 > sg.t0) {
                    const uint32_t lb = lse_n & 1, lph = (lse_n >> 1) & 1;
                    ++lse_n;
                    if (warp == 10) TRACE(3, 1);
                    ok = counter_wait(p.counters + unit * p.HG + head_local, p.cph, ctl, 31);
                    if (!ok) break;
                    if (warp == 10) TRACE(3, 2);
                    __threadfence();
                    ok = mbar_wait(B.lse_empty + 8 * lb, lph ^ 1, ctl, 32);
                    if (!ok) break;
                    const float2* src = p.ml_part + ((int64_t)(unit % kRing) * p.HG + head_local) * p.cph * R;
                    for (int r = R + tid; r < N; r += 64) lse_s[lb * 128 + r] = 1.0e30f;  // padded rows: P = 0
                    for (int r = tid; r < R; r += 64) {
                        float M = -INFINITY, L = 0.f;
                        for (int k0 = 0; k0 < p.cph; k0 += 8) {  // batches of 8 independent loads
                            float2 x[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                x[u] = (k0 + u < p.cph) ? __ldcg(src + (int64_t)(k0 + u) * R + r)
                                                        : make_float2(0.f, 0.f);
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                if (x[u].y > 0.f) {
                                    const float Mn = fmaxf(M, x[u].x);
                                    L = L * exp2f(M - Mn) + x[u].y * exp2f(x[u].x - Mn);
                                    M = Mn;
                                }
                            }
                        }
                        const float lse2 = M + log2f(L);
                        lse_s[lb * 128 + r] = lse2;
                        if (rank == p.cph - 1 && p.a.lse) {  // the last rank always owns at least one tile
                            const int j = r / G, g = r - j * G;
                            const int64_t row = (((int64_t)sg.layer * p.a.kv.batch + sg.b) * p.a.n_q + j) * p.a.kv.n_q_heads + sg.h * G + g;
                            p.a.lse[row] = lse2 * 0.69314718055994530942f;
                        }
                    }
                    ok = group_sync(B.aux_sync, sync_n, ctl, 33);
                    if (!ok) break;
                    if (tid == 0) mbar_arrive(B.lse_full + 8 * lb);
                    if (warp == 10) TRACE(3, 3);
                }
            }
            if (round >= 2) ok = reduce_unit(round - 2);
            if (warp == 10) TRACE(3, 4);
        }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------------
// host side

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
    int HG, cph, n_units, N, n_slots, p_bufs, box_rows, boxes;
    size_t smem_bytes;
    size_t ctr_off, ml_off, o_off, total, trace_off;
};

int box_rows_for(int page_size)
{
    if (page_size >= kTile) return (page_size % kTile == 0) ? kTile : 0;
    if (page_size >= 8 && kTile % page_size == 0) return page_size;
    return 0;
}

bool make_plan(const KvView& kv, int n_q, int max_ctx_len, Plan* pl)
{
    const int G = kv.n_q_heads / kv.n_kv_heads, R = n_q * G;
    if (kv.head_dim != kD || R > 128 || G > 256 || n_q > 256) return false;
    const int box_rows = box_rows_for(kv.page_size);
    if (box_rows == 0) return false;
    const int nsm = sm_count();
    const int N = (R + 15) / 16 * 16;
    const int nb = (max_ctx_len + kTile - 1) / kTile;
    const long lb = (long)kv.n_layers * kv.batch;
    int best_hg = 0;
    double best_score = -1.0;
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
        if (score > best_score) {
            best_score = score;
            best_hg = hg;
        }
    }
    if (best_hg == 0) return false;
    pl->HG = best_hg;
    pl->cph = nsm / best_hg;
    pl->n_units = (int)(lb * (kv.n_kv_heads / best_hg));
    pl->N = N;
    pl->box_rows = box_rows;
    pl->boxes = kTile / box_rows;
    pl->p_bufs = N <= 64 ? 2 : 1;
    const size_t fixed = 1024 /*alignment slack*/ + 2 * (size_t)N * 256 + (size_t)pl->p_bufs * 2 * N * 256 + 8192;
    const size_t cap = 227 * 1024;
    int slots = (int)((cap - fixed) / kSlotBytes);
    if (slots > 8) slots = 8;
    if (slots < 3) return false;
    pl->n_slots = slots;
    pl->smem_bytes = fixed + (size_t)slots * kSlotBytes;
    size_t off = kStatusBytes;
    pl->ctr_off = off;
    off += (size_t)2 * pl->n_units * pl->HG * sizeof(int);
    off = (off + 255) & ~(size_t)255;
    pl->ml_off = off;
    off += (size_t)kRing * pl->HG * pl->cph * R * sizeof(float2);
    off = (off + 255) & ~(size_t)255;
    pl->o_off = off;
    off += (size_t)kRing * pl->HG * pl->cph * R * kD * sizeof(float);
    pl->total = (off + 255) & ~(size_t)255;
#ifdef SPEC_TRACE
    pl->trace_off = pl->total;
    pl->total += (size_t)nsm * 4 * 64 * sizeof(long long);
#endif
    return true;
}

bool encode_kv_map(CUtensorMap* map, const void* base, const KvView& kv, int n_pages, int box_rows)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[5] = {(cuuint64_t)kD, (cuuint64_t)kv.page_size, (cuuint64_t)kv.n_kv_heads,
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

bool encode_q_map(CUtensorMap* map, const void* q, const KvView& kv, int n_q, int G)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)kv.n_q_heads,
                                (cuuint64_t)kv.n_layers * kv.batch * n_q};
    const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)kv.n_q_heads * kD * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)n_q};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NH>
int launch_nh(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const FastParams& fp,
              const Plan& pl, cudaStream_t stream)
{
    auto kern = verify_sm100_kernel<NH>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem_bytes) != cudaSuccess)
        return SPEC_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pl.cph * pl.HG);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = pl.smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, kern, tk, tv, tq, fp) != cudaSuccess) {
        cudaGetLastError();
        return SPEC_ERR_CUDA;
    }
    count_launch(1);
    return SPEC_OK;
}

}  // namespace

bool verify_sm100_supported(const KvView& kv, int n_q)
{
    Plan pl;
    if (!make_plan(kv, n_q, kTile, &pl)) return false;
    // TMA: 16-byte aligned base and strides (strides are multiples of 8 elements by contract)
    if (kv.slot_stride < kD) return false;
    return true;
}

size_t verify_sm100_workspace(const KvView& kv, int n_q, int max_ctx_len)
{
    Plan pl;
    if (!make_plan(kv, n_q, max_ctx_len, &pl)) return 0;
    return pl.total;
}

int verify_sm100_launch(const VerifyArgs& a, cudaStream_t stream)
{
    Plan pl;
    if (!make_plan(a.kv, a.n_q, a.max_ctx_len, &pl)) return SPEC_ERR_UNSUPPORTED_SHAPE;
    if (a.workspace_bytes < pl.total) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const int n_pages = a.kv.n_pages;
    CUtensorMap tk, tv, tq;
    if (!encode_kv_map(&tk, a.kv.k, a.kv, n_pages, pl.box_rows) ||
        !encode_kv_map(&tv, a.kv.v, a.kv, n_pages, pl.box_rows) || !encode_q_map(&tq, a.q, a.kv, a.n_q, G))
        return SPEC_ERR_CUDA;
    char* ws = static_cast<char*>(a.workspace);
    FastParams fp;
    fp.a = a;
    fp.HG = pl.HG;
    fp.NHG = a.kv.n_kv_heads / pl.HG;
    fp.cph = pl.cph;
    fp.n_units = pl.n_units;
    fp.N = pl.N;
    fp.R = a.n_q * G;
    fp.G = G;
    fp.n_slots = pl.n_slots;
    fp.p_bufs = pl.p_bufs;
    fp.box_rows = pl.box_rows;
    fp.boxes = pl.boxes;
    fp.scale_log2 = a.kv.scale * 1.4426950408889634f;
    fp.counters = reinterpret_cast<int*>(ws + pl.ctr_off);
    fp.ml_part = reinterpret_cast<float2*>(ws + pl.ml_off);
    fp.o_part = reinterpret_cast<float*>(ws + pl.o_off);
    fp.status = reinterpret_cast<int*>(ws);
    fp.n_pages = n_pages;
    fp.trace = nullptr;
#ifdef SPEC_TRACE
    fp.trace = reinterpret_cast<long long*>(ws + pl.trace_off);
#endif
    if (cudaMemsetAsync(ws + pl.ctr_off, 0, (size_t)2 * pl.n_units * pl.HG * sizeof(int), stream) != cudaSuccess)
        return SPEC_ERR_CUDA;
    switch (pl.N / 2) {
        case 8: return launch_nh<8>(tk, tv, tq, fp, pl, stream);
        case 16: return launch_nh<16>(tk, tv, tq, fp, pl, stream);
        case 24: return launch_nh<24>(tk, tv, tq, fp, pl, stream);
        case 32: return launch_nh<32>(tk, tv, tq, fp, pl, stream);
        case 40: return launch_nh<40>(tk, tv, tq, fp, pl, stream);
        case 48: return launch_nh<48>(tk, tv, tq, fp, pl, stream);
        case 56: return launch_nh<56>(tk, tv, tq, fp, pl, stream);
        case 64: return launch_nh<64>(tk, tv, tq, fp, pl, stream);
        default: return SPEC_ERR_UNSUPPORTED_SHAPE;
    }
}

}  // namespace spec
