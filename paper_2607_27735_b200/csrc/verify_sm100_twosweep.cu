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
#include "sm100_common.cuh"
#include "verify_sm100.cuh"

namespace spec {
namespace sm100 {

namespace {

// Walks the tile tasks of one CTA in execution order: for round r = 0..U, the P1 tiles of unit r
// (phase 0) then the P2 tiles of unit r-1 (phase 1).  Tracks the global task index (selects the
// score buffer), the ring position of the task's K tile, and which Q buffer the task uses.
struct Cursor {
    int round, phase, t, t0, t1;
    uint32_t idx, slot, qn, qb, qph, qb_p1;
    bool done;

    __device__ bool load_stage(const FastParams& p, int head_local, int rank)
    {
        const int unit = phase == 0 ? round : round - 1;
        if (unit < 0 || unit >= p.n_units) return false;
        const Seg sg = get_seg(p, unit, head_local, rank);
        if (sg.t1 <= sg.t0) return false;
        t0 = sg.t0;
        t1 = sg.t1;
        t = sg.t0;
        if (phase == 0) {  // a non-empty P1 stage claims the next Q buffer; its P2 stage reuses it
            qb = qn & 1;
            qph = (qn >> 1) & 1;
            ++qn;
            qb_p1 = qb;
        } else {
            qb = qb_prev;
        }
        return true;
    }
    uint32_t qb_prev;
    __device__ void seek(const FastParams& p, int head_local, int rank)
    {
        for (;;) {
            if (load_stage(p, head_local, rank)) return;
            if (phase == 0) {
                phase = 1;
            } else {
                phase = 0;
                qb_prev = qb_p1;
                ++round;
                if (round > p.n_units) {
                    done = true;
                    return;
                }
            }
        }
    }
    __device__ void start(const FastParams& p, int head_local, int rank)
    {
        round = 0; phase = 0; t = t0 = t1 = 0;
        idx = slot = qn = qb = qph = qb_p1 = qb_prev = 0;
        done = false;
        seek(p, head_local, rank);
    }
    __device__ void next(const FastParams& p, int head_local, int rank)
    {
        ++idx;
        slot += phase == 0 ? 1 : 2;
        if (++t < t1) return;
        if (phase == 0) {
            phase = 1;
        } else {
            phase = 0;
            qb_prev = qb_p1;
            ++round;
            if (round > p.n_units) {
                done = true;
                return;
            }
        }
        seek(p, head_local, rank);
    }
};
struct Bars {  // mbarrier addresses (shared space)
    uint32_t slot_full, slot_empty, q_full, q_empty, s_full, s_empty, p_full, p_empty, o_full, o_empty,
        lse_full, lse_empty, sm_sync, aux_sync, stat_full;
};

// ---------------------------------------------------------------------------------------------
template <int NH>
__global__ void __launch_bounds__(kThreads, 1)
verify_twosweep_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    const __grid_constant__ CUtensorMap tm_q, const FastParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));  // generic pointer to the aligned base

    const int N = p.N, R = p.R, G = p.G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head_local = blockIdx.x / p.cph, rank = blockIdx.x % p.cph;
    const int q_bytes = N * 256;      // one Q buffer: 2 halves x N rows x 128 B
    const int p_bytes = ((2 * N + 63) / 64) * 16384;  // one P buffer: [hi | lo] rows in 64-row blocks of 128 keys x 128 B

    const uint32_t s_slots = sbase;
    const uint32_t s_q = s_slots + p.n_slots * kSlotBytes;
    const uint32_t s_p = s_q + 2 * q_bytes;
    const uint32_t s_misc = s_p + p.p_bufs * p_bytes;
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

    Ctl ctl{abort_flag, p.status, p.wait_limit};

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
            if (round < U) {
                const Seg sg = get_seg(p, round, head_local, rank);
                if (lane == 0) check_len(p, sg);
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
            // O^T += V^T [P_hi | P_lo]^T : A = V^T and B = P^T both MN-major, N = 2 * rows
            const uint32_t idesc_pv = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                                      ((uint32_t)((2 * N) >> 3) << 17) | ((128u >> 4) << 24);
            // The tile tasks of this CTA form one sequence (P1 tiles of unit r, then P2 tiles of
            // unit r-1, for r = 0..U).  Two cursors walk it: QK^T runs `lookahead` tasks ahead of
            // P V so that the next score tiles are ready while the softmax warps work.
            Cursor qc, pc;
            qc.start(p, head_local, rank);
            pc.start(p, head_local, rank);
            while (!pc.done && pc.phase == 0) pc.next(p, head_local, rank);  // PV only visits P2 tasks
            const uint32_t lookahead = p.n_slots >= 4 ? 2u : 1u;
            uint32_t pv_idx = 0, o_phase = 0;
            bool ok = true;
            auto issue_qk = [&]() -> bool {
                const uint32_t s = qc.slot % p.n_slots, sph = (qc.slot / p.n_slots) & 1;
                const uint32_t sb = qc.idx & 1, sbph = (qc.idx >> 1) & 1;
                if (qc.phase == 0 && qc.t == qc.t0) {
                    if (!mbar_wait(B.q_full + 8 * qc.qb, qc.qph, ctl, 15)) return false;
                }
                if (!mbar_wait(B.slot_full + 8 * s, sph, ctl, 13)) return false;
                if (!mbar_wait(B.s_empty + 8 * sb, sbph ^ 1, ctl, 14)) return false;
                tc_fence_after();
                const uint32_t k_addr = s_slots + s * kSlotBytes;
                const uint32_t q_addr = s_q + qc.qb * q_bytes;
                const uint32_t d_s = tmem_base + (sb ? kColS1 : kColS0);
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t a = desc_kmajor(k_addr + (ks >> 2) * 16384 + (ks & 3) * 32);
                    const uint64_t b = desc_kmajor(q_addr + (ks >> 2) * (N * 128) + (ks & 3) * 32);
                    tc_mma(d_s, a, b, idesc_qk, ks ? 1u : 0u);
                }
                tc_commit(B.s_full + 8 * sb);
                tc_commit(B.slot_empty + 8 * s);
                if (qc.phase == 1 && qc.t == qc.t1 - 1) tc_commit(B.q_empty + 8 * qc.qb);  // last use of this Q
                return true;
            };
            auto issue_pv = [&]() -> bool {
                const uint32_t vslot = pc.slot + 1;  // the V tile follows the K tile in the ring
                const uint32_t s = vslot % p.n_slots, sph = (vslot / p.n_slots) & 1;
                const uint32_t pb = pv_idx % p.p_bufs, pph = (pv_idx / p.p_bufs) & 1;
                ++pv_idx;
                const bool first = pc.t == pc.t0, last = pc.t == pc.t1 - 1;
                if (!mbar_wait(B.slot_full + 8 * s, sph, ctl, 10)) return false;
                if (!mbar_wait(B.p_full + 8 * pb, pph, ctl, 11)) return false;
                if (first) {
                    if (!mbar_wait(B.o_empty, o_phase ^ 1, ctl, 12)) return false;
                }
                tc_fence_after();
                const uint32_t v_addr = s_slots + s * kSlotBytes;
                const uint32_t p_addr = s_p + pb * p_bytes;
                const uint32_t d_o = tmem_base + kColO;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t a = desc_mnmajor(v_addr + ks * 2048);
                    const uint64_t b = desc_mnmajor(p_addr + ks * 2048);
                    tc_mma(d_o, a, b, idesc_pv, (first && ks == 0) ? 0u : 1u);
                }
                tc_commit(B.slot_empty + 8 * s);
                tc_commit(B.p_empty + 8 * pb);
                if (last) {
                    tc_commit(B.o_full);
                    o_phase ^= 1;
                }
                return true;
            };
            while (ok && !(qc.done && pc.done)) {
                if (!qc.done && (pc.done || qc.idx < pc.idx + lookahead)) {
                    ok = issue_qk();
                    qc.next(p, head_local, rank);
                } else {
                    ok = issue_pv();
                    do pc.next(p, head_local, rank);
                    while (!pc.done && pc.phase == 0);
                }
            }
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
            if (round >= 1 && ok) {
                // ------------------------------ P2 ------------------------------
                const Seg sg = get_seg(p, round - 1, head_local, rank);
                const int64_t obase = (((int64_t)((round - 1) % kRing) * p.HG + head_local) * p.cph + rank) * R * kD;
                if (prev_nonempty) {
                    const uint32_t lb = prev_lse_idx & 1, lph = (prev_lse_idx >> 1) & 1;
                    ok = mbar_wait(B.lse_full + 8 * lb, lph, ctl, 21);
                    if (!ok) break;
                    const float4* lse4 = reinterpret_cast<const float4*>(lse_s + lb * 128 + c0);
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
                        // [P_hi | P_lo]^T as the B operand, rows contiguous (MN-major, 128-byte swizzle):
                        // 16-byte chunk j (rows 8j..8j+7 of the concatenation) of key k lives at
                        // (j/8)*16384 + k*128 + ((j%8) ^ (k%8))*16
                        uint8_t* p_row = sgen + (s_p - sbase) + pb * p_bytes + key_l * 128;
#pragma unroll
                        for (int nb = 0; nb < NH / 8; ++nb) {
                            uint32_t hi[4], lo[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                // p = hi + lo with both parts cut to bf16 by truncation (plain integer ops, no

                                // conversion instructions): hi keeps the top 16 bits, lo the top 16 bits of the exact

                                // remainder, so p - (hi + lo) < 2^-14 p

                                const uint32_t ua = __float_as_uint(pr[nb * 8 + 2 * q]), ub = __float_as_uint(pr[nb * 8 + 2 * q + 1]);

                                hi[q] = __byte_perm(ua, ub, 0x7632);

                                const float ra = __uint_as_float(ua) - __uint_as_float(ua & 0xffff0000u);

                                const float rb = __uint_as_float(ub) - __uint_as_float(ub & 0xffff0000u);

                                lo[q] = __byte_perm(__float_as_uint(ra), __float_as_uint(rb), 0x7632);
                            }
                            const int jh = wg * (NH / 8) + nb, jl = jh + 2 * NH / 8;
                            *reinterpret_cast<uint4*>(p_row + (jh >> 3) * 16384 + (((jh & 7) ^ (key_l & 7)) << 4)) =
                                make_uint4(hi[0], hi[1], hi[2], hi[3]);
                            *reinterpret_cast<uint4*>(p_row + (jl >> 3) * 16384 + (((jl & 7) ^ (key_l & 7)) << 4)) =
                                make_uint4(lo[0], lo[1], lo[2], lo[3]);
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
                            if (key < sg.T) {
                                float* dst = p.a.stats + sg.prob * p.a.stat_stride + key;
                                const float v = st + stat_tmp[sq * 128 + key_l];
                                *dst = p.a.stat_accumulate ? *dst + v : v;
                            }
                        }
                    }
                    if (!ok) break;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(B.lse_empty + 8 * lb);
                    // ---- epilogue: O^T (d on lanes, rows on columns) -> partial [r][d] ----
                    ok = mbar_wait(B.o_full, o_phase, ctl, 25);
                    if (!ok) break;
                    o_phase ^= 1;
                    tc_fence_after();
                    uint32_t v[NH], w[NH];
                    load_cols<NH>(t_lane + kColO + c0, v);          // P_hi part
                    load_cols<NH>(t_lane + kColO + N + c0, w);      // P_lo part
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(B.o_empty);
#pragma unroll
                    for (int i = 0; i < NH; ++i) {
                        const int r = c0 + i;
                        if (r < R) p.o_part[obase + (int64_t)r * kD + key_l] = __uint_as_float(v[i]) + __uint_as_float(w[i]);
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
                if (p.a.out_bf16)
                    reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.a.out) + row * kD)[d4] =
                        make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
                else
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
                    ok = counter_wait(p.counters + unit * p.HG + head_local, p.cph, ctl, 31);
                    if (!ok) break;
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
                }
            }
            if (round >= 2) ok = reduce_unit(round - 2);
        }
    }

    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    if (!*abort_flag) reset_counters_if_last(p, reinterpret_cast<int*>(const_cast<uint32_t*>(tmem_slot)));
}

template <int NH>
int launch_nh(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const FastParams& fp,
              int grid, size_t smem_bytes, cudaStream_t stream)
{
    auto kern = verify_twosweep_kernel<NH>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
        return SPEC_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs must be co-resident: they wait on each other
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

int launch_twosweep(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const FastParams& fp,
                    int grid, size_t smem_bytes, cudaStream_t stream)
{
    switch (fp.N / 2) {
        case 8: return launch_nh<8>(tk, tv, tq, fp, grid, smem_bytes, stream);
        case 16: return launch_nh<16>(tk, tv, tq, fp, grid, smem_bytes, stream);
        case 24: return launch_nh<24>(tk, tv, tq, fp, grid, smem_bytes, stream);
        case 32: return launch_nh<32>(tk, tv, tq, fp, grid, smem_bytes, stream);
        case 40: return launch_nh<40>(tk, tv, tq, fp, grid, smem_bytes, stream);
        case 48: return launch_nh<48>(tk, tv, tq, fp, grid, smem_bytes, stream);
        case 56: return launch_nh<56>(tk, tv, tq, fp, grid, smem_bytes, stream);
        case 64: return launch_nh<64>(tk, tv, tq, fp, grid, smem_bytes, stream);
        default: return SPEC_ERR_UNSUPPORTED_SHAPE;
    }
}

}  // namespace sm100
}  // namespace spec
