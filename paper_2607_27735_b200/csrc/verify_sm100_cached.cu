// Verification attention + Eq. 3 statistic for sm_100a, score-cache variant: one persistent,
// warp-specialised kernel on TMA (no multicast), tcgen05.mma with TMEM accumulators and
// mbarrier pipelines, in which K and V are each read exactly once from memory.
//
// Eq. 3 sums softmax PROBABILITIES over the window rows, so a key's contribution
// exp(s - LSE_row) needs every row's global normaliser, which is known only after all keys
// of the head were seen.  Instead of sweeping K twice, every CTA keeps the score tiles
// S^T = K Q^T of its share of the keys in tensor memory (512 columns per SM hold the output
// accumulator plus (512 - 2N) / N tiles of 128 keys x N rows):
//   P1   stream K, S^T tile -> TMEM (kept), per-row running (max, sum) -> this CTA's partial,
//        published to the CTAs that share the head;
//   P2a  stream V, P~ = exp2(S - lse_local) from the cached tile (needs nothing from other CTAs,
//        so the exchange of the partials hides behind it): O^T += V^T [P~_hi | P~_lo]^T on the
//        tensor cores (bf16 hi + lo split of P~ keeps the 2e-3 bar when one key takes most of the
//        mass); P~ replaces the scores in tensor memory;
//   --   the partials of the head's CTAs are combined into the row LSE (the only cross-CTA
//        dependency), by the publisher warp during P2a when few CTAs share the head;
//   P2b  cached P~ weighted per row with exp2(lse_local - LSE): column sums -> stats;
//   --   the accumulator, rescaled per row the same way, is this CTA's partial output.
// A unit (a group of KV heads of one (layer, sequence)) is cut so that a CTA's share of keys
// fits the cache; larger shares go to the two-sweep variant.
//
// TMEM tile layout: keys on the 128 lanes, the R = n_q * group query rows on the columns, so
// one thread owns one key: the statistic is a thread-local sum and the P1 row max/sum is
// thread-local state reduced once per unit.
//
// Roles (128 + 128 CG threads): warp 0 TMA producer, warp 1 tcgen05.mma issuer (+ TMEM alloc),
// warp 2 publisher (fences, counters, LSE combine), warp 3 reduces the per-CTA O partials (fixed
// order: deterministic), warps 4.. CG softmax warpgroups that split the columns.
//
// All CTAs must become co-resident (they wait on each other's partials): the grid never exceeds
// the SM count at one CTA per SM (see the launcher).  Every wait is bounded; on expiry the kernel
// records SPEC_ERR_TIMEOUT in the status word and drains.
#include "sm100_common.cuh"

namespace spec {
namespace sm100 {

namespace {


constexpr int kMaxCache = 32;
constexpr int kLsePubMax = 48;  // CTAs per head up to which the publisher warp alone combines the LSE partials

// Cross-lane reduction of per-column (max, sum of exp2(x - max)) pairs.  While the number of
// columns a lane carries is even, partners exchange halves (the lane with bit `o` set keeps the
// upper half), so the traffic halves at every step; an odd count is reduced in place on both
// partners.  Afterwards a lane holds ml_final_n(NH) columns starting at `col`, and lanes that
// differ only in the bits of ml_dupmask(NH) hold the same ones.
__host__ __device__ constexpr int ml_final_n(int n)
{
    for (int o = 16; o >= 1; o >>= 1)
        if (n % 2 == 0) n /= 2;
    return n;
}
__host__ __device__ constexpr uint32_t ml_dupmask(int n)
{
    uint32_t d = 0;
    for (int o = 16; o >= 1; o >>= 1) {
        if (n % 2 == 0) n /= 2;
        else d |= (uint32_t)o;
    }
    return d;
}
template <int NHT, int n, int o>
__device__ __forceinline__ void ml_step(float (&m)[NHT], float (&l)[NHT], int lane, int& col)
{
    if constexpr (o >= 1) {
        if constexpr (n % 2 == 0) {
            constexpr int h = n / 2;
            const bool up = (lane & o) != 0;
#pragma unroll
            for (int j = 0; j < h; ++j) {
                const float sm = up ? m[j] : m[j + h], sl = up ? l[j] : l[j + h];
                const float km = up ? m[j + h] : m[j], kl = up ? l[j + h] : l[j];
                const float rm = __shfl_xor_sync(0xffffffffu, sm, o), rl = __shfl_xor_sync(0xffffffffu, sl, o);
                const float M = fmaxf(km, rm);
                m[j] = M;
                l[j] = kl * ex2(km - M) + rl * ex2(rm - M);
            }
            col += up ? h : 0;
            ml_step<NHT, h, o / 2>(m, l, lane, col);
        } else {
#pragma unroll
            for (int j = 0; j < n; ++j) {
                const float rm = __shfl_xor_sync(0xffffffffu, m[j], o), rl = __shfl_xor_sync(0xffffffffu, l[j], o);
                const float M = fmaxf(m[j], rm);
                l[j] = l[j] * ex2(m[j] - M) + rl * ex2(rm - M);
                m[j] = M;
            }
            ml_step<NHT, n, o / 2>(m, l, lane, col);
        }
    }
}

// Four e4m3 bytes as two packed fp16 pairs (bytes 0, 1 and bytes 2, 3): exact, subnormals included.
// (The same by integer instructions - the byte's low seven bits shifted into bits 7..13 of an fp16 give the
// value times 2^-8 - measured slower: the softmax warps are bound by instruction issue, and that takes four
// instructions per pair instead of one.)
__device__ __forceinline__ void e4m3x4_to_f16x4(uint32_t w, uint32_t& lo, uint32_t& hi)
{
    asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.rn.f16x2.e4m3x2 %0, a;\n\tcvt.rn.f16x2.e4m3x2 %1, b;\n\t}"
        : "=r"(lo), "=r"(hi)
        : "r"(w));
}

struct CBars {  // mbarrier addresses (shared space)
    uint32_t slot_full, slot_empty, q_full, q_empty, s_full, s_free, p_full, p_empty, o_full, o_empty, sm_sync,
        pub_p1, pub_o, lse_ready, raw_full, raw_empty, q_ready;
};

// NC = score columns per softmax warpgroup, CG = number of such warpgroups (N = NC * CG):
// more, narrower warpgroups hide the latency of the serial softmax sections.
// LP: the publisher warp combines the LSE partials (few CTAs per head); otherwise the softmax warps do.
// PH: one Eq. 3 score per attention head (stats [.., n_q_heads, stride]) instead of per KV head,
// for groups of at most 8 heads (a short statistic pass when the group size divides 8).
// SC: per-(layer, KV head) scales of K and V (an 8-bit cache, expanded to bf16 beforehand or here).
// F8: the cache holds e4m3 bytes.  TMA brings a tile's bytes (16 KB) into a ring of raw stages; the
// softmax warps expand a tile one or two places ahead into the operand slot while the tensor cores
// work on the current one (cvt.rn.f16x2.e4m3x2: every e4m3 value is an fp16 value).  Both products then run on
// fp16 operands: Q is converted once per unit in shared memory, P~ is split into an fp16 rounding of
// 2^14 P~ and the fp16 rounding of 2^11 times its remainder (the two accumulator halves are added with
// that weight in the epilogue); the powers of two join the scales.
template <int NC, int CG, bool LP, bool PH, bool SC, bool F8>
__global__ void __launch_bounds__(128 + 128 * CG, 1)
verify_cached_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     const __grid_constant__ CUtensorMap tm_q, const FastParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));  // generic pointer to the aligned base

    constexpr int NH = NC;                       // columns per thread
    constexpr int kBlock = 128 + 128 * CG;       // threads per CTA
    constexpr int kSW = 4 * CG;                  // softmax warps
    const int N = p.N, R = p.R, G = p.G;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int head_local = fast_div(p, 2, blockIdx.x), rank = blockIdx.x - head_local * p.cph;
    const int q_bytes = N * 256;                       // one Q buffer: 2 halves x N rows x 128 B
    const int p_bytes = 2 * N * 256;                   // one P buffer: [hi | lo] rows, 8-row blocks x 128 keys x 16 B

    const uint32_t s_slots = sbase;
    const uint32_t s_raw = s_slots + p.n_slots * kSlotBytes;  // F8: n_raw stages of 16 KB
    const uint32_t s_q = s_raw + (F8 ? p.n_raw * 16384 : 0);
    const uint32_t s_p = s_q + q_bytes;                // one Q buffer: the next unit's Q lands after this unit's last QK^T
    const uint32_t s_misc = s_p + p.p_bufs * p_bytes;
    uint8_t* misc = sgen + (s_misc - sbase);
    CBars B;
    {
        uint32_t o = s_misc;
        B.slot_full = o; o += 8 * 8;
        B.slot_empty = o; o += 8 * 8;
        B.q_full = o; o += 16;
        B.q_empty = o; o += 16;
        B.s_full = o; o += 8 * kMaxCache;
        B.s_free = o; o += 8 * kMaxCache;
        B.p_full = o; o += 32;  // up to four P buffers
        B.p_empty = o; o += 32;  // four: indexed by tile sequence number mod 4 (see the P2 loop)
        B.o_full = o; o += 8;
        B.o_empty = o; o += 8;
        B.sm_sync = o; o += 8;
        B.pub_p1 = o; o += 8;   // the last softmax warp stored this CTA's (max, sum) partial
        B.pub_o = o; o += 8;    // every softmax warp stored its share of the output partial
        B.lse_ready = o; o += 8;  // the publisher warp left the row LSE and the rescale factors in shared memory
        B.raw_full = o; o += 32;  // F8: a tile's bytes have landed in a raw stage
        B.raw_empty = o; o += 32; // F8: every softmax warp has expanded its part of the stage
        B.q_ready = o; o += 8;    // F8: Q is fp16 in shared memory
    }
    float* lse_s = reinterpret_cast<float*>(misc + 1024);                 // [128] global row LSE (log2 domain)
    float* loc_s = reinterpret_cast<float*>(misc + 1024 + 512);           // [128] CTA-local row LSE
    float* fac_s = reinterpret_cast<float*>(misc + 2048);                 // [128] exp2(local - global)
    uint32_t* hist_s = reinterpret_cast<uint32_t*>(misc + 2560);          // [1024] packed 16-bit counts of score bins, 4 KB
    float2* red = reinterpret_cast<float2*>(misc + 8192);                 // [kSW warps][NC] (m, l), <= 4 KB
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 12288);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    Ctl ctl{abort_flag, p.status, p.wait_limit};

    if (threadIdx.x < kMaxCache) {  // one region's pair of barriers per thread
        mbar_init(B.s_full + 8 * threadIdx.x, 1);
        mbar_init(B.s_free + 8 * threadIdx.x, 4);
    } else if (threadIdx.x < kMaxCache + 8) {
        const int i = threadIdx.x - kMaxCache;
        if (i < p.n_slots) {
            mbar_init(B.slot_full + 8 * i, F8 ? kSW : 1);  // F8: filled by the softmax warps, not by TMA
            mbar_init(B.slot_empty + 8 * i, 1);
        }
        if (F8 && i < 4) {
            mbar_init(B.raw_full + 8 * i, 1);
            mbar_init(B.raw_empty + 8 * i, kSW);
        }
        if (i < 2) {
            mbar_init(B.q_full + 8 * i, 1);
            mbar_init(B.q_empty + 8 * i, 1);
        }
        if (i < 4) {
            mbar_init(B.p_full + 8 * i, kSW);
            mbar_init(B.p_empty + 8 * i, 1);
        }
    } else if (threadIdx.x == kMaxCache + 8) {
        mbar_init(B.o_full, 1);
        mbar_init(B.o_empty, kSW);
        mbar_init(B.sm_sync, kSW);
        mbar_init(B.pub_p1, 1);
        mbar_init(B.pub_o, kSW);
        mbar_init(B.lse_ready, 1);
        if (F8) mbar_init(B.q_ready, kSW);
        *abort_flag = 0;
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // zero the Q buffers once: rows R..N-1 are padding the TMA never writes
    for (int i = threadIdx.x; i < q_bytes / 16; i += kBlock)
        *reinterpret_cast<uint4*>(sgen + (s_q - sbase) + 16 * i) = make_uint4(0, 0, 0, 0);
    if (p.a.hist)
        for (int i = threadIdx.x; i < kScoreBins / 2; i += kBlock) hist_s[i] = 0u;
    if (p.D == 64) {  // the upper 64-wide half of every tile slot is never loaded: zero rows of V^T (and of K)
        for (int i = threadIdx.x; i < p.n_slots * 1024; i += kBlock)
            *reinterpret_cast<uint4*>(sgen + (s_slots - sbase) + (i >> 10) * kSlotBytes + 16384 + 16 * (i & 1023)) =
                make_uint4(0, 0, 0, 0);
    }
    for (int r = R + threadIdx.x; r < 128; r += kBlock) {  // padded rows: P = 0
        lse_s[r] = 1.0e30f;
        loc_s[r] = 1.0e30f;
        fac_s[r] = 0.f;
    }
    fence_proxy_async();
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // Programmatic dependent launch: this kernel's prologue above may run while the previous
    // kernel in the stream drains; nothing before this point touches global memory the stream
    // produces (the workspace is shared with the previous call).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const int U = p.n_units;
    const uint32_t col_o = 0, col_s = 2 * N;  // O^T (hi | lo) first, then the cached S^T tiles

    if (warp == 0) {
        // =========================== TMA producer ===========================
        uint32_t slot_idx = 0, qn = 0;
        const int boxes = p.boxes, box_rows = p.box_rows;
        const uint32_t box_bytes = box_rows * 128;
        const int halves = p.D / 64;  // 64-wide halves of the head dimension
        bool ok = true;
        auto load_tile = [&](const CUtensorMap* map, const Seg& sg, int tile) -> bool {
            if (F8) {
                // the tile's bytes (128 per key) go to a raw stage; the softmax warps expand them into a slot
                const uint32_t r = slot_idx % p.n_raw, rph = (slot_idx / p.n_raw) & 1;
                ++slot_idx;
                bool got = true;
                if (lane == 0) got = mbar_wait(B.raw_empty + 8 * r, rph ^ 1, ctl, 3);
                if (!__shfl_sync(0xffffffffu, got ? 1 : 0, 0)) return false;
                const int key0 = tile * kTile;
                const int n_box = min(boxes, (sg.T - key0 + box_rows - 1) / box_rows);
                if (lane == 0) mbar_expect_tx(B.raw_full + 8 * r, (uint32_t)n_box * box_bytes);
                __syncwarp();
                for (int bx = lane; bx < n_box; bx += 32) {
                    const int pos = key0 + bx * box_rows;
                    const int page = page_of(p.a.kv, pos), slot_in_page = pos - page * p.a.kv.page_size;
                    int phys = p.a.kv.page_table ? __ldg(p.a.kv.page_table + (int64_t)sg.b * p.a.kv.max_pages + page)
                                                 : sg.b * p.a.kv.max_pages + page;
                    if (phys < 0 || phys >= p.n_pages) {
                        set_status(p.status, SPEC_ERR_BAD_INDEX);
                        phys = 0;
                    }
                    tma_load_5d(s_raw + r * 16384 + bx * box_bytes, map, B.raw_full + 8 * r, 0, slot_in_page, sg.h, phys,
                                sg.layer, kEvictFirst);
                }
                __syncwarp();
                return true;
            }
            const uint32_t s = slot_idx % p.n_slots, ph = (slot_idx / p.n_slots) & 1;
            ++slot_idx;
            bool got = true;
            if (lane == 0) got = mbar_wait(B.slot_empty + 8 * s, ph ^ 1, ctl, 1);  // one lane polls
            if (!__shfl_sync(0xffffffffu, got ? 1 : 0, 0)) return false;
            // boxes of this tile that hold at least one key < T (pages past the context may not exist)
            const int key0 = tile * kTile;
            const int n_box = min(boxes, (sg.T - key0 + box_rows - 1) / box_rows);
            if (lane == 0) mbar_expect_tx(B.slot_full + 8 * s, (uint32_t)halves * n_box * box_bytes);
            __syncwarp();
            for (int i = lane; i < halves * n_box; i += 32) {
                const int half = i >= n_box ? 1 : 0, bx = i - half * n_box;  // i < 2 * n_box
                const int pos = key0 + bx * box_rows;
                const int page = page_of(p.a.kv, pos), slot_in_page = pos - page * p.a.kv.page_size;
                int phys = p.a.kv.page_table ? __ldg(p.a.kv.page_table + (int64_t)sg.b * p.a.kv.max_pages + page)
                                             : sg.b * p.a.kv.max_pages + page;
                if (phys < 0 || phys >= p.n_pages) {
                    set_status(p.status, SPEC_ERR_BAD_INDEX);
                    phys = 0;
                }
                const uint32_t dst = s_slots + s * kSlotBytes + half * 16384 + bx * box_bytes;
                tma_load_5d(dst, map, B.slot_full + 8 * s, half * 64, slot_in_page, sg.h, phys, sg.layer, kEvictFirst);
            }
            __syncwarp();
            return true;
        };
        for (int u = 0; u < U && ok; ++u) {
            const Seg sg = get_seg(p, u, head_local, rank);
            if (lane == 0) check_len(p, sg);
            if (sg.t1 <= sg.t0) continue;
            const uint32_t qb = 0, qph = qn & 1;
            ++qn;
            ok = mbar_wait(B.q_empty + 8 * qb, qph ^ 1, ctl, 2);
            if (!ok) break;
            if (lane == 0) {
                mbar_expect_tx(B.q_full + 8 * qb, (uint32_t)halves * R * 128);
                const int row0 = (sg.layer * p.a.kv.batch + sg.b) * p.a.n_q;
                tma_load_3d(s_q + qb * q_bytes, &tm_q, B.q_full + 8 * qb, 0, sg.h * G, row0);
                if (halves == 2) tma_load_3d(s_q + qb * q_bytes + N * 128, &tm_q, B.q_full + 8 * qb, 64, sg.h * G, row0);
            }
            __syncwarp();
            for (int t = sg.t0; t < sg.t1 && ok; ++t) ok = load_tile(&tm_k, sg, t);
            for (int t = sg.t0; t < sg.t1 && ok; ++t) ok = load_tile(&tm_v, sg, t);
        }
        if (!ok) {  // let copies in flight land before the CTA's shared memory is released
            const long long t0 = clock64();
            while (clock64() - t0 < 400000ll) __nanosleep(1000);
        }
    } else if (warp == 1) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            // operand formats (bits 7-9 and 10-12): 1 = bf16, 0 = fp16 (F8: both products on fp16 operands)
            const uint32_t ab_fmt = F8 ? 0u : ((1u << 7) | (1u << 10));
            const uint32_t idesc_qk = (1u << 4) | ab_fmt | ((uint32_t)(N >> 3) << 17) | ((128u >> 4) << 24);
            // O^T += V^T [P_hi | P_lo]^T : A = V^T and B = P^T both MN-major, N = 2 * rows
            const uint32_t idesc_pv = (1u << 4) | ab_fmt | (1u << 15) | (1u << 16) |
                                      ((uint32_t)((2 * N) >> 3) << 17) | ((128u >> 4) << 24);
            // Two independent queues, issued in whichever order their inputs become ready: the
            // QK^T tiles of unit u+1 may overtake the P V tiles of unit u that still wait for P.
            struct Queue {
                int u = -1, t = 0, t0 = 0, t1 = 0;
                uint32_t slot_base = 0;  // ring index of the unit's first K tile
                uint32_t next_base = 0;  // ring index where the following unit starts
                uint32_t qn = 0, qb = 0, qph = 0;
                bool done = false;
            } qq, pq;
            auto seek = [&](Queue& c) {  // advance to the next unit with tiles
                for (;;) {
                    ++c.u;
                    if (c.u >= U) {
                        c.done = true;
                        return;
                    }
                    const Seg sg = get_seg(p, c.u, head_local, rank);
                    if (sg.t1 > sg.t0) {
                        c.t0 = sg.t0;
                        c.t1 = sg.t1;
                        c.t = sg.t0;
                        c.slot_base = c.next_base;
                        c.next_base += 2 * (sg.t1 - sg.t0);
                        c.qb = 0;
                        c.qph = c.qn & 1;
                        ++c.qn;
                        return;
                    }
                }
            };
            seek(qq);
            seek(pq);
            uint32_t sfree_par = 0;  // per cache region: parity of the next "region free" phase
            uint32_t pv_idx = 0, o_phase = 0;
            bool ok = true;
            auto qk_ready = [&]() -> bool {
                const int c = qq.t - qq.t0;
                const uint32_t slot = qq.slot_base + c;
                const uint32_t s = slot % p.n_slots, sph = (slot / p.n_slots) & 1;
                if (c == 0 && !mbar_test_wait(F8 ? B.q_ready : B.q_full + 8 * qq.qb, qq.qph)) return false;
                if (!mbar_test_wait(B.slot_full + 8 * s, sph)) return false;
                return mbar_test_wait(B.s_free + 8 * c, ((sfree_par >> c) & 1) ^ 1);
            };
            auto issue_qk = [&]() {
                const int c = qq.t - qq.t0;
                const uint32_t slot = qq.slot_base + c;
                const uint32_t s = slot % p.n_slots;
                sfree_par ^= 1u << c;
                tc_fence_after();
                const uint32_t k_addr = s_slots + s * kSlotBytes;
                const uint32_t q_addr = s_q + qq.qb * q_bytes;
                const uint32_t d_s = tmem_base + col_s + c * N;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    if (ks * 16 < p.D) {  // head_dim 64: the first four 16-wide steps
                        const uint64_t a = desc_kmajor(k_addr + (ks >> 2) * 16384 + (ks & 3) * 32);
                        const uint64_t b = desc_kmajor(q_addr + (ks >> 2) * (N * 128) + (ks & 3) * 32);
                        tc_mma(d_s, a, b, idesc_qk, ks ? 1u : 0u);
                    }
                }
                tc_commit(B.s_full + 8 * c);
                tc_commit(B.slot_empty + 8 * s);
                if (qq.t == qq.t1 - 1) tc_commit(B.q_empty + 8 * qq.qb);  // last use of this Q buffer
                if (++qq.t == qq.t1) seek(qq);
            };
            auto pv_ready = [&]() -> bool {
                const int c = pq.t - pq.t0;
                const uint32_t slot = pq.slot_base + (pq.t1 - pq.t0) + c;
                const uint32_t s = slot % p.n_slots, sph = (slot / p.n_slots) & 1;
                const uint32_t pb = pv_idx % p.p_bufs, pph = (pv_idx / p.p_bufs) & 1;
                if (!mbar_test_wait(B.p_full + 8 * pb, pph)) return false;
                if (!mbar_test_wait(B.slot_full + 8 * s, sph)) return false;
                if (c == 0 && !mbar_test_wait(B.o_empty, o_phase ^ 1)) return false;
                return true;
            };
            auto issue_pv = [&]() {
                const int c = pq.t - pq.t0;
                const uint32_t slot = pq.slot_base + (pq.t1 - pq.t0) + c;
                const uint32_t s = slot % p.n_slots;
                const uint32_t pb = pv_idx % p.p_bufs;
                const uint32_t pe = pv_idx & 3;
                ++pv_idx;
                const bool first = c == 0, last = pq.t == pq.t1 - 1;
                tc_fence_after();
                const uint32_t v_addr = s_slots + s * kSlotBytes;
                const uint32_t p_addr = s_p + pb * p_bytes;
                const uint32_t d_o = tmem_base + col_o;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t a = desc_mnmajor(v_addr + ks * 2048);
                    const uint64_t b = desc_mnmajor_nosw(p_addr + ks * 256);
                    tc_mma(d_o, a, b, idesc_pv, (first && ks == 0) ? 0u : 1u);
                }
                tc_commit(B.slot_empty + 8 * s);
                tc_commit(B.p_empty + 8 * pe);
                if (last) {
                    tc_commit(B.o_full);
                    o_phase ^= 1;
                }
                if (++pq.t == pq.t1) seek(pq);
            };
            long long t_idle = clock64();
            uint32_t spins = 0;
            while (ok && !(qq.done && pq.done)) {
                bool progressed = false;
                // a unit's P V tiles can only follow its own QK^T tiles
                if (!pq.done && (qq.done || qq.u > pq.u) && pv_ready()) {
                    issue_pv();
                    progressed = true;
                }
                if (!qq.done && qk_ready()) {
                    issue_qk();
                    progressed = true;
                }
                if (progressed) {
                    spins = 0;
                    continue;
                }
                __nanosleep(40);  // idle: leave the issue slots of this sub-core to the softmax warps
                if ((++spins & 63u) == 0) {
                    if (spins == 64) t_idle = clock64();
                    if (*ctl.abort_flag) ok = false;
                    else if (clock64() - t_idle > ctl.limit) {
                        report_timeout(ctl, 16);
                        ok = false;
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 2) {
        // =========================== publisher warp ===========================
        // Makes this CTA's partials visible to the other CTAs (device-scope fence + counter), so
        // that no softmax warp ever waits for that round trip: they only arrive on a CTA barrier.
        // It also combines the (max, sum) partials of the CTAs that share the head into the row
        // LSE while the softmax warps are busy with the P V pass.
        bool ok = true;
        for (int unit = 0; unit < U && ok; ++unit) {
            if (lane == 0) {
                ok = mbar_wait(B.pub_p1, unit & 1, ctl, 34);
                if (ok) {
                    __threadfence();
                    atomicAdd(p.counters + unit * p.HG + head_local, 1);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const Seg sg = get_seg(p, unit, head_local, rank);
            if (LP && sg.t1 > sg.t0) {
                // ---- row LSE from the partials of the CTAs that share this head ----
                if (lane == 0) ok = counter_wait(p.counters + unit * p.HG + head_local, p.cph, ctl, 31);
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;  // lane 0's acquire, then warp-wide
                if (!ok) break;
                const float2* src = p.ml_part + ((int64_t)(unit % kRing) * p.HG + head_local) * p.cph * R;
                // two lanes per row, 16 rows per pass: each lane folds every other partial, 20 loads in flight
                const int sub = lane & 1;
                for (int r0 = 0; r0 < R; r0 += 16) {
                    const int r = r0 + (lane >> 1);
                    float M = -1.0e30f, Ls = 0.f;
                    if (r < R) {
                        for (int k0 = sub; k0 < p.cph; k0 += 40) {
                            float2 x[20];
                            const float2* q = src + (int64_t)k0 * R + r;
                            const int n_ld = (p.cph - k0 + 1) >> 1;  // partials k0, k0 + 2, ... below cph
#pragma unroll
                            for (int u = 0; u < 20; ++u) {
                                x[u] = make_float2(-1.0e30f, 0.f);
                                if (u < n_ld) x[u] = __ldcg(q + u * 2 * R);
                            }
                            float Mn = M;
#pragma unroll
                            for (int u = 0; u < 20; ++u) Mn = fmaxf(Mn, x[u].x);
                            Ls *= ex2(M - Mn);
#pragma unroll
                            for (int u = 0; u < 20; ++u) Ls = fmaf(x[u].y, ex2(x[u].x - Mn), Ls);
                            M = Mn;
                        }
                    }
                    const float M2 = __shfl_xor_sync(0xffffffffu, M, 1);
                    const float L2 = __shfl_xor_sync(0xffffffffu, Ls, 1);
                    const float Mn = fmaxf(M, M2);
                    Ls = Ls * ex2(M - Mn) + L2 * ex2(M2 - Mn);
                    M = Mn;
                    if (sub == 0 && r < R) {
                        const float lse2 = M + log2f(Ls);
                        lse_s[r] = lse2;
                        const float loc = loc_s[r];
                        fac_s[r] = loc < 1.0e29f ? ex2(loc - lse2) : 0.f;  // local -> global normaliser
                        if (rank == p.cph - 1 && p.a.lse) {  // the last rank always owns at least one tile
                            const int j = r / G, g = r - j * G;
                            const int64_t row = (((int64_t)sg.layer * p.a.kv.batch + sg.b) * p.a.n_q + j) * p.a.kv.n_q_heads + sg.h * G + g;
                            p.a.lse[row] = lse2 * 0.69314718055994530942f;
                        }
                    }
                }
            }
            // signalled for every unit, empty ones too: the softmax warps wait for it before they go
            // on, so they are never more than one barrier phase ahead of this warp
            __syncwarp();
            if (lane == 0) mbar_arrive(B.lse_ready);
            if (lane == 0) {
                ok = mbar_wait(B.pub_o, unit & 1, ctl, 35);
                if (ok) {
                    __threadfence();
                    atomicAdd(p.counters + U * p.HG + unit * p.HG + head_local, 1);
                }
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        }
    } else if (warp == 3) {
        // =========================== O reduction warp ===========================
        const int tid = lane;
        bool ok = true;
        for (int unit = 0; unit < U && ok; ++unit) {
            if (lane == 0) ok = counter_wait(p.counters + U * p.HG + unit * p.HG + head_local, p.cph, ctl, 30);
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const Seg sg = get_seg(p, unit, head_local, rank);
            const int E4 = R * kD / 4;
            const int lo = fast_div(p, 2, rank * E4), hi = fast_div(p, 2, (rank + 1) * E4);  // products far below 2^31
            const float4* src = reinterpret_cast<const float4*>(
                p.o_part + ((int64_t)(unit % kRing) * p.HG + head_local) * p.cph * R * kD);
            for (int e = lo + tid; e < hi; e += 32) {
                const int r = e / (kD / 4), d4 = e - r * (kD / 4);
                if (d4 * 4 >= p.D) continue;  // head_dim 64: the partial's upper columns are padding
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int k0 = 0; k0 < p.cph; k0 += 16) {  // batches of 16 independent loads
                    float4 x[16];
                    const float4* q = src + (int64_t)k0 * E4 + e;
                    const int n_ld = p.cph - k0;
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        x[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (u < n_ld) x[u] = __ldcg(q + u * E4);
                    }
#pragma unroll
                    for (int u = 0; u < 16; ++u) {
                        acc.x += x[u].x;
                        acc.y += x[u].y;
                        acc.z += x[u].z;
                        acc.w += x[u].w;
                    }
                }
                const int j = r / G, g = r - j * G;
                const int64_t row = (((int64_t)sg.layer * p.a.kv.batch + sg.b) * p.a.n_q + j) * p.a.kv.n_q_heads + sg.h * G + g;
                if (p.a.out_bf16)
                    reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.a.out) + row * p.D)[d4] =
                        make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
                else
                    reinterpret_cast<float4*>(p.a.out + row * p.D)[d4] = acc;
            }
        }
    } else {
        // =========================== softmax warpgroups ===========================
        const int sw = warp - 4;                 // 0..kSW-1
        const int wg = sw >> 2;                  // column group
        const int quarter = warp & 3;            // TMEM lane quarter this warp may touch
        const int key_l = quarter * 32 + lane;   // key within the tile (P1/P2) or d (epilogue)
        const int tid_s = threadIdx.x - 128;     // 0..128*CG-1
        const int c0 = wg * NH;                  // first column of this warpgroup
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const int stat_r0 = p.a.first_stat_row * G;
        const bool ph_fast = (8 % G) == 0;  // per-head statistic: column i of a 16-column chunk is head i mod 8 mod G
        const float cs0 = p.scale_log2;
        float vsc = 1.f;  // SC: scale of this unit's V
        // F8: powers of two that travel with the operands (see the kernel's header)
        constexpr float kPExp = 16384.f;         // P~ is held times 2^14
        constexpr float kLoExp = 2048.f;         // the remainder of its fp16 rounding times 2^11
        uint32_t g_conv = 0, g_total = 0;        // F8: tiles expanded so far / in this launch (K and V of every unit)
        const uint32_t f8_ahead = F8 ? (uint32_t)min(p.n_slots - 2, 2) : 0u;  // tiles expanded ahead of the one in use
        int q_next = 0;                          // F8: first unit whose Q is not converted yet
        uint32_t qn_s = 0;                       // F8: Q buffers seen (phase of q_full / q_ready)
        if (F8) {
            for (int u = 0; u < U; ++u) {
                const Seg s2 = get_seg(p, u, head_local, rank);
                g_total += 2u * (uint32_t)max(s2.t1 - s2.t0, 0);
            }
        }
        // F8: expands the next raw tile (in the order the producer loads them) into the next operand slot.
        // A thread of the softmax warps takes 16-byte pieces of the tile's 1024: piece q of row r holds
        // d = 16 q .. 16 q + 15, i.e. the 16-byte chunks 2 (q % 4) and 2 (q % 4) + 1 of row r in the 64-wide
        // half q / 4 (rows of 128 B, chunks swizzled with the row's low three bits).
        uint32_t cv_r = 0, cv_rph = 0, cv_s = 0, cv_sph = 0;  // ring positions of the next tile to expand (no division per tile)
        // The thread's pieces, the same for every tile: source offset in the raw stage (low half) and offset of
        // the first of the two 16-byte chunks in the slot (high half; the second is its neighbour, offset ^ 16).
        // Eight consecutive threads take eight consecutive rows and eight different pieces: their loads and
        // both of their stores then fall on eight different 16-byte bank groups.
        constexpr int kIter = (1024 + 128 * CG - 1) / (128 * CG);
        uint32_t cv_off[kIter];
#pragma unroll
        for (int k = 0; k < kIter; ++k) {
            const int i = tid_s + k * 128 * CG;
            const int l = i & 7, blk = i >> 3, row = 8 * (blk >> 3) + l, q = (l + blk) & 7;
            const int c0 = (q & 3) * 2, sw = row & 7;
            cv_off[k] = (uint32_t)(row * 128 + q * 16) | ((uint32_t)((q >> 2) * 16384 + row * 128 + ((c0 ^ sw) << 4)) << 16);
        }
        auto convert_tile = [&]() -> bool {
            const uint32_t r = cv_r, rph = cv_rph, s = cv_s, sph = cv_sph;
            if (++cv_r == (uint32_t)p.n_raw) {
                cv_r = 0;
                cv_rph ^= 1;
            }
            if (++cv_s == (uint32_t)p.n_slots) {
                cv_s = 0;
                cv_sph ^= 1;
            }
            if (!mbar_wait(B.raw_full + 8 * r, rph, ctl, 40)) return false;
            if (!mbar_wait(B.slot_empty + 8 * s, sph ^ 1, ctl, 41)) return false;
            const uint8_t* raw = sgen + (s_raw - sbase) + r * 16384;
            uint8_t* slot = sgen + (s_slots - sbase) + s * kSlotBytes;
            uint4 in[kIter];
#pragma unroll
            for (int k = 0; k < kIter; ++k)  // every load of the thread is in flight before the first is used
                if (tid_s + k * 128 * CG < 1024) in[k] = *reinterpret_cast<const uint4*>(raw + (cv_off[k] & 0xffffu));
#pragma unroll
            for (int k = 0; k < kIter; ++k) {
                if (tid_s + k * 128 * CG < 1024) {
                    uint32_t o[8];
                    e4m3x4_to_f16x4(in[k].x, o[0], o[1]);
                    e4m3x4_to_f16x4(in[k].y, o[2], o[3]);
                    e4m3x4_to_f16x4(in[k].z, o[4], o[5]);
                    e4m3x4_to_f16x4(in[k].w, o[6], o[7]);
                    uint8_t* dst = slot + (cv_off[k] >> 16);
                    *reinterpret_cast<uint4*>(dst) = make_uint4(o[0], o[1], o[2], o[3]);
                    *reinterpret_cast<uint4*>(reinterpret_cast<uintptr_t>(dst) ^ 16) = make_uint4(o[4], o[5], o[6], o[7]);
                }
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(B.slot_full + 8 * s);
                mbar_arrive(B.raw_empty + 8 * r);
            }
            return true;
        };
        auto ensure_converted = [&](uint32_t g_need) -> bool {
            while (g_conv <= g_need && g_conv < g_total) {
                if (!convert_tile()) return false;
                ++g_conv;
            }
            return true;
        };
        // F8: Q of every unit up to `unit` as fp16, in place (a 16-bit element stays where it is, so the
        // swizzle does not matter); exact for magnitudes in [6.1e-5, 65504]
        auto ensure_q = [&](int unit) -> bool {
            for (; q_next <= unit && q_next < U; ++q_next) {
                const Seg s2 = get_seg(p, q_next, head_local, rank);
                if (s2.t1 <= s2.t0) continue;
                if (!mbar_wait(B.q_full, qn_s & 1, ctl, 42)) return false;
                ++qn_s;
                uint32_t* qw = reinterpret_cast<uint32_t*>(sgen + (s_q - sbase));
                for (int i = tid_s; i < q_bytes / 4; i += 128 * CG) {
                    const uint32_t w = qw[i];
                    const __half2 h = __floats2half2_rn(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
                    qw[i] = *reinterpret_cast<const uint32_t*>(&h);
                }
                fence_proxy_async();
                __syncwarp();
                if (lane == 0) mbar_arrive(B.q_ready);
            }
            return true;
        };
        constexpr float kNegBig = -1.0e30f;      // finite stand-in for -inf: keeps ex2 arguments NaN-free
        uint32_t pv_idx = 0, slot_base = 0, o_phase = 0, sync_n = 0, sfull_par = 0;
        bool ok = true;

        // O^T (d on lanes, rows on columns, hi and lo parts), rescaled from the CTA-local to the
        // global normaliser -> this CTA's partial [r][d]
        auto epilogue = [&](int unit, bool nonempty) -> bool {
            const int64_t obase = (((int64_t)(unit % kRing) * p.HG + head_local) * p.cph + rank) * R * kD;
            if (nonempty) {
                if (!mbar_wait(B.o_full, o_phase, ctl, 25)) return false;
                o_phase ^= 1;
                tc_fence_after();
                uint32_t v[NH], w[NH];
                load_cols<NH>(t_lane + col_o + c0, v);
                load_cols<NH>(t_lane + col_o + N + c0, w);
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(B.o_empty);
#pragma unroll
                for (int i = 0; i < NH; ++i) {
                    const int r = c0 + i;
                    if (r < R)
                        p.o_part[obase + (int64_t)r * kD + key_l] =
                            (F8 ? fmaf(__uint_as_float(w[i]), 1.f / kLoExp, __uint_as_float(v[i]))
                                : __uint_as_float(v[i]) + __uint_as_float(w[i])) * (SC ? fac_s[r] * vsc : fac_s[r]);
                }
            } else {
                for (int i = tid_s; i < R * kD; i += 128 * CG) p.o_part[obase + i] = 0.f;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(B.pub_o);  // the publisher warp fences and bumps the counter
            return true;
        };

        for (int unit = 0; unit < U && ok; ++unit) {
            const Seg sg = get_seg(p, unit, head_local, rank);
            const int n_t = sg.t1 - sg.t0;
            const bool nonempty = n_t > 0;
            // SC (an 8-bit cache expanded to bf16 without its scales): K's per-(layer, KV head) scale joins
            // the softmax scale, V's the output
            float cs = cs0;
            if (SC) {
                const int64_t sh = (int64_t)sg.layer * p.a.kv.n_kv_heads + sg.h;
                if (p.a.kv.k_scale) cs *= __ldg(p.a.kv.k_scale + sh);
                vsc = p.a.kv.v_scale ? __ldg(p.a.kv.v_scale + sh) : 1.f;
            }
            if (F8) {
                vsc *= 1.f / kPExp;
                ok = ensure_q(unit);
                if (!ok) break;
            }
            // ------------------------------ P1 ------------------------------
            float m[NH], l[NH];
#pragma unroll
            for (int i = 0; i < NH; ++i) {
                m[i] = kNegBig;
                l[i] = 0.f;
            }
            for (int c = 0; c < n_t && ok; ++c) {
                const int t = sg.t0 + c;
                if (F8) {
                    ok = ensure_converted(slot_base + c + f8_ahead);
                    if (!ok) break;
                }
                ok = mbar_wait(B.s_full + 8 * c, (sfull_par >> c) & 1, ctl, 20);
                if (!ok) break;
                sfull_par ^= 1u << c;
                tc_fence_after();
                uint32_t v[NH];
                load_cols<NH>(t_lane + col_s + c * N + c0, v);
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
            // reduce (m, l) over the 32 key lanes of this warp, then over the 4 warps via smem:
            // a butterfly that halves the columns a lane carries at every step (see ml_step)
            {
                int col = 0;
                ml_step<NH, NH, 16>(m, l, lane, col);
                constexpr uint32_t kDup = ml_dupmask(NH);
                constexpr int kLeft = ml_final_n(NH);
                if ((lane & kDup) == 0) {
#pragma unroll
                    for (int j = 0; j < kLeft; ++j) red[sw * NC + col + j] = make_float2(m[j], l[j]);
                }
            }
            ok = group_sync(B.sm_sync, sync_n, ctl, 26);
            if (!ok) break;
            if (sw == kSW - 1) {
                // the last softmax warp merges the four lane quarters of every column, publishes the
                // CTA's partial and leaves the CTA-local normaliser for the P V pass
                const int64_t base = (((int64_t)(unit % kRing) * p.HG + head_local) * p.cph + rank) * R;
                for (int col = lane; col < R; col += 32) {
                    const int wgi = col / NC, ci = col - wgi * NC;
                    float M = kNegBig;
#pragma unroll
                    for (int w = 0; w < 4; ++w) M = fmaxf(M, red[(wgi * 4 + w) * NC + ci].x);
                    float Ls = 0.f;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const float2 ml = red[(wgi * 4 + w) * NC + ci];
                        Ls += ml.y * ex2(ml.x - M);
                    }
                    const bool has = nonempty && M > 0.5f * kNegBig;  // the row saw at least one key here
                    p.ml_part[base + col] = make_float2(M, has ? Ls : 0.f);
                    loc_s[col] = has ? M + log2f(Ls) : 1.0e30f;       // no key: P = exp2(s - big) = 0
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(B.pub_p1);  // the publisher warp takes it from here
            }
            ok = group_sync(B.sm_sync, sync_n, ctl, 27);
            if (!ok) break;
            if (nonempty) {
                // ------------------------------ P2a: P V with the CTA-local normaliser ------------------
                // P~ = exp2(S - lse_local) needs nothing from other CTAs, so V streams and the tensor
                // cores run while the partials of the other CTAs are still on their way; the partial
                // O is rescaled by exp2(lse_local - LSE) per row in the epilogue.
                // Column-split like P1: every warpgroup works on the same tile, NC columns each, so
                // a tile's P is ready after one short pass; the score columns of the next tile are
                // fetched from tensor memory while the current ones are being turned into P.
                {
                    const float4* loc4 = reinterpret_cast<const float4*>(loc_s + c0);
                    uint32_t v[NH];
                    if (n_t > 0) {
#pragma unroll
                        for (int q = 0; q < NH; q += 8) tmem_ld8(t_lane + col_s + c0 + q, v + q);
                    }
                    for (int c = 0; c < n_t && ok; ++c) {
                        const int t = sg.t0 + c;
                        const uint32_t vslot = slot_base + n_t + c;
                        const uint32_t vs = vslot % p.n_slots, vsph = (vslot / p.n_slots) & 1;
                        const uint32_t pvi = pv_idx + c;
                        const uint32_t pb = pvi % p.p_bufs;
                        const int key = t * kTile + key_l;
                        if (F8) {  // V tile c + 2 (or the next unit's first K tiles) becomes an operand meanwhile
                            ok = ensure_converted(slot_base + n_t + c + f8_ahead);
                            if (!ok) break;
                        }
                        tc_wait_ld();
                        float pr[NH];
#pragma unroll
                        for (int i = 0; i < NH; i += 4) {
                            const float4 ls = loc4[i >> 2];
                            // F8: 2^14 P~ (the fp16 parts below then stay normal numbers down to 2^-28)
                            pr[i + 0] = ex2(fmaf(__uint_as_float(v[i + 0]), cs, F8 ? 14.f - ls.x : -ls.x));
                            pr[i + 1] = ex2(fmaf(__uint_as_float(v[i + 1]), cs, F8 ? 14.f - ls.y : -ls.y));
                            pr[i + 2] = ex2(fmaf(__uint_as_float(v[i + 2]), cs, F8 ? 14.f - ls.z : -ls.z));
                            pr[i + 3] = ex2(fmaf(__uint_as_float(v[i + 3]), cs, F8 ? 14.f - ls.w : -ls.w));
                        }
                        if (c + 1 < n_t) {  // next tile's columns: in flight during the rest of this tile
#pragma unroll
                            for (int q = 0; q < NH; q += 8) tmem_ld8(t_lane + col_s + (c + 1) * N + c0 + q, v + q);
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
                        // P~ replaces the tile's scores in tensor memory: the statistic pass then only
                        // weights it with exp2(lse_local - LSE) per row, no second exponential
#pragma unroll
                        for (int q = 0; q < NH; q += 8)
                            tmem_st8(t_lane + col_s + c * N + c0 + q, reinterpret_cast<const uint32_t*>(pr) + q);
                        // the P buffer is free once the P V product p_bufs tiles back is done ("done"
                        // barriers are indexed by the tile's sequence number mod 4)
                        if (pvi >= (uint32_t)p.p_bufs) {
                            const uint32_t prev = pvi - p.p_bufs;
                            ok = mbar_wait(B.p_empty + 8 * (prev & 3), (prev >> 2) & 1, ctl, 23);
                            if (!ok) break;
                        }
                        // [P_hi | P_lo]^T as the B operand, rows contiguous (MN-major, no swizzle): the
                        // 16-byte vector of row block j (rows 8j..8j+7 of the concatenation) and key k
                        // lives at j*2048 + (k/8)*128 + (k%8)*16
                        uint8_t* p_row = sgen + (s_p - sbase) + pb * p_bytes + (key_l >> 3) * 128 + (key_l & 7) * 16;
#pragma unroll
                        for (int nb = 0; nb < NH / 8; ++nb) {
                            uint32_t hi[4], lo[4];
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                // p = hi + lo with both parts cut to bf16 by truncation (plain integer ops, no
                                // conversion instructions): hi keeps the top 16 bits, lo the top 16 bits of the
                                // exact remainder, so p - (hi + lo) < 2^-14 p
                                const uint32_t ua = __float_as_uint(pr[nb * 8 + 2 * q]), ub = __float_as_uint(pr[nb * 8 + 2 * q + 1]);
                                if (F8) {
                                    // fp16 rounding of 2^14 P~ and the fp16 rounding of 2^11 times what it left over
                                    const __half2 h = __floats2half2_rn(__uint_as_float(ua), __uint_as_float(ub));
                                    const float2 hf = __half22float2(h);
                                    const __half2 l = __floats2half2_rn((__uint_as_float(ua) - hf.x) * kLoExp,
                                                                        (__uint_as_float(ub) - hf.y) * kLoExp);
                                    hi[q] = *reinterpret_cast<const uint32_t*>(&h);
                                    lo[q] = *reinterpret_cast<const uint32_t*>(&l);
                                    continue;
                                }
                                hi[q] = __byte_perm(ua, ub, 0x7632);
                                const float ra = __uint_as_float(ua) - __uint_as_float(ua & 0xffff0000u);
                                const float rb = __uint_as_float(ub) - __uint_as_float(ub & 0xffff0000u);
                                lo[q] = __byte_perm(__float_as_uint(ra), __float_as_uint(rb), 0x7632);
                            }
                            const int jh = wg * (NH / 8) + nb, jl = jh + N / 8;
                            *reinterpret_cast<uint4*>(p_row + jh * 2048) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
                            *reinterpret_cast<uint4*>(p_row + jl * 2048) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
                        }
                        if (t * kTile + kTile > sg.T) {
                            // ragged last tile: V rows at or beyond T may hold anything; zero them in
                            // shared memory so that 0 * garbage never reaches the accumulator
                            ok = mbar_wait(B.slot_full + 8 * vs, vsph, ctl, 24);
                            if (!ok) break;
                            if (key >= sg.T && wg < 2) {  // warpgroups 0 and 1 clear one 64-wide half each
                                uint8_t* vrow = sgen + (s_slots - sbase) + vs * kSlotBytes + wg * 16384 + key_l * 128;
#pragma unroll
                                for (int ch = 0; ch < 8; ++ch) *reinterpret_cast<uint4*>(vrow + 16 * ch) = make_uint4(0, 0, 0, 0);
                            }
                        }
                        fence_proxy_async();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(B.p_full + 8 * pb);
                    }
                }
                if (!ok) break;
                tc_wait_st();
                tc_fence_before();
                pv_idx += n_t;
                slot_base += 2 * n_t;
                // ---- the row LSE and the rescale factors, combined by the publisher warp meanwhile ----
                ok = mbar_wait(B.lse_ready, unit & 1, ctl, 31);
                if (!ok) break;
                if (!LP) {  // many CTAs per head: too many partials for one warp, all softmax threads fold them
                    if (lane == 0) ok = counter_wait(p.counters + unit * p.HG + head_local, p.cph, ctl, 33);
                    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;  // lane 0's acquire, then warp-wide
                    if (!ok) break;
                    const float2* src = p.ml_part + ((int64_t)(unit % kRing) * p.HG + head_local) * p.cph * R;
                    // tpr threads of one warp share a row: each folds every tpr-th partial, then shuffles
                    int tpr = 32;
                    while (tpr * R > 128 * CG) tpr >>= 1;
                    const int r = tid_s / tpr, sub = tid_s - r * tpr;
                    float M = kNegBig, Ls = 0.f;
                    if (r < R) {
                        for (int k0 = sub; k0 < p.cph; k0 += 8 * tpr) {  // batches of 8 independent loads
                            float2 x[8];
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                x[u] = (k0 + u * tpr < p.cph) ? __ldcg(src + (int64_t)(k0 + u * tpr) * R + r)
                                                              : make_float2(kNegBig, 0.f);
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const float Mn = fmaxf(M, x[u].x);
                                Ls = Ls * ex2(M - Mn) + x[u].y * ex2(x[u].x - Mn);
                                M = Mn;
                            }
                        }
                    }
                    for (int o = tpr >> 1; o > 0; o >>= 1) {
                        const float M2 = __shfl_xor_sync(0xffffffffu, M, o);
                        const float L2 = __shfl_xor_sync(0xffffffffu, Ls, o);
                        const float Mn = fmaxf(M, M2);
                        Ls = Ls * ex2(M - Mn) + L2 * ex2(M2 - Mn);
                        M = Mn;
                    }
                    if (sub == 0 && r < R) {
                        const float lse2 = M + log2f(Ls);
                        lse_s[r] = lse2;
                        const float loc = loc_s[r];
                        fac_s[r] = loc < 1.0e29f ? ex2(loc - lse2) : 0.f;  // local -> global normaliser
                        if (rank == p.cph - 1 && p.a.lse) {  // the last rank always owns at least one tile
                            const int j = r / G, g = r - j * G;
                            const int64_t row = (((int64_t)sg.layer * p.a.kv.batch + sg.b) * p.a.n_q + j) * p.a.kv.n_q_heads + sg.h * G + g;
                            p.a.lse[row] = lse2 * 0.69314718055994530942f;
                        }
                    }
                }
                if (F8) {  // the next unit's Q has landed by now: its K Q^T can start as the statistic pass frees regions
                    ok = ensure_q(unit + 1);
                    if (!ok) break;
                }
                ok = group_sync(B.sm_sync, sync_n, ctl, 22);  // every warp is done with the P V pass
                if (!ok) break;
                tc_fence_after();  // the P~ stores of the other warps, ordered by the barrier
                // ------------------------------ P2b: the Eq. 3 statistic ------------------------------
                // second visit of the cached tiles, which hold P~ = exp2(S - lse_local) by now (masked
                // entries are 0): weighted with exp2(lse_local - LSE) per row they are the exactly
                // normalised probabilities, whose column sums are the statistic.  No exponential, no
                // shared memory, no tensor cores; the tile's TMEM region is released afterwards.
                for (int c = wg; c < n_t; c += CG) {
                    const int t = sg.t0 + c;
                    const int key = t * kTile + key_l;
                    float st = 0.f;
                    float sth[PH ? 8 : 1];  // PH: column i belongs to head i mod G, and G divides 8
#pragma unroll
                    for (int i = 0; i < (PH ? 8 : 1); ++i) sth[i] = 0.f;
#pragma unroll 1
                    for (int cb = 0; cb < N; cb += 16) {
                        if (cb + 16 <= stat_r0) continue;  // rows outside the statistic window
                        uint32_t v[16];
                        tmem_ld8(t_lane + col_s + c * N + cb, v);
                        tmem_ld8(t_lane + col_s + c * N + cb + 8, v + 8);
                        tc_wait_ld();
                        const float4* fac4 = reinterpret_cast<const float4*>(fac_s + cb);
                        float pr[16];
#pragma unroll
                        for (int i = 0; i < 16; i += 4) {
                            const float4 f = fac4[i >> 2];
                            pr[i + 0] = __uint_as_float(v[i + 0]) * f.x;
                            pr[i + 1] = __uint_as_float(v[i + 1]) * f.y;
                            pr[i + 2] = __uint_as_float(v[i + 2]) * f.z;
                            pr[i + 3] = __uint_as_float(v[i + 3]) * f.w;
                        }
                        if (PH && ph_fast) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) sth[i & 7] += (cb + i >= stat_r0) ? pr[i] : 0.f;
                        } else if (PH) {
                            // any group size up to 8: accumulator g takes the columns r with r mod G == g
                            int g = cb % G;
#pragma unroll
                            for (int i = 0; i < 16; ++i) {
                                const float val = (cb + i >= stat_r0) ? pr[i] : 0.f;
#pragma unroll
                                for (int t = 0; t < 8; ++t) sth[t] += (g == t) ? val : 0.f;
                                g = (g + 1 == G) ? 0 : g + 1;
                            }
                        } else if (cb >= stat_r0) {
#pragma unroll
                            for (int i = 0; i < 16; ++i) st += pr[i];
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) st += (cb + i >= stat_r0) ? pr[i] : 0.f;
                        }
                    }
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(B.s_free + 8 * c);
                    if (PH) {
                        // fast path: fold the eight residues mod 8 down to the G residues mod G
                        if (ph_fast && G <= 4) {
#pragma unroll
                            for (int i = 0; i < 4; ++i) sth[i] += sth[i + 4];
                        }
                        if (ph_fast && G <= 2) {
                            sth[0] += sth[2];
                            sth[1] += sth[3];
                        }
                        if (ph_fast && G == 1) sth[0] += sth[1];
                        if (key < sg.T && p.a.stat_group_max) {
                            // one score per KV head: the largest of the group's per-head scores
                            float best = sth[0];
#pragma unroll
                            for (int g = 1; g < 8; ++g)
                                if (g < G) best = fmaxf(best, sth[g]);
                            float* dst = p.a.stats + sg.prob * p.a.stat_stride + key;
                            const float val = p.a.stat_accumulate ? *dst + best : best;
                            *dst = val;
                            if (p.a.hist) atomicAdd(p.a.hist + sg.prob * kScoreBins + (__float_as_uint(val) >> 21), 1u);
                        } else if (key < sg.T) {
#pragma unroll
                            for (int g = 0; g < 8; ++g) {
                                if (g < G) {
                                    float* dst = p.a.stats + (sg.prob * G + g) * p.a.stat_stride + key;
                                    const float val = p.a.stat_accumulate ? *dst + sth[g] : sth[g];
                                    *dst = val;
                                    if (p.a.hist) atomicAdd(p.a.hist + (sg.prob * G + g) * kScoreBins + (__float_as_uint(val) >> 21), 1u);
                                }
                            }
                        }
                    } else if (key < sg.T) {
                        float* dst = p.a.stats + sg.prob * p.a.stat_stride + key;
                        if (F8) st *= 1.f / kPExp;  // the cache holds 2^14 P~
                        const float val = p.a.stat_accumulate ? *dst + st : st;
                        *dst = val;
                        // first radix pass of the selection, fused: count the score's top 11 bits in this
                        // CTA's shared-memory histogram (two 16-bit counters per word: a CTA holds at most
                        // 4096 keys of a head)
                        if (p.a.hist) {
                            const uint32_t bin = __float_as_uint(val) >> 21;
                            atomicAdd(hist_s + (bin >> 1), 1u << ((bin & 1u) * 16));
                        }
                    }
                }
                if (!PH && p.a.hist) {
                    // the CTA's counts of this head join the global ones: one reduction per bin that is not
                    // empty (a few dozen), and the shared-memory copy is clear again for the next unit
                    ok = group_sync(B.sm_sync, sync_n, ctl, 28);
                    if (!ok) break;
                    uint32_t* hg = p.a.hist + sg.prob * kScoreBins;
                    for (int w = tid_s; w < kScoreBins / 2; w += 128 * CG) {
                        const uint32_t v = hist_s[w];
                        if (v) {
                            hist_s[w] = 0u;
                            if (v & 0xffffu) atomicAdd(hg + 2 * w, v & 0xffffu);
                            if (v >> 16) atomicAdd(hg + 2 * w + 1, v >> 16);
                        }
                    }
                }
            }
            else {
                ok = mbar_wait(B.lse_ready, unit & 1, ctl, 32);  // keeps step with the publisher warp (see there)
                if (!ok) break;
            }
            // ---- this unit's accumulator: rescale and hand to the reducers ----
            ok = epilogue(unit, nonempty);
            if (!ok) break;
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

template <int NC, int CG, bool LP, bool PH, bool SC, bool F8>
int launch_cfg(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const FastParams& fp,
               int grid, size_t smem_bytes, cudaStream_t stream)
{
    auto kern = verify_cached_kernel<NC, CG, LP, PH, SC, F8>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_bytes) != cudaSuccess)
        return SPEC_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(128 + 128 * CG);
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    // All CTAs must become co-resident (they wait on each other's partials).  The grid never exceeds
    // the SM count at one CTA per SM, so that follows as soon as the previous kernel's CTAs have left:
    // the launch only asks for programmatic stream serialisation, which lets each CTA take an SM the
    // moment the previous layer's CTA on it exits (a cooperative launch would wait for the whole
    // previous grid first: 1.4 us per layer).  A CTA whose peers cannot become resident (SMs held by
    // an unrelated long kernel) ends in SPEC_ERR_TIMEOUT like any other stall.  If the driver refuses
    // the attribute the launch falls back to a cooperative one.
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see griddepcontrol in the kernel
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    static bool pdl_refused[64] = {};  // per device: a driver that refuses the attribute is asked only once
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
    const bool pdl_ok = !pdl_refused[dev];
    cudaError_t err = pdl_ok ? cudaLaunchKernelEx(&cfg, kern, tk, tv, tq, fp) : cudaErrorNotSupported;
    if (err != cudaSuccess) {
        if (pdl_ok) cudaGetLastError();
        pdl_refused[dev] = true;
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        err = cudaLaunchKernelEx(&cfg, kern, tk, tv, tq, fp);
    }
    if (err != cudaSuccess) {
        cudaGetLastError();
        return SPEC_ERR_CUDA;
    }
    count_launch(1);
    return SPEC_OK;
}

}  // namespace

int launch_cached(const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tq, const FastParams& fp,
                  int grid, size_t smem_bytes, cudaStream_t stream)
{
    const bool lp = fp.cph <= kLsePubMax, ph = fp.a.stat_per_head != 0 || fp.a.stat_group_max != 0;
    // per-(layer, KV head) scales: instances of their own (the bf16 instances carry no code for them),
    // built for the per-KV-head statistic only
    const bool sc = fp.a.kv.k_scale != nullptr || fp.a.kv.v_scale != nullptr;
    const bool f8 = fp.a.kv.fp8 != 0;  // 8-bit cache read directly (always an SC instance)
    if ((sc || f8) && ph) return SPEC_ERR_UNSUPPORTED_SHAPE;
#define SPEC_CASE(n, nc, cg)                                                                                            \
    case n:                                                                                                             \
        if (f8) return lp ? launch_cfg<nc, cg, true, false, true, true>(tk, tv, tq, fp, grid, smem_bytes, stream)       \
                          : launch_cfg<nc, cg, false, false, true, true>(tk, tv, tq, fp, grid, smem_bytes, stream);     \
        if (sc) return lp ? launch_cfg<nc, cg, true, false, true, false>(tk, tv, tq, fp, grid, smem_bytes, stream)      \
                          : launch_cfg<nc, cg, false, false, true, false>(tk, tv, tq, fp, grid, smem_bytes, stream);    \
        if (ph) return lp ? launch_cfg<nc, cg, true, true, false, false>(tk, tv, tq, fp, grid, smem_bytes, stream)      \
                          : launch_cfg<nc, cg, false, true, false, false>(tk, tv, tq, fp, grid, smem_bytes, stream);    \
        return lp ? launch_cfg<nc, cg, true, false, false, false>(tk, tv, tq, fp, grid, smem_bytes, stream)             \
                  : launch_cfg<nc, cg, false, false, false, false>(tk, tv, tq, fp, grid, smem_bytes, stream);
    switch (fp.N) {  // (columns per warpgroup, warpgroups)
        SPEC_CASE(16, 8, 2)
        SPEC_CASE(32, 8, 4)
        SPEC_CASE(48, 16, 3)
        SPEC_CASE(64, 16, 4)
        SPEC_CASE(80, 40, 2)
        SPEC_CASE(96, 24, 4)
        SPEC_CASE(112, 56, 2)
        SPEC_CASE(128, 32, 4)
        default: return SPEC_ERR_UNSUPPORTED_SHAPE;
    }
#undef SPEC_CASE
}

}  // namespace sm100
}  // namespace spec
