// Sparse draft attention of Eq. 5, streaming variant: every warp walks its own 16-key chunks of
// the recalled rows through a private ring of shared-memory stages, so that the gather (16-byte
// cp.async copies straight from the dense cache by index) of the chunks ahead runs under the
// tensor-core work of the current one, and no block-wide barrier sits in the loop.  Several
// small CTAs share an SM, which keeps gathers in flight on every SM for the whole call.
//
// Per chunk (16 keys x head_dim), in registers, with the G <= 8 query heads of the group packed
// into the M dimension of mma.sync m16n8k16:
//   S = Q K^T      A = Q (rows 0..7 = heads, rows 8..15 zero), B = K rows as they lie in memory;
//   online softmax per head (running max with a lazy rescale, running sum);
//   O += P V       A = [P_hi ; P_lo] (rows 0..7 the bf16 rounding of P, rows 8..15 its remainder:
//                  the second half of the M dimension is free, so the split costs no extra MMA),
//                  B = V rows through ldmatrix.trans.
// The warps of a CTA merge their (max, sum, O) through shared memory, the CTAs of a cluster
// (one cluster per (layer, sequence, KV head)) deposit theirs in the cluster's first CTA with
// asynchronous distributed-shared-memory stores counted on an mbarrier; it merges them in rank
// order, so the result is deterministic.  One launch per call, no global scratch.
#include "spec_common.cuh"
#include <type_traits>
#include "draft_common.cuh"

namespace spec {

namespace {

using namespace draft;

constexpr int kChunk = 16;
constexpr uint32_t kNoRow = 0xffffffffu;

template <int D, bool F8>
struct Geo {
    static constexpr int ES = F8 ? 1 : 2;            // bytes per cache element (e4m3 or bf16)
    static constexpr int ROWB = D * ES + 16;         // bytes per shared-memory row: 16 B of padding spread the banks
    static constexpr int STAGE = 2 * kChunk * ROWB;  // a chunk's K rows, then its V rows
};

// Shared memory of one CTA: [NW warps][ST stages][STAGE] | row offsets uint32 [per] |
// per-warp (max, sum) float2 [NW][8] | deposit barrier (16 B) | deposit area float [cs][G * (D + 2)]
template <int D, bool F8>
__host__ __device__ inline size_t stream_smem_bytes(int G, int nw, int st, int per, int cs)
{
    return (size_t)nw * st * Geo<D, F8>::STAGE + (size_t)per * 4 + (size_t)nw * 8 * 8 + 16 + (size_t)cs * G * (D + 2) * 4;
}

__device__ __forceinline__ void mma_f16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// two e4m3 bytes (the low 16 bits of `two`) as a packed fp16 pair: exact
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two)
{
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)(two & 0xffffu), __NV_E4M3);
    return (uint32_t)h.x | ((uint32_t)h.y << 16);
}
__device__ __forceinline__ uint32_t pack_f16(float x, float y)
{
    const __half2 v = __floats2half2_rn(x, y);
    return *reinterpret_cast<const uint32_t*>(&v);
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};\n"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// transpose of an 8x8 matrix of 16-bit elements held across the warp (thread (grp, quad) holds row grp,
// columns 2 quad and 2 quad + 1, before and after)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

// F8: the cache holds e4m3 bytes.  The rows are gathered as they are (half the bytes), turned into fp16
// pairs on their way into the MMA fragments (fp16 holds every e4m3 value), and the two products run as
// fp16 MMAs; the heads' scales join the softmax scale (K) and the final output (V).
template <int D, int NW, int ST, bool F8>
__global__ void __launch_bounds__(NW * 32)
draft_stream_kernel(DraftArgs a, StreamShape shp, int* __restrict__ status)
{
    constexpr int ROWB = Geo<D, F8>::ROWB, STAGE = Geo<D, F8>::STAGE, ES = Geo<D, F8>::ES;
    constexpr int NT = NW * 32;
    constexpr int KS = D / 16;  // 16-wide steps of the head dimension
    constexpr float kLog2e = 1.4426950408889634f;
    extern __shared__ __align__(16) uint8_t smem[];
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const int per = shp.per, PS = G * (D + 2);
    uint8_t* stages = smem;
    uint32_t* rowoff = reinterpret_cast<uint32_t*>(smem + (size_t)NW * ST * STAGE);
    float2* wml = reinterpret_cast<float2*>(rowoff + per);        // [NW][8]
    uint64_t* dep_bar = reinterpret_cast<uint64_t*>(wml + NW * 8);
    float* comb = reinterpret_cast<float*>(dep_bar + 2);          // [cs][PS]: O rows [G][D], then (maximum, sum) per head

    const int CS = gridDim.x, rank = blockIdx.x, h = blockIdx.y;
    const int layer = blockIdx.z / a.kv.batch, b = blockIdx.z % a.kv.batch;
    const int64_t prob = (int64_t)blockIdx.z * a.kv.n_kv_heads + h;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grp = lane >> 2, quad = lane & 3;

    // The next kernel of the stream may start while this one runs (programmatic dependent launch).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (CS > 1) {
        if (rank == 0 && tid == 0) {
            mbar_init(smem_addr(dep_bar), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            mbar_arrive_expect_tx(smem_addr(dep_bar), (uint32_t)(CS - 1) * PS * 4);
        }
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }
    // Without the early-gather promise the launch is an ordinary one: all earlier work is complete.
    bool waited = !a.early_gather;

    const int n_rec = min(max(__ldg(a.n_indices + prob), 0), a.k_total);
    const int ts = __ldg(a.tail_start + b);
    int cl = __ldg(a.cur_len + b);
    const int64_t cap = (int64_t)a.kv.max_pages * a.kv.page_size;
    if (cl > cap) {  // a length beyond the cache: clamp, so that no row address leaves it
        if (tid == 0) set_status(status, SPEC_ERR_BAD_INDEX);
        cl = (int)cap;
    }
    int n_tail = max(cl - ts, 0);
    if (n_tail > a.max_tail) {  // the launch was sized for max_tail rows: the rest is dropped, and reported
        if (tid == 0) set_status(status, SPEC_ERR_BAD_INDEX);
        n_tail = a.max_tail;
    }
    const int n = n_rec + n_tail;
    const int k0 = min(n, rank * per), k1 = min(n, k0 + per);
    const int nch = (k1 - k0 + kChunk - 1) / kChunk;
    const int first_tail = max(n_rec, k0) - k0;  // local rows [first_tail, k1 - k0) come from the dense tail

    // ---- resolve the rows of this CTA's share once: position -> offset of the row in 16-byte units ----
    const int hm = a.head_div > 1 ? h / a.head_div : h;  // the cache head this problem's rows come from
    {
        const int32_t* idx = a.indices + prob * a.k_total;
        const int32_t* ptab = a.kv.page_table ? a.kv.page_table + (int64_t)b * a.kv.max_pages : nullptr;
        for (int lr = tid; lr < nch * kChunk; lr += NT) {
            uint32_t off = kNoRow;
            if (k0 + lr < k1) {
                const int li = k0 + lr;
                const int pos = li < n_rec ? __ldg(idx + li) : ts + (li - n_rec);
                if (pos < 0 || pos >= cl) {
                    set_status(status, SPEC_ERR_BAD_INDEX);
                } else {
                    const int page = page_of(a.kv, pos);
                    const int slot_in = pos - page * a.kv.page_size;
                    const int64_t phys = ptab ? (int64_t)__ldg(ptab + page) : (int64_t)b * a.kv.max_pages + page;
                    if (phys < 0 || phys >= a.kv.n_pages) set_status(status, SPEC_ERR_BAD_INDEX);
                    else off = (uint32_t)((phys * a.kv.page_stride + (int64_t)slot_in * a.kv.slot_stride) >> (F8 ? 4 : 3));
                }
            }
            rowoff[lr] = off;
        }
    }
    __syncthreads();

    // ---- per-warp pipeline over the chunks warp, warp + NW, ... of the share ----
    // one instruction copies 16-byte pieces of 32 / (2 * PIECES) rows: the K pieces and the V pieces of each
    constexpr int PIECES = D * ES / 16, RPI = 32 / (2 * PIECES);
    const int piece = lane % PIECES, is_v = (lane / PIECES) & 1, rsub = lane / (2 * PIECES);
    const uint8_t* gbase = (F8 ? (is_v ? a.kv.v8 : a.kv.k8)
                               : reinterpret_cast<const uint8_t*>(is_v ? a.kv.v : a.kv.k)) +
                           (layer * a.kv.layer_stride + hm * a.kv.head_stride) * ES + piece * 16;
    uint8_t* wst = stages + (size_t)warp * ST * STAGE;
    const uint32_t dst_lane = (is_v ? kChunk * ROWB : 0) + rsub * ROWB + piece * 16;

    auto issue = [&](int c, int stage) {  // gather chunk c (local index) into a stage; always one commit group
        if (c < nch) {
            if (!waited && c * kChunk + kChunk > first_tail && first_tail < k1 - k0) {
                asm volatile("griddepcontrol.wait;" ::: "memory");  // rows of the dense tail are written by the stream
                waited = true;
            }
            const uint32_t mine = rowoff[c * kChunk + (lane & 15)];
            uint8_t* dst = wst + stage * STAGE + dst_lane;
#pragma unroll
            for (int r = 0; r < kChunk; r += RPI) {
                const uint32_t o = __shfl_sync(0xffffffffu, mine, r + rsub);
                cp_async16(dst + r * ROWB, gbase + ((int64_t)(o == kNoRow ? 0u : o) << 4), o == kNoRow ? 0u : 16u);
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < ST; ++s) issue(warp + s * NW, s);

    if (!waited && tid < G)  // Q is written by an earlier kernel of the stream: ask L2 for its lines meanwhile
        prefetch_l2(a.q + (((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + tid) * D, D * 2);
    if (!waited) {
        asm volatile("griddepcontrol.wait;" ::: "memory");  // Q is written by the stream
        waited = true;
    }
    // A fragments of Q (heads x d): the thread holds head grp at d = 16 ks + 2 quad + {0, 1} and + {8, 9}.
    // F8: the K fragment of a step comes from ONE 4-byte load (d = 16 ks + 4 quad + 0..3), so the step's
    // sixteen d's are visited in that order and Q follows it: d = 16 ks + 4 quad + {0, 1} and + {2, 3},
    // as fp16.
    // keys_on_rows (see below): Q is the B operand and its eight columns are the heads 0, 0, 1, 1, 2, 2, 3, 3
    const bool keys_on_rows = G <= 4;
    const int qh = keys_on_rows ? grp >> 1 : grp;  // the head whose row this thread's fragments come from
    uint32_t qa[KS][2];
    {
        const int64_t row = ((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + qh;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(a.q + row * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            if (F8) {
                const uint32_t w0 = qh < G ? __ldg(qrow + ks * 8 + 2 * quad) : 0u;
                const uint32_t w1 = qh < G ? __ldg(qrow + ks * 8 + 2 * quad + 1) : 0u;
                qa[ks][0] = pack_f16(bf16_lo(w0), bf16_hi(w0));
                qa[ks][1] = pack_f16(bf16_lo(w1), bf16_hi(w1));
            } else {
                qa[ks][0] = qh < G ? __ldg(qrow + ks * 8 + quad) : 0u;
                qa[ks][1] = qh < G ? __ldg(qrow + ks * 8 + 4 + quad) : 0u;
            }
        }
    }

    const float sc = a.kv.scale * kLog2e * (F8 ? kv_scale_of(a.kv.k_scale, a.kv, layer, hm) : 1.f);
    float M = kNegBig, L = 0.f;
    float o[D / 8][4];
#pragma unroll
    for (int i = 0; i < D / 8; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

    // S = Q K^T of the chunk in a stage: keys 0..7 and 8..15 are the two 8-wide column blocks
    auto qk = [&](const uint8_t* ksm, float (&s0)[4], float (&s1)[4]) {
        {
            float t0[4] = {0.f, 0.f, 0.f, 0.f}, t1[4] = {0.f, 0.f, 0.f, 0.f};  // four accumulation chains
            if (F8) {
                // key grp (and grp + 8), bytes 16 ks + 4 quad .. + 3: one load per key block and step
                const uint8_t* kp = ksm + grp * ROWB + 4 * quad;
#pragma unroll
                for (int ks = 0; ks < KS; ks += 2) {
                    const uint32_t k00 = *reinterpret_cast<const uint32_t*>(kp + ks * 16);
                    const uint32_t k01 = *reinterpret_cast<const uint32_t*>(kp + 8 * ROWB + ks * 16);
                    const uint32_t k10 = *reinterpret_cast<const uint32_t*>(kp + ks * 16 + 16);
                    const uint32_t k11 = *reinterpret_cast<const uint32_t*>(kp + 8 * ROWB + ks * 16 + 16);
                    mma_f16_16816(s0, qa[ks][0], 0u, qa[ks][1], 0u, e4m3x2_to_f16x2(k00), e4m3x2_to_f16x2(k00 >> 16));
                    mma_f16_16816(s1, qa[ks][0], 0u, qa[ks][1], 0u, e4m3x2_to_f16x2(k01), e4m3x2_to_f16x2(k01 >> 16));
                    mma_f16_16816(t0, qa[ks + 1][0], 0u, qa[ks + 1][1], 0u, e4m3x2_to_f16x2(k10), e4m3x2_to_f16x2(k10 >> 16));
                    mma_f16_16816(t1, qa[ks + 1][0], 0u, qa[ks + 1][1], 0u, e4m3x2_to_f16x2(k11), e4m3x2_to_f16x2(k11 >> 16));
                }
            } else {
                const uint8_t* kp = ksm + ((lane & 7) + ((lane >> 4) & 1) * 8) * ROWB + ((lane >> 3) & 1) * 16;
#pragma unroll
                for (int ks = 0; ks < KS; ks += 2) {
                    uint32_t kf[4], kg[4];
                    ldmatrix_x4(kf, kp + ks * 32);
                    ldmatrix_x4(kg, kp + ks * 32 + 32);
                    mma_bf16_16816(s0, qa[ks][0], 0u, qa[ks][1], 0u, kf[0], kf[1]);
                    mma_bf16_16816(s1, qa[ks][0], 0u, qa[ks][1], 0u, kf[2], kf[3]);
                    mma_bf16_16816(t0, qa[ks + 1][0], 0u, qa[ks + 1][1], 0u, kg[0], kg[1]);
                    mma_bf16_16816(t1, qa[ks + 1][0], 0u, qa[ks + 1][1], 0u, kg[2], kg[3]);
                }
            }
            s0[0] += t0[0];
            s0[1] += t0[1];
            s1[0] += t1[0];
            s1[1] += t1[1];
        }
    };
    // the chunk's four scores of this thread (keys 2 quad, 2 quad + 1, 8 + 2 quad, 9 + 2 quad), scaled; masked rows carry no offset
    auto scores = [&](int c, const float (&s0)[4], const float (&s1)[4], float (&sv)[4]) {
        const uint2 va = *reinterpret_cast<const uint2*>(rowoff + c * kChunk + 2 * quad);
        const uint2 vb = *reinterpret_cast<const uint2*>(rowoff + c * kChunk + 8 + 2 * quad);
        sv[0] = va.x != kNoRow ? s0[0] * sc : kNegBig;
        sv[1] = va.y != kNoRow ? s0[1] * sc : kNegBig;
        sv[2] = vb.x != kNoRow ? s1[0] * sc : kNegBig;
        sv[3] = vb.y != kNoRow ? s1[1] * sc : kNegBig;
    };
    // O += [P_hi ; P_lo] V of the chunk in a stage, p = the thread's four probabilities
    auto pv = [&](const uint8_t* vsm, const float (&p)[4]) {
        // [P_hi ; P_lo] as the A operand: rows 0..7 the 16-bit rounding, rows 8..15 the remainder
        uint32_t ah0, al0, ah1, al1;
        if (F8) {
            const __half2 h01 = __floats2half2_rn(p[0], p[1]), h23 = __floats2half2_rn(p[2], p[3]);
            ah0 = *reinterpret_cast<const uint32_t*>(&h01);
            ah1 = *reinterpret_cast<const uint32_t*>(&h23);
            al0 = pack_f16(p[0] - __low2float(h01), p[1] - __high2float(h01));
            al1 = pack_f16(p[2] - __low2float(h23), p[3] - __high2float(h23));
        } else {
            const __nv_bfloat162 h01 = __floats2bfloat162_rn(p[0], p[1]), h23 = __floats2bfloat162_rn(p[2], p[3]);
            ah0 = *reinterpret_cast<const uint32_t*>(&h01);
            ah1 = *reinterpret_cast<const uint32_t*>(&h23);
            al0 = pack_bf16(p[0] - __low2float(h01), p[1] - __high2float(h01));
            al1 = pack_bf16(p[2] - __low2float(h23), p[3] - __high2float(h23));
        }
        // ---- O += [P_hi ; P_lo] V ----
        if (F8) {
            // A transposing 8x8 load works on 2-byte units, so a thread gets, for keys 2 quad and 2 quad + 1,
            // the byte PAIR d = 2 grp, 2 grp + 1 (of a 16-byte column block): bytes 0 and 2 of the register are
            // the B fragment of the even d, bytes 1 and 3 of the odd d.  Four column blocks of 8 come out
            // of one x4 load (32 bytes of every row); the accumulators therefore hold the head dimension in
            // the order d = 32 j + 16 (t / 2) + 4 quad + (t % 2) + {0, 2} for block 4 j + t (see the store).
            const uint8_t* vp = vsm + ((lane & 7) + ((lane >> 3) & 1) * 8) * ROWB + ((lane >> 4) & 1) * 16;
#pragma unroll
            for (int j = 0; j < D / 32; ++j) {
                uint32_t vf[4];
                ldmatrix_x4_trans(vf, vp + j * 32);
                mma_f16_16816(o[4 * j + 0], ah0, al0, ah1, al1, e4m3x2_to_f16x2(__byte_perm(vf[0], 0u, 0x4420)),
                              e4m3x2_to_f16x2(__byte_perm(vf[1], 0u, 0x4420)));
                mma_f16_16816(o[4 * j + 1], ah0, al0, ah1, al1, e4m3x2_to_f16x2(__byte_perm(vf[0], 0u, 0x4431)),
                              e4m3x2_to_f16x2(__byte_perm(vf[1], 0u, 0x4431)));
                mma_f16_16816(o[4 * j + 2], ah0, al0, ah1, al1, e4m3x2_to_f16x2(__byte_perm(vf[2], 0u, 0x4420)),
                              e4m3x2_to_f16x2(__byte_perm(vf[3], 0u, 0x4420)));
                mma_f16_16816(o[4 * j + 3], ah0, al0, ah1, al1, e4m3x2_to_f16x2(__byte_perm(vf[2], 0u, 0x4431)),
                              e4m3x2_to_f16x2(__byte_perm(vf[3], 0u, 0x4431)));
            }
        } else {
            const uint8_t* vp = vsm + ((lane & 7) + ((lane >> 3) & 1) * 8) * ROWB + ((lane >> 4) & 1) * 16;
#pragma unroll
            for (int nb = 0; nb < KS; ++nb) {
                uint32_t vf[4];
                ldmatrix_x4_trans(vf, vp + nb * 32);
                mma_bf16_16816(o[2 * nb], ah0, al0, ah1, al1, vf[0], vf[1]);
                mma_bf16_16816(o[2 * nb + 1], ah0, al0, ah1, al1, vf[2], vf[3]);
            }
        }
    };

    if (keys_on_rows) {
        // Groups of at most four heads: the keys take the MMA's 16 rows instead of the heads.
        // S^T = K Q^T is ONE m16n8k16 per 16 d (Q's fragments are the same registers as in the head-major form,
        // now the B operand, with every head in two neighbouring columns), and O^T = V^T P^T one per 16 d as
        // well, the column pair of a head being the bf16 rounding of its probabilities and the remainder.
        // Thread (grp, quad) then owns head `quad` throughout: the scores of keys grp and grp + 8, its maximum
        // and sum, and O^T for d = 16 j + grp and + 8.  Half the tensor-core instructions of the head-major
        // form below, whose 16 rows are mostly padding.
        float ot[D / 16][4];  // O^T: rows d = 16 j + grp (and + 8), columns (rounding, remainder) of head quad
#pragma unroll
        for (int j = 0; j < D / 16; ++j) ot[j][0] = ot[j][1] = ot[j][2] = ot[j][3] = 0.f;
        // scores of keys grp, grp + 8 of the chunk in a stage (both columns of the pair hold the same number)
        auto tr_qk = [&](const uint8_t* ksm, float (&st)[2]) {
            float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};  // two accumulation chains
            if (F8) {
                // rows grp and grp + 8, bytes 16 ks + 4 quad .. + 3: one 4-byte load per row and step gives the
                // row's two fragment registers (the step's sixteen d's are visited in that order, as Q's are)
                const uint8_t* kp = ksm + grp * ROWB + 4 * quad;
#pragma unroll
                for (int ks = 0; ks < KS; ks += 2) {
                    const uint32_t k00 = *reinterpret_cast<const uint32_t*>(kp + ks * 16);
                    const uint32_t k01 = *reinterpret_cast<const uint32_t*>(kp + 8 * ROWB + ks * 16);
                    const uint32_t k10 = *reinterpret_cast<const uint32_t*>(kp + ks * 16 + 16);
                    const uint32_t k11 = *reinterpret_cast<const uint32_t*>(kp + 8 * ROWB + ks * 16 + 16);
                    mma_f16_16816(c0, e4m3x2_to_f16x2(k00), e4m3x2_to_f16x2(k01), e4m3x2_to_f16x2(k00 >> 16),
                                  e4m3x2_to_f16x2(k01 >> 16), qa[ks][0], qa[ks][1]);
                    mma_f16_16816(c1, e4m3x2_to_f16x2(k10), e4m3x2_to_f16x2(k11), e4m3x2_to_f16x2(k10 >> 16),
                                  e4m3x2_to_f16x2(k11 >> 16), qa[ks + 1][0], qa[ks + 1][1]);
                }
            } else {
                const uint8_t* kp = ksm + ((lane & 7) + ((lane >> 3) & 1) * 8) * ROWB + (lane >> 4) * 16;
#pragma unroll
                for (int ks = 0; ks < KS; ks += 2) {
                    uint32_t ka[4], kb[4];
                    ldmatrix_x4(ka, kp + ks * 32);
                    ldmatrix_x4(kb, kp + ks * 32 + 32);
                    mma_bf16_16816(c0, ka[0], ka[1], ka[2], ka[3], qa[ks][0], qa[ks][1]);
                    mma_bf16_16816(c1, kb[0], kb[1], kb[2], kb[3], qa[ks + 1][0], qa[ks + 1][1]);
                }
            }
            st[0] = c0[0] + c1[0];
            st[1] = c0[2] + c1[2];
        };
        // scaled, masked (a key without a row counts for nothing)
        auto tr_mask = [&](int c, float (&st)[2]) {
            st[0] = rowoff[c * kChunk + grp] != kNoRow ? st[0] * sc : kNegBig;
            st[1] = rowoff[c * kChunk + 8 + grp] != kNoRow ? st[1] * sc : kNegBig;
        };
        auto tr_pv = [&](const uint8_t* vsm, float p0, float p1) {
            // source of P^T: rows = keys (0..7 and 8..15), columns 2 quad, 2 quad + 1 = (rounding, remainder)
            uint32_t x0, x1;
            if (F8) {
                const float h0 = __half2float(__float2half_rn(p0)), h1 = __half2float(__float2half_rn(p1));
                x0 = pack_f16(h0, p0 - h0);
                x1 = pack_f16(h1, p1 - h1);
            } else {
                const float h0 = __bfloat162float(__float2bfloat16_rn(p0)), h1 = __bfloat162float(__float2bfloat16_rn(p1));
                x0 = pack_bf16(h0, p0 - h0);
                x1 = pack_bf16(h1, p1 - h1);
            }
            // transposed: the B operand (keys 2 quad, 2 quad + 1 of each half; column grp)
            const uint32_t b0 = movmatrix_trans(x0), b1 = movmatrix_trans(x1);
            // V^T as the A operand: a transposing load of the chunk's V rows [key][d]
            const uint8_t* vp = vsm + ((lane & 7) + ((lane >> 4) & 1) * 8) * ROWB + ((lane >> 3) & 1) * 16;
            if (F8) {
                // The load transposes 2-byte units, so a thread gets, for keys 2 quad and 2 quad + 1 (and + 8), the
                // byte PAIR d = 2 grp, 2 grp + 1 of a 16-byte column block: bytes 0 and 2 of the register are the
                // fragment of the even d, bytes 1 and 3 of the odd d.  The even d's take rows 0..7 of the MMA and
                // the odd ones rows 8..15, so block jj's accumulator holds d = 16 jj + 2 grp (c0, c1) and
                // d = 16 jj + 2 grp + 1 (c2, c3): see the store.
#pragma unroll
                for (int j = 0; j < D / 32; ++j) {
                    uint32_t vf[4];  // keys 0..7 x bytes 0..15, keys 0..7 x bytes 16..31, keys 8..15 x the same
                    ldmatrix_x4_trans(vf, vp + j * 32);
                    mma_f16_16816(ot[2 * j], e4m3x2_to_f16x2(__byte_perm(vf[0], 0u, 0x4420)),
                                  e4m3x2_to_f16x2(__byte_perm(vf[0], 0u, 0x4431)),
                                  e4m3x2_to_f16x2(__byte_perm(vf[2], 0u, 0x4420)),
                                  e4m3x2_to_f16x2(__byte_perm(vf[2], 0u, 0x4431)), b0, b1);
                    mma_f16_16816(ot[2 * j + 1], e4m3x2_to_f16x2(__byte_perm(vf[1], 0u, 0x4420)),
                                  e4m3x2_to_f16x2(__byte_perm(vf[1], 0u, 0x4431)),
                                  e4m3x2_to_f16x2(__byte_perm(vf[3], 0u, 0x4420)),
                                  e4m3x2_to_f16x2(__byte_perm(vf[3], 0u, 0x4431)), b0, b1);
                }
            } else {
#pragma unroll
                for (int j = 0; j < D / 16; ++j) {
                    uint32_t vf[4];
                    ldmatrix_x4_trans(vf, vp + j * 32);
                    mma_bf16_16816(ot[j], vf[0], vf[1], vf[2], vf[3], b0, b1);
                }
            }
        };
        if (nch <= NW * ST) {
            // every chunk of this warp is in its own stage already (the usual case of a call per layer): one pass,
            // the score blocks of up to ST chunks side by side, one maximum and one sum per head, no rescaling
            cp_async_wait<0>();
            __syncwarp();
            float st[ST][2];
#pragma unroll
            for (int s = 0; s < ST; ++s) tr_qk(wst + s * STAGE, st[s]);  // (for every stage: the chains interleave)
            float mx = kNegBig;
#pragma unroll
            for (int s = 0; s < ST; ++s) {
                const int c = warp + s * NW;
                if (c < nch) tr_mask(c, st[s]);
                else st[s][0] = st[s][1] = kNegBig;  // a stage without a chunk holds whatever it held
                mx = fmaxf(mx, fmaxf(st[s][0], st[s][1]));
            }
#pragma unroll
            for (int o2 = 4; o2 < 32; o2 <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o2));  // over the key lanes
            M = mx;
#pragma unroll
            for (int s = 0; s < ST; ++s) {
                if (warp + s * NW < nch) {  // warp-uniform
                    const float p0 = st[s][0] > 0.5f * kNegBig ? ex2f(st[s][0] - M) : 0.f;
                    const float p1 = st[s][1] > 0.5f * kNegBig ? ex2f(st[s][1] - M) : 0.f;
                    L += p0 + p1;
                    tr_pv(wst + s * STAGE + kChunk * ROWB, p0, p1);
                }
            }
        } else {
            int stage = 0;
            for (int c = warp; c < nch; c += NW) {
                cp_async_wait<ST - 1>();
                __syncwarp();
                const uint8_t* ksm = wst + stage * STAGE;
                float st[2];
                tr_qk(ksm, st);
                tr_mask(c, st);
                float mx = fmaxf(st[0], st[1]);
#pragma unroll
                for (int o2 = 4; o2 < 32; o2 <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o2));
                // the running maximum moves only when some head's chunk maximum beats it by 2^8 (warp-uniform branch)
                if (__any_sync(0xffffffffu, mx > M + 8.f)) {
                    const float Mn = fmaxf(M, mx);
                    const float alpha = ex2f(M - Mn);
                    M = Mn;
                    L *= alpha;
#pragma unroll
                    for (int j = 0; j < D / 16; ++j) {
                        ot[j][0] *= alpha;
                        ot[j][1] *= alpha;
                        ot[j][2] *= alpha;
                        ot[j][3] *= alpha;
                    }
                }
                const float p0 = st[0] > 0.5f * kNegBig ? ex2f(st[0] - M) : 0.f;
                const float p1 = st[1] > 0.5f * kNegBig ? ex2f(st[1] - M) : 0.f;
                L += p0 + p1;
                tr_pv(ksm + kChunk * ROWB, p0, p1);
                __syncwarp();  // every lane is done with the stage before it is refilled
                issue(c + ST * NW, stage);
                stage = stage + 1 == ST ? 0 : stage + 1;
            }
            cp_async_wait<0>();
        }
#pragma unroll
        for (int o2 = 4; o2 < 32; o2 <<= 1) L += __shfl_xor_sync(0xffffffffu, L, o2);
        // the warp's result block [head][D + 8] (its own first stage), as the head-major form leaves it
        __syncwarp();  // every lane is done with stage 0
        float* ow = reinterpret_cast<float*>(wst);
        if (F8) {  // rows of a block: even d's then odd d's (see the V product); the head's V scale joins here
            const float vs = kv_scale_of(a.kv.v_scale, a.kv, layer, hm);
#pragma unroll
            for (int j = 0; j < D / 16; ++j)
                *reinterpret_cast<float2*>(ow + quad * (D + 8) + 16 * j + 2 * grp) =
                    make_float2((ot[j][0] + ot[j][1]) * vs, (ot[j][2] + ot[j][3]) * vs);
        } else {
#pragma unroll
            for (int j = 0; j < D / 16; ++j) {
                ow[quad * (D + 8) + 16 * j + grp] = ot[j][0] + ot[j][1];
                ow[quad * (D + 8) + 16 * j + 8 + grp] = ot[j][2] + ot[j][3];
            }
        }
        if (grp == 0) wml[warp * 8 + quad] = make_float2(M, L);
    } else if (nch <= NW * ST) {
        // Every chunk of this warp is in its own stage already (the usual case of a call per layer): one pass
        // over all of them - the score blocks of up to ST chunks accumulate side by side, one maximum and one
        // sum per head, no rescaling, and the P V products of the chunks follow one another.
        cp_async_wait<0>();
        __syncwarp();
        // (the products run for every stage, so that their chains interleave; a stage without a chunk holds
        // whatever it held, and its scores are replaced, not scaled)
        float s0[ST][4], s1[ST][4];
#pragma unroll
        for (int s = 0; s < ST; ++s) {
            s0[s][0] = s0[s][1] = s0[s][2] = s0[s][3] = 0.f;
            s1[s][0] = s1[s][1] = s1[s][2] = s1[s][3] = 0.f;
        }
#pragma unroll
        for (int s = 0; s < ST; ++s) qk(wst + s * STAGE, s0[s], s1[s]);
        float sv[ST][4];
        float mx = kNegBig;
#pragma unroll
        for (int s = 0; s < ST; ++s) {
            const int c = warp + s * NW;
            sv[s][0] = sv[s][1] = sv[s][2] = sv[s][3] = kNegBig;
            if (c < nch) scores(c, s0[s], s1[s], sv[s]);
            mx = fmaxf(mx, fmaxf(fmaxf(sv[s][0], sv[s][1]), fmaxf(sv[s][2], sv[s][3])));
        }
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        M = mx;
#pragma unroll
        for (int s = 0; s < ST; ++s) {
            const int c = warp + s * NW;
            if (c < nch) {
                float p[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) p[i] = sv[s][i] > 0.5f * kNegBig ? ex2f(sv[s][i] - M) : 0.f;
                L += (p[0] + p[1]) + (p[2] + p[3]);
                pv(wst + s * STAGE + kChunk * ROWB, p);
            }
        }
    } else {
        int stage = 0;
        for (int c = warp; c < nch; c += NW) {
            cp_async_wait<ST - 1>();
            __syncwarp();
            const uint8_t* ksm = wst + stage * STAGE;
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
            qk(ksm, s0, s1);
            float sv[4];
            scores(c, s0, s1, sv);
            float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            // the running maximum moves only when some head's chunk maximum beats it by 2^8 (warp-uniform branch)
            if (__any_sync(0xffffffffu, mx > M + 8.f)) {
                const float Mn = fmaxf(M, mx);
                const float alpha = ex2f(M - Mn);
                M = Mn;
                L *= alpha;
#pragma unroll
                for (int i = 0; i < D / 8; ++i) {
                    o[i][0] *= alpha;
                    o[i][1] *= alpha;
                    o[i][2] *= alpha;
                    o[i][3] *= alpha;
                }
            }
            float p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = sv[i] > 0.5f * kNegBig ? ex2f(sv[i] - M) : 0.f;
            L += (p[0] + p[1]) + (p[2] + p[3]);
            pv(ksm + kChunk * ROWB, p);
            __syncwarp();  // every lane is done with the stage before it is refilled
            issue(c + ST * NW, stage);
            stage = stage + 1 == ST ? 0 : stage + 1;
        }
    }
    cp_async_wait<0>();
    // ---- the warps of the CTA: (max, sum, O) through shared memory (each warp's own first stage) ----
    __syncwarp();
    if (!keys_on_rows) {
        L += __shfl_xor_sync(0xffffffffu, L, 1);
        L += __shfl_xor_sync(0xffffffffu, L, 2);
        float* ow = reinterpret_cast<float*>(wst);  // [8 heads][D + 8]: the padding keeps the heads on different banks
        if (F8) {  // undo the order of the head dimension (see the V product) and apply the head's V scale
            const float vs = kv_scale_of(a.kv.v_scale, a.kv, layer, hm);
#pragma unroll
            for (int i = 0; i < D / 8; ++i) {
                const int d0 = 32 * (i >> 2) + 16 * ((i >> 1) & 1) + 4 * quad + (i & 1);
                ow[grp * (D + 8) + d0] = (o[i][0] + o[i][2]) * vs;
                ow[grp * (D + 8) + d0 + 2] = (o[i][1] + o[i][3]) * vs;
            }
        } else {
#pragma unroll
            for (int i = 0; i < D / 8; ++i)
                *reinterpret_cast<float2*>(ow + grp * (D + 8) + i * 8 + 2 * quad) = make_float2(o[i][0] + o[i][2], o[i][1] + o[i][3]);
        }
        if (quad == 0) wml[warp * 8 + grp] = make_float2(M, L);
    }
    __syncthreads();
    // every CTA of the cluster knows by now that the first CTA's deposit barrier is armed
    if (CS > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    const bool remote = rank != 0;
    float* mine = comb + rank * PS;
    const uint32_t mine_r = remote ? map_to_rank(smem_addr(mine), 0) : 0u;
    const uint32_t bar_r = remote ? map_to_rank(smem_addr(dep_bar), 0) : 0u;
    // V neighbouring d of a head per thread: the warps' weights are computed once for all of them, and a remote
    // deposit is one vector store (a store into another CTA's shared memory costs the same for 4 to 16 bytes)
    auto merge_warps = [&](auto vec) {
        constexpr int V = decltype(vec)::value;
        for (int i = tid; i < G * (D / V); i += NT) {
            const int r = i / (D / V), d = V * (i - r * (D / V));
            float2 ml[NW];
            float Mc = kNegBig;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                ml[w] = wml[w * 8 + r];
                Mc = fmaxf(Mc, ml[w].x);
            }
            float Lc = 0.f, o[V];
#pragma unroll
            for (int k = 0; k < V; ++k) o[k] = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) {  // fixed order: deterministic
                const float wgt = ex2f(ml[w].x - Mc);
                const float* ov = reinterpret_cast<const float*>(stages + (size_t)w * ST * STAGE) + r * (D + 8) + d;
                Lc += ml[w].y * wgt;
                if (V == 4) {
                    const float4 x = *reinterpret_cast<const float4*>(ov);
                    o[0] += x.x * wgt;
                    o[1] += x.y * wgt;
                    o[V - 2] += x.z * wgt;
                    o[V - 1] += x.w * wgt;
                } else {
                    const float2 x = *reinterpret_cast<const float2*>(ov);
                    o[0] += x.x * wgt;
                    o[1] += x.y * wgt;
                }
            }
            if (V == 4) {
                if (remote) st_async_f32x4(mine_r + 4 * (r * D + d), make_float4(o[0], o[1], o[V - 2], o[V - 1]), bar_r);
                else *reinterpret_cast<float4*>(mine + r * D + d) = make_float4(o[0], o[1], o[V - 2], o[V - 1]);
            } else {
                if (remote) st_async_f32x2(mine_r + 4 * (r * D + d), o[0], o[1], bar_r);
                else *reinterpret_cast<float2*>(mine + r * D + d) = make_float2(o[0], o[1]);
            }
            if (d == 0) {  // (maximum, sum) of the head: one store
                if (remote) st_async_f32x2(mine_r + 4 * (G * D + 2 * r), Mc, Lc, bar_r);
                else *reinterpret_cast<float2*>(mine + G * D + 2 * r) = make_float2(Mc, Lc);
            }
        }
    };
    // a CTA's slot is G (D + 2) floats: its rows start on 16 bytes for an even G, on 8 bytes otherwise
    if (G % 2 == 0) merge_warps(std::integral_constant<int, 4>{});
    else merge_warps(std::integral_constant<int, 2>{});
    if (remote) return;
    if (CS > 1) wait_deposits(smem_addr(dep_bar), a.wait_limit, status);
    __syncthreads();  // this CTA's own slot
    merge_and_store<D, NT>(a, comb, CS, G, layer, b, h, tid);
}

template <int D, int NW, int ST, bool F8>
int launch_inst(const DraftArgs& a, const StreamShape& shp, size_t smem, cudaStream_t stream)
{
    auto kern = draft_stream_kernel<D, NW, ST, F8>;
    if (!opt_in_smem(reinterpret_cast<const void*>(kern), smem)) return SPEC_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(shp.cs, a.kv.n_kv_heads, a.kv.n_layers * a.kv.batch);
    cfg.blockDim = dim3(NW * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = shp.cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // Only a call that carries the early-gather promise may start under the preceding kernel; any
    // other call is an ordinary launch, so whatever follows it finds that kernel's predecessors complete.
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.early_gather ? 2 : 1;
    if (cudaLaunchKernelEx(&cfg, kern, a, shp, static_cast<int*>(a.workspace)) != cudaSuccess) {
        cudaGetLastError();
        return SPEC_ERR_CUDA;
    }
    count_launch(1);
    return SPEC_OK;
}

template <int D, bool F8>
int launch_shape(const DraftArgs& a, const StreamShape& shp, cudaStream_t stream)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const size_t smem = stream_smem_bytes<D, F8>(G, shp.nw, shp.st, shp.per, shp.cs);
    if (smem > kSmemLimit) return SPEC_ERR_UNSUPPORTED_SHAPE;
#define SPEC_INST(W_, S_) \
    if (shp.nw == W_ && shp.st == S_) return launch_inst<D, W_, S_, F8>(a, shp, smem, stream);
    SPEC_INST(4, 2)
    SPEC_INST(4, 3)
    SPEC_INST(8, 1)
    SPEC_INST(8, 2)
    SPEC_INST(8, 3)
    SPEC_INST(12, 2)
#undef SPEC_INST
    return SPEC_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace

// How a call is split: CTAs per cluster (one cluster per (layer, sequence, KV head)), keys per CTA,
// warps per CTA and stages per warp.
//  - Few problems (a per-layer call at batch 1): the call is a chain of latencies, so every chunk
//    should be in flight at once on as many SMs as a cluster reaches, and the CTAs of three
//    consecutive calls should fit the GPU together (a call's early gather runs under the calls
//    before it): 8 warps x 3 stages, one CTA per SM, clusters of 8, or of 6 where three calls of
//    8-CTA clusters would not fit and a warp still gets about three chunks.
//  - Many problems: several small CTAs per SM whose gathers overlap each other's arithmetic; the
//    split is the one a simple cost model likes best (waves of CTAs x the longer of "bytes an SM
//    pulls at about 48 GB/s" and "trips to memory of one warp").
bool stream_plan(const KvView& kv, int head_dim, int n_keys_max, StreamShape* out)
{
    const long probs = (long)kv.n_layers * kv.batch * kv.n_kv_heads;
    const int G = kv.n_q_heads / kv.n_kv_heads;
    const int keys = n_keys_max > 0 ? n_keys_max : 1;
    const int chunks = (keys + kChunk - 1) / kChunk;
    const int nsm = sm_count();
    const size_t stage = kv.fp8 ? (head_dim == 128 ? Geo<128, true>::STAGE : Geo<64, true>::STAGE)
                                : (head_dim == 128 ? Geo<128, false>::STAGE : Geo<64, false>::STAGE);
    auto smem_of = [&](int cs, int nw, int st, int per) {
        return (size_t)nw * st * stage + (size_t)per * 4 + (size_t)nw * 64 + 16 + (size_t)cs * G * (head_dim + 2) * 4;
    };
    if (probs * draft::kMaxCluster <= nsm) {
        int cs = draft::kMaxCluster;
        if (3 * probs * 8 > nsm && 3 * probs * 6 <= nsm && chunks <= 6 * 8 * 3) cs = 6;
        while (cs > 1 && (chunks + cs - 1) / cs < 8) --cs;  // at least a chunk per warp
        const int per = (chunks + cs - 1) / cs * kChunk;
        int st = 3;
        while (st > 1 && smem_of(cs, 8, st, per) > draft::kSmemLimit) --st;
        if (smem_of(cs, 8, st, per) > draft::kSmemLimit) return false;
        *out = StreamShape{cs, per, 8, st};
        // more chunks than 8 warps x 3 stages hold at once: 12 warps x 2 stages finish the share in fewer trips
        if (per / kChunk > 24 && smem_of(cs, 12, 2, per) <= draft::kSmemLimit) *out = StreamShape{cs, per, 12, 2};
        return true;
    }
    static const int kCombos[4][2] = {{4, 2}, {4, 3}, {8, 2}, {8, 3}};
    double best = 1e30;
    StreamShape bs = {0, 0, 0, 0};
    for (int cs = 1; cs <= draft::kMaxCluster; ++cs) {
        const int cc = (chunks + cs - 1) / cs;  // chunks per CTA
        const int per = cc * kChunk;
        for (const auto& nwst : kCombos) {
            const int nw = nwst[0], st = nwst[1];
            const size_t smem = smem_of(cs, nw, st, per);
            if (smem > draft::kSmemLimit) continue;
            int occ = (int)((228 * 1024) / (smem + 1024));
            occ = occ < 1 ? 1 : occ;
            if (occ * nw > 48) occ = 48 / nw;  // registers: about 140 per thread
            const long ctas = probs * cs;
            const long slots = (long)nsm * occ;
            const long waves = (ctas + slots - 1) / slots;
            const int wc = (cc + nw - 1) / nw;     // chunks per warp
            const int rounds = (wc + st - 1) / st;  // latency-bound trips to memory per warp
            const double sm_ctas = ctas >= slots ? occ : (double)ctas / nsm > 1.0 ? (double)ctas / nsm : 1.0;
            const double bytes_us = sm_ctas * cc * (double)stage / 48.0e3;
            const double trips_us = rounds * 1.3 + wc * 0.18;
            const double t = waves * (bytes_us > trips_us ? bytes_us : trips_us) + 0.25 * cs + 0.02 * nw;
            if (t < best) {
                best = t;
                bs = StreamShape{cs, per, nw, st};
            }
        }
    }
    if (bs.cs == 0) return false;
    *out = bs;
    return true;
}

int draft_stream_launch(const DraftArgs& a, const StreamShape& shp, cudaStream_t stream)
{
    if (a.kv.head_dim == 128) return a.kv.fp8 ? launch_shape<128, true>(a, shp, stream) : launch_shape<128, false>(a, shp, stream);
    if (a.kv.head_dim == 64) return a.kv.fp8 ? launch_shape<64, true>(a, shp, stream) : launch_shape<64, false>(a, shp, stream);
    return SPEC_ERR_UNSUPPORTED_SHAPE;
}

size_t draft_workspace(const KvView&, int) { return kStatusBytes; }

int draft_launch(const DraftArgs& a, cudaStream_t stream)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    if (G > draft::kMaxGroup) return SPEC_ERR_UNSUPPORTED_SHAPE;
    if (a.workspace_bytes < kStatusBytes) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    // row offsets travel as 32-bit counts of 16-byte units: a layer's K (or V) must stay below 64 GiB
    if ((int64_t)a.kv.n_pages * a.kv.page_stride >= ((int64_t)1 << (a.kv.fp8 ? 36 : 35))) return SPEC_ERR_UNSUPPORTED_SHAPE;
    StreamShape shp;
    if (!stream_plan(a.kv, a.kv.head_dim, a.k_total + a.max_tail, &shp)) return SPEC_ERR_UNSUPPORTED_SHAPE;
    return draft_stream_launch(a, shp, stream);
}

}  // namespace spec
