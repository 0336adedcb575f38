// Sparse draft attention of Eq. 5: one query per sequence attends the recalled rows
// Gather(K, I), Gather(V, I) plus the dense tail of tokens drafted this round.  The gather is
// fused: 16-byte asynchronous copies (cp.async) pull every indexed K and V row straight from the
// dense cache into shared memory; nothing gathered is written back to global memory.
//
// The call is latency-bound (a few thousand recalled keys per head), so the kernel is built to
// be short rather than wide.  A thread-block cluster splits the key list of one (sequence, KV
// head); each CTA keeps its whole share (up to 288 keys) in shared memory and runs three short
// phases on it, separated by two block barriers:
//   1. scores: every warp takes 16-key chunks, S^T = K q^T on the tensor cores (mma.sync
//      m16n8k16 with the keys as the M dimension and the G <= 8 query heads of the group as N),
//      and publishes its running maximum;
//   2. probabilities: with the CTA-wide maximum known, P = 2^(S - max) is written once to
//      shared memory as bf16 hi + lo parts;
//   3. values: each warp owns a 16-wide slice of the head dimension and accumulates
//      O^T = V^T P^T over all keys of the share, so no merge between warps is needed.
// The CTAs of the cluster deposit (max, sum, O) in the first CTA through distributed shared
// memory (asynchronous stores counted on an mbarrier there); it merges them in rank order
// (deterministic) once every byte has landed.
// One launch per call, no global scratch, no second kernel.
#include <cstdio>
#include <cstdlib>

#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kCap = 352;      // most K rows (and V rows) resident per CTA
constexpr int kRound = 176;    // keys per round when a share exceeds kCap (two buffers of kRound = kCap rows)
constexpr int kThreads = 512;  // four warps per scheduler: the phases are dependent chains that need interleaving
constexpr int kWarps = kThreads / 32;
constexpr int kRedPitch = kWarps + 2;  // float2 per quad row of the per-warp maxima / sums: the 16 B of padding keeps the four rows on different banks
constexpr int kMaxGroup = 8;    // query heads per KV head
constexpr int kMaxCluster = 8;  // portable cluster size (a GPC cannot hold two clusters of 16)
constexpr float kNegBig = -1.0e30f;  // "minus infinity" that stays finite under subtraction
constexpr long long kTimeoutCycles = 2000ll * 1000ll * 1000ll;  // bound of the deposit wait: about a second

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
// 4 bytes into the shared memory of another CTA of the cluster; the bytes are counted on that
// CTA's mbarrier when they have landed (no fence, no cluster barrier needed on either side)
__device__ __forceinline__ void st_async_f32(uint32_t remote_addr, float v, uint32_t remote_bar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
                 ::"r"(remote_addr), "r"(__float_as_uint(v)), "r"(remote_bar) : "memory");
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
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
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
__device__ __forceinline__ float group_max(float x)  // over the 8 lanes that share lane % 4
{
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 4));
    x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 8));
    return fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 16));
}
__device__ __forceinline__ float group_sum(float x)
{
    x += __shfl_xor_sync(0xffffffffu, x, 4);
    x += __shfl_xor_sync(0xffffffffu, x, 8);
    return x + __shfl_xor_sync(0xffffffffu, x, 16);
}

// How a call is split: CTAs per cluster (one cluster per (layer, sequence, KV head)), keys per
// CTA, keys per round, K rows resident per CTA.
struct DraftShape {
    int cs, per, rk, rows;
    int packed;  // G <= 4: [P hi | P lo] share the eight MMA columns in phase 3
};

// Shared memory of one CTA, in this order (every block 16-byte aligned):
//   K [rows][D + 8] bf16 | V [rows][D + 8] bf16 | P hi, P lo [8][rk + 8] bf16 each |
//   row offsets int64 [rows] | key positions int [rows] | per-warp maxima, per-warp sums float2 [4][16 warps + 2] each |
//   partial O of the warps that share a head-dim slice float [16 - D/16 warps][32 lanes][4] |
//   deposit barrier (16 B) | deposit area float [cs][G * (D + 2)] (used in the first CTA of the cluster)
// The 16 bytes of padding per K/V row spread the banks for ldmatrix.
__host__ __device__ inline size_t draft_smem_bytes(int D, int G, const DraftShape& s)
{
    return (size_t)2 * s.rows * (D + 8) * 2 + (size_t)2 * kMaxGroup * (s.rk + 8) * 2 + (size_t)s.rows * 12 +
           (size_t)2 * 8 * kRedPitch * 4 + (size_t)(kWarps - D / 16) * 512 + 16 + (size_t)s.cs * G * (D + 2) * 4;
}

template <int D>
__global__ void __launch_bounds__(kThreads)
draft_cluster_kernel(DraftArgs a, DraftShape shp, int* __restrict__ status)
{
    constexpr int PITCH = D + 8;
    constexpr int CH = D / 8;               // 16-byte pieces per row
    constexpr int RPP = kThreads / CH;      // rows covered by one pass of the block
    constexpr int MAXJ = (kCap / 16 + kWarps - 1) / kWarps;  // 16-key chunks per warp and round
    constexpr int NSL = D / 16;             // 16-wide slices of the head dimension
    constexpr int KH = kWarps / NSL;        // warps per slice: each takes every KH-th chunk in phase 3
    constexpr float kLog2e = 1.4426950408889634f;
    extern __shared__ __align__(16) uint8_t smem[];
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    const int per = shp.per, RK = shp.rk, PP = RK + 8, PS = G * (D + 2);
    __nv_bfloat16* Ks = reinterpret_cast<__nv_bfloat16*>(smem);
    __nv_bfloat16* Vs = Ks + shp.rows * PITCH;
    __nv_bfloat16* Ph = Vs + shp.rows * PITCH;
    __nv_bfloat16* Pl = Ph + kMaxGroup * PP;
    int64_t* rowoff = reinterpret_cast<int64_t*>(Pl + kMaxGroup * PP);  // element offset of the row, -1 if masked
    int* keypos = reinterpret_cast<int*>(rowoff + shp.rows);
    float* wmax = reinterpret_cast<float*>(keypos + shp.rows);
    float* wl = wmax + 8 * kRedPitch;
    float* opart = wl + 8 * kRedPitch;  // [kWarps - NSL][32][4]
    uint64_t* dep_bar = reinterpret_cast<uint64_t*>(opart + (kWarps - NSL) * 128);  // first CTA: counts deposited bytes
    float* comb = reinterpret_cast<float*>(dep_bar + 2);  // [CS][PS]: O rows [G][D], then the maxima [G], then the sums [G]

#ifdef SPEC_TRACE
#define DSTAMP(i) do { if (threadIdx.x == 0) { \
        const size_t blk_ = ((size_t)blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x; \
        if (a.workspace_bytes >= 256 + (blk_ + 1) * 128) { \
            unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); \
            reinterpret_cast<unsigned long long*>(status)[32 + blk_ * 16 + (i)] = t_; } } } while (0)
#else
#define DSTAMP(i) do { } while (0)
#endif
    DSTAMP(0);
    const int CS = gridDim.x;              // the cluster spans the x dimension
    const int rank = blockIdx.x;
    const int h = blockIdx.y;
    const int layer = blockIdx.z / a.kv.batch, b = blockIdx.z % a.kv.batch;
    const int64_t prob = (int64_t)blockIdx.z * a.kv.n_kv_heads + h;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int grp = lane >> 2, quad = lane & 3;
    const int slice = warp % NSL, kh = warp / NSL;

    // Programmatic dependent launch: the next kernel in the stream may start its own prologue
    // (index loads, gather of recalled rows) while this one is still computing.  Everything this
    // kernel reads before griddepcontrol.wait below is immutable during a drafting round (indices,
    // lengths, recalled rows of the dense cache); Q, the dense tail and the outputs come after.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    // The first CTA of the cluster counts the bytes the others deposit at the end on an mbarrier.
    // It is armed here; the cluster barrier that tells the others so is split around the gather.
    if (CS > 1) {
        if (rank == 0 && tid == 0) {
            mbar_init(smem_addr(dep_bar), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
            mbar_arrive_expect_tx(smem_addr(dep_bar), (uint32_t)(CS - 1) * PS * 4);
        }
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }

    const int32_t* idx = a.indices + prob * a.k_total;
    // contiguous shares in multiples of the 16-key chunk; the share size depends only on host-side
    // bounds, so every CTA of the cluster agrees on it without exchanging anything
    const int NB = RK < per ? 2 : 1;  // buffers of RK rows (two when the share takes several rounds)
    const int n_rec = min(max(__ldg(a.n_indices + prob), 0), a.k_total);
    const int ts = __ldg(a.tail_start + b), cl = __ldg(a.cur_len + b);

    // Gather of round r into its buffer, in two short loops (the code is kept small on purpose:
    // a kernel this short is paced by instruction fetch when its loops are unrolled into long
    // straight-line code).  First one thread per row resolves the row: position, validity, offset
    // in the cache (page-table lookup) -> shared memory.  After a barrier CH threads per row copy
    // one 16-byte piece of the K row and one of the V row each; masked rows are zero-filled (they
    // meet P = 0 in the P V product and must be finite).
    // mode 0: recalled rows and the masked padding of the last chunk (readable before the
    // dependency wait), 1: rows of the dense tail only, 2: all.
    const int slot = tid / CH, piece = tid % CH;
    const int hm = a.head_div > 1 ? h / a.head_div : h;  // the cache head this problem's rows come from
    const __nv_bfloat16* kbase = a.kv.k + layer * a.kv.layer_stride + hm * a.kv.head_stride + piece * 8;
    const __nv_bfloat16* vbase = a.kv.v + layer * a.kv.layer_stride + hm * a.kv.head_stride + piece * 8;
    const int32_t* ptab = a.kv.page_table ? a.kv.page_table + (int64_t)b * a.kv.max_pages : nullptr;
    auto gather = [&](int r, int mode, int k0, int k1) {
        const int base = k0 + r * RK;
        const int nk = max(min(RK, k1 - base), 0);
        const int row0 = NB == 2 ? (r & 1) * kRound : 0;
        const int first_tail = min(max(n_rec - base, 0), nk);  // rows [first_tail, nk) come from the dense tail
        const int lo = mode == 1 ? first_tail : 0;
        const int hi = mode == 1 ? nk : ((nk + 15) & ~15);
        for (int lr = lo + tid; lr < hi; lr += kThreads) {
            const bool is_tail = lr >= first_tail && lr < nk;
            if (mode == 0 && is_tail) continue;
            int pos = -1;
            if (lr < nk) {
                pos = is_tail ? ts + (base + lr - n_rec) : __ldg(idx + base + lr);
                if (pos < 0 || pos >= cl) {
                    set_status(status, SPEC_ERR_BAD_INDEX);
                    pos = -1;
                }
            }
            int64_t off = -1;
            if (pos >= 0) {
                const int page = page_of(a.kv, pos);
                const int slot_in = pos - page * a.kv.page_size;
                const int64_t phys = ptab ? (int64_t)__ldg(ptab + page) : (int64_t)b * a.kv.max_pages + page;
                off = phys * a.kv.page_stride + (int64_t)slot_in * a.kv.slot_stride;
            }
            keypos[row0 + lr] = pos;
            rowoff[row0 + lr] = off;
        }
        __syncthreads();
#pragma unroll 2
        for (int lr = lo + slot; lr < hi; lr += RPP) {
            if (mode == 0 && lr >= first_tail && lr < nk) continue;
            const int64_t off = rowoff[row0 + lr];
            const uint32_t nbytes = off >= 0 ? 16u : 0u;
            cp_async16(Ks + (row0 + lr) * PITCH + piece * 8, kbase + (off >= 0 ? off : 0), nbytes);
            cp_async16(Vs + (row0 + lr) * PITCH + piece * 8, vbase + (off >= 0 ? off : 0), nbytes);
        }
    };

    // the share is known once the list length is; recalled rows never depend on the previous kernel
    const int n_tail = min(max(cl - ts, 0), a.max_tail);
    const int n = n_rec + n_tail;
    const int k0 = min(n, rank * per);
    const int k1 = min(n, k0 + per);
    const int n_rounds = (k1 - k0 + RK - 1) / RK;
    for (int r = 0; r < min(n_rounds, NB); ++r) gather(r, 0, k0, k1);
    cp_async_commit();
    // Q and the dense tail are written by earlier kernels of the stream and read after the wait;
    // asking L2 for their lines now is harmless (L2 is the point of coherence: a later write
    // lands in the same line) and spares the wait a trip to DRAM when they were not there yet
    if (tid < G)
        prefetch_l2(a.q + (((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + tid) * D, D * 2);
    else if (tid >= 32 && tid < 32 + k1 - max(n_rec, k0)) {
        const int pos = ts + (max(n_rec, k0) + tid - 32 - n_rec);
        if (pos >= 0 && pos < cl) {
            const int page = page_of(a.kv, pos);
            const int64_t phys = ptab ? (int64_t)__ldg(ptab + page) : (int64_t)b * a.kv.max_pages + page;
            const int64_t off = layer * a.kv.layer_stride + hm * a.kv.head_stride + phys * a.kv.page_stride +
                                (int64_t)(pos - page * a.kv.page_size) * a.kv.slot_stride;
            prefetch_l2(a.kv.k + off, D * 2);
            prefetch_l2(a.kv.v + off, D * 2);
        }
    }
    DSTAMP(1);
    if (CS > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    DSTAMP(2);
    // Rows of the dense tail.  A share that is resident in one round: the warp that owns a tail row's
    // chunk in phase 1 copies the row itself and waits for it only when it reaches that chunk, so the
    // fetch runs beside the Q loads instead of in front of the block barrier.  Shares that take
    // several rounds use the common gather.
    const int t0 = max(n_rec, k0) - k0, t1 = k1 - k0;  // local rows [t0, t1) of the share come from the tail
    if (NB == 1) {
        constexpr int LPR = 2 * CH;  // lanes per row: CH pieces of K, CH pieces of V
        for (int c = t0 >> 4; c * 16 < t1; ++c) {
            if (c % kWarps != warp) continue;
            const int lo = max(c * 16, t0), n = min(c * 16 + 16, t1) - lo;  // n <= 16 rows, one lane resolves each
            int64_t off = -1;
            if (lane < n) {
                int pos = ts + (k0 + lo + lane - n_rec);
                if (pos < 0 || pos >= cl) {
                    set_status(status, SPEC_ERR_BAD_INDEX);
                    pos = -1;
                }
                keypos[lo + lane] = pos;
                if (pos >= 0) {
                    const int page = page_of(a.kv, pos);
                    const int slot_in = pos - page * a.kv.page_size;
                    const int64_t phys = ptab ? (int64_t)__ldg(ptab + page) : (int64_t)b * a.kv.max_pages + page;
                    off = phys * a.kv.page_stride + (int64_t)slot_in * a.kv.slot_stride;
                }
            }
            const bool is_v = (lane % LPR) >= CH;  // kbase / vbase already point at this lane's piece (lane % CH)
            for (int i = 0; i < n; i += 32 / LPR) {
                const int row = i + lane / LPR;
                const int64_t o = __shfl_sync(0xffffffffu, off, row & 31);
                if (row < n)
                    cp_async16((is_v ? Vs : Ks) + (lo + row) * PITCH + piece * 8, (is_v ? vbase : kbase) + (o >= 0 ? o : 0),
                               o >= 0 ? 16u : 0u);
            }
        }
        cp_async_commit();
    } else if (t1 > t0) {  // the same answer in every thread
        for (int r = 0; r < min(n_rounds, NB); ++r) gather(r, 1, k0, k1);
        cp_async_commit();
    }
    // B fragments of q^T (d x g) straight from global memory: the thread holds q[g = grp] at
    // d = 16 ks + 2 quad + {0, 1} and + {8, 9}; heads beyond the group are zero
    uint32_t qb[D / 16][2];
    {
        const int64_t row = ((int64_t)layer * a.kv.batch + b) * a.kv.n_q_heads + h * G + grp;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(a.q + row * D);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
            qb[ks][0] = grp < G ? __ldg(qrow + ks * 8 + quad) : 0u;
            qb[ks][1] = grp < G ? __ldg(qrow + ks * 8 + 4 + quad) : 0u;
        }
    }

    if (NB == 1) cp_async_wait<1>();  // everything but the tail rows just requested
    else cp_async_wait<0>();
    __syncthreads();
    DSTAMP(3);

    // running state of the share; the thread tracks heads g = 2 quad and 2 quad + 1 (every thread
    // of the CTA computes the same values for them from shared memory)
    const float sc = a.kv.scale * kLog2e;
    const bool packed = shp.packed != 0;  // see phase 3
    float M0 = kNegBig, M1 = kNegBig, L0 = 0.f, L1 = 0.f;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;

    for (int r = 0; r < n_rounds; ++r) {
        if (r > 0) {  // all but the newest group (the round after this one) have landed
            cp_async_wait<1>();
            __syncthreads();
        }
        const int row0 = NB == 2 ? (r & 1) * kRound : 0;
        const int nk = min(RK, k1 - (k0 + r * RK));
        const int nch = (nk + 15) >> 4;
        const int* kp = keypos + row0;

        // ---- phase 1: S^T = K q^T for this warp's chunks (keys x heads), masked and scaled ----
        float s[MAXJ][4];
        float mx0 = kNegBig, mx1 = kNegBig;
#pragma unroll
        for (int j = 0; j < MAXJ; ++j) {
            const int c = warp + kWarps * j;
            s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
            if (c < nch) {
                if (NB == 1 && c * 16 + 16 > t0 && c * 16 < t1) {  // this warp copied the chunk's tail rows
                    cp_async_wait<0>();
                    __syncwarp();
                }
                uint32_t kf[D / 16][4];  // all fragments of the chunk are requested before the first MMA
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    ldmatrix_x4(kf[ks], Ks + (row0 + c * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * PITCH + ks * 16 +
                                            (lane >> 4) * 8);
                float s2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < D / 16; ks += 2) {  // two accumulation chains
                    mma_bf16(s[j], kf[ks], qb[ks][0], qb[ks][1]);
                    mma_bf16(s2, kf[ks + 1], qb[ks + 1][0], qb[ks + 1][1]);
                }
                const bool ka = kp[c * 16 + grp] >= 0, kb = kp[c * 16 + grp + 8] >= 0;
                s[j][0] = ka ? (s[j][0] + s2[0]) * sc : kNegBig;
                s[j][1] = ka ? (s[j][1] + s2[1]) * sc : kNegBig;
                s[j][2] = kb ? (s[j][2] + s2[2]) * sc : kNegBig;
                s[j][3] = kb ? (s[j][3] + s2[3]) * sc : kNegBig;
                mx0 = fmaxf(mx0, fmaxf(s[j][0], s[j][2]));
                mx1 = fmaxf(mx1, fmaxf(s[j][1], s[j][3]));
            }
        }
        mx0 = group_max(mx0);
        mx1 = group_max(mx1);
        if (grp == 0) reinterpret_cast<float2*>(wmax)[quad * kRedPitch + warp] = make_float2(mx0, mx1);
        cp_async_wait<0>();  // tail rows of V: seen by every warp after the barrier
        __syncthreads();
        if (r == 0) DSTAMP(8);

        // ---- phase 2: P = 2^(S - max) against the CTA-wide maximum, stored as bf16 hi + lo ----
        float Mn0 = M0, Mn1 = M1;
        {   // [quad][warp] pairs: two warps per 16-byte load, every lane of a quad reads the same words
            const float4* wm = reinterpret_cast<const float4*>(wmax) + quad * (kRedPitch / 2);
            float a0 = kNegBig, a1 = kNegBig, b0 = kNegBig, b1 = kNegBig;
#pragma unroll
            for (int w = 0; w < kWarps / 2; ++w) {
                const float4 t = wm[w];
                a0 = fmaxf(a0, t.x);
                a1 = fmaxf(a1, t.y);
                b0 = fmaxf(b0, t.z);
                b1 = fmaxf(b1, t.w);
            }
            Mn0 = fmaxf(Mn0, fmaxf(a0, b0));
            Mn1 = fmaxf(Mn1, fmaxf(a1, b1));
        }
        const float alpha0 = ex2f(M0 - Mn0), alpha1 = ex2f(M1 - Mn1);
        float ls0 = 0.f, ls1 = 0.f;
#pragma unroll
        for (int j = 0; j < MAXJ; ++j) {
            const int c = warp + kWarps * j;
            if (c < nch) {
                float p[4];
                p[0] = s[j][0] > 0.5f * kNegBig ? ex2f(s[j][0] - Mn0) : 0.f;
                p[1] = s[j][1] > 0.5f * kNegBig ? ex2f(s[j][1] - Mn1) : 0.f;
                p[2] = s[j][2] > 0.5f * kNegBig ? ex2f(s[j][2] - Mn0) : 0.f;
                p[3] = s[j][3] > 0.5f * kNegBig ? ex2f(s[j][3] - Mn1) : 0.f;
                ls0 += p[0] + p[2];
                ls1 += p[1] + p[3];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int g = 2 * quad + (e & 1), key = c * 16 + grp + (e >> 1) * 8;
                    const __nv_bfloat16 hi = __float2bfloat16_rn(p[e]);
                    Ph[g * PP + key] = hi;
                    // G <= 4: the lo parts go to rows 4..7 of the hi array (see phase 3)
                    (packed ? Ph + 4 * PP : Pl)[g * PP + key] = __float2bfloat16_rn(p[e] - __bfloat162float(hi));
                }
            }
        }
        ls0 = group_sum(ls0);
        ls1 = group_sum(ls1);
        if (grp == 0) reinterpret_cast<float2*>(wl)[quad * kRedPitch + warp] = make_float2(ls0, ls1);
        __syncthreads();
        if (r == 0) DSTAMP(9);
        {
            const float4* wlp = reinterpret_cast<const float4*>(wl) + quad * (kRedPitch / 2);
            float t0 = 0.f, t1 = 0.f, u0 = 0.f, u1 = 0.f;
#pragma unroll
            for (int w = 0; w < kWarps / 2; ++w) {  // fixed order: even warps, odd warps, then both
                const float4 t = wlp[w];
                t0 += t.x;
                t1 += t.y;
                u0 += t.z;
                u1 += t.w;
            }
            t0 += u0;
            t1 += u1;
            L0 = L0 * alpha0 + t0;
            L1 = L1 * alpha1 + t1;
            M0 = Mn0;
            M1 = Mn1;
        }

        // ---- phase 3: O^T += V^T P^T on this warp's 16-wide slice of the head dimension ----
        // With G <= 4 the eight columns of the MMA hold [P hi | P lo] of the four heads side by
        // side, so one MMA per chunk covers both parts (the two halves are added at the end);
        // larger groups take one MMA for each part.
        {
            if (r > 0) {
                float a0 = alpha0, a1 = alpha1;
                if (packed) {  // columns 4..7 belong to heads 0..3 again
                    a0 = __shfl_sync(0xffffffffu, alpha0, (lane & ~3) | (quad & 1));
                    a1 = __shfl_sync(0xffffffffu, alpha1, (lane & ~3) | (quad & 1));
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[i][0] *= a0;
                    acc[i][1] *= a1;
                    acc[i][2] *= a0;
                    acc[i][3] *= a1;
                }
            }
            const __nv_bfloat16* vb = Vs + (row0 + (lane & 7) + ((lane >> 4) & 1) * 8) * PITCH + slice * 16 +
                                      ((lane >> 3) & 1) * 8;
            // no branches inside the loops: a chunk index past the end is clamped to a valid chunk
            // and meets P = 0 (uniform branches around the asm blocks cost more than the work)
            if (packed) {
                const uint32_t* pp = reinterpret_cast<const uint32_t*>(Ph + grp * PP) + quad;
                const bool real = (grp & 3) < G;
                for (int kc0 = kh; kc0 < nch; kc0 += 4 * KH) {  // four chunks requested, then four MMAs on four chains
                    uint32_t vf[4][4], pb[4][2];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool ok = kc0 + u * KH < nch;
                        const int kc = ok ? kc0 + u * KH : kc0;
                        ldmatrix_x4_trans(vf[u], vb + kc * 16 * PITCH);
                        const uint32_t v0 = pp[kc * 8], v1 = pp[kc * 8 + 4];
                        pb[u][0] = real && ok ? v0 : 0u;
                        pb[u][1] = real && ok ? v1 : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) mma_bf16(acc[u], vf[u], pb[u][0], pb[u][1]);
                }
            } else {
                const uint32_t* ph = reinterpret_cast<const uint32_t*>(Ph + grp * PP) + quad;
                const uint32_t* pl = reinterpret_cast<const uint32_t*>(Pl + grp * PP) + quad;
                const bool real = grp < G;
                for (int kc0 = kh; kc0 < nch; kc0 += 4 * KH) {  // four chunks requested, then eight MMAs on four chains
                    uint32_t vf[4][4], pb[4][4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool ok = kc0 + u * KH < nch;
                        const int kc = ok ? kc0 + u * KH : kc0;
                        ldmatrix_x4_trans(vf[u], vb + kc * 16 * PITCH);
                        const uint32_t v0 = ph[kc * 8], v1 = ph[kc * 8 + 4], v2 = pl[kc * 8], v3 = pl[kc * 8 + 4];
                        pb[u][0] = real && ok ? v0 : 0u;
                        pb[u][1] = real && ok ? v1 : 0u;
                        pb[u][2] = real && ok ? v2 : 0u;
                        pb[u][3] = real && ok ? v3 : 0u;
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        mma_bf16(acc[(u & 1) * 2], vf[u], pb[u][0], pb[u][1]);
                        mma_bf16(acc[(u & 1) * 2 + 1], vf[u], pb[u][2], pb[u][3]);
                    }
                }
            }
        }
        if (NB == 2) {  // refill the buffer just consumed with the round after next
            __syncthreads();
            if (r + NB < n_rounds) gather(r + NB, 2, k0, k1);
            cp_async_commit();
        }
    }
    DSTAMP(4);

    // ---- deposit (max, sum, O) of the share in the first CTA of the cluster ----
    float o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        o[i] = (acc[0][i] + acc[1][i]) + (acc[2][i] + acc[3][i]);
        if (packed) o[i] += __shfl_xor_sync(0xffffffffu, o[i], 2);  // hi columns + lo columns
    }
    // the warps that share a slice add up through shared memory, in a fixed order
    if (kh > 0) *reinterpret_cast<float4*>(opart + ((kh - 1) * NSL + slice) * 128 + lane * 4) = make_float4(o[0], o[1], o[2], o[3]);
    __syncthreads();
    // the first CTA writes its own slot; the others send theirs with asynchronous stores that
    // count on its mbarrier, and are done: no fence, no closing cluster barrier
    const bool remote = rank != 0;
    float* mine = comb + rank * PS;
    const uint32_t mine_r = remote ? map_to_rank(smem_addr(mine), 0) : 0u;
    const uint32_t bar_r = remote ? map_to_rank(smem_addr(dep_bar), 0) : 0u;
    auto put = [&](int i, float v) {
        if (remote) st_async_f32(mine_r + 4 * i, v, bar_r);
        else mine[i] = v;
    };
    if (kh == 0) {
#pragma unroll
        for (int k = 1; k < KH; ++k) {
            const float4 t = *reinterpret_cast<const float4*>(opart + ((k - 1) * NSL + slice) * 128 + lane * 4);
            o[0] += t.x;
            o[1] += t.y;
            o[2] += t.z;
            o[3] += t.w;
        }
        const int d = slice * 16 + grp, g0 = 2 * quad;
        if (g0 < G) {
            put(g0 * D + d, o[0]);
            put(g0 * D + d + 8, o[2]);
        }
        if (g0 + 1 < G) {
            put((g0 + 1) * D + d, o[1]);
            put((g0 + 1) * D + d + 8, o[3]);
        }
    }
    if (warp == 0 && grp == 0) {
        if (2 * quad < G) {
            put(G * D + 2 * quad, M0);
            put(G * D + G + 2 * quad, L0);
        }
        if (2 * quad + 1 < G) {
            put(G * D + 2 * quad + 1, M1);
            put(G * D + G + 2 * quad + 1, L1);
        }
    }
    DSTAMP(5);
    if (remote) return;
    if (CS > 1) {  // every byte of the other CTAs has landed (bounded: a stall ends in a status code)
        const long long t_start = clock64();
        while (!mbar_try_wait(smem_addr(dep_bar), 0)) {
            if (clock64() - t_start > kTimeoutCycles) {
                set_status(status, SPEC_ERR_TIMEOUT);
                break;
            }
        }
    }
    __syncthreads();  // this CTA's own slot
    DSTAMP(6);
    // ---- merge the CTAs of the cluster, in rank order ----
    for (int i = tid; i < G * (D / 2); i += kThreads) {
        const int r = i / (D / 2), dp = i - r * (D / 2);
        float Mc[kMaxCluster], Lc[kMaxCluster];
        float2 oc[kMaxCluster];
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) {  // every load is in flight before the first is used
            if (c < CS) {
                const float* pc = comb + c * PS;
                Mc[c] = pc[G * D + r];
                Lc[c] = pc[G * D + G + r];
                oc[c] = *(reinterpret_cast<const float2*>(pc + r * D) + dp);
            }
        }
        float M = kNegBig;
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c)
            if (c < CS) M = fmaxf(M, Mc[c]);
        float Lsum = 0.f, o0 = 0.f, o1 = 0.f;
#pragma unroll
        for (int c = 0; c < kMaxCluster; ++c) {
            if (c < CS && Lc[c] > 0.f) {
                const float wgt = ex2f(Mc[c] - M);
                Lsum += Lc[c] * wgt;
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
    DSTAMP(7);
}

constexpr size_t kSmemLimit = 227 * 1024;

DraftShape make_shape(int D, int G, int keys, int cs)
{
    DraftShape s;
    s.cs = cs;
    s.packed = G <= 4;
    s.per = ((keys + cs - 1) / cs + 15) & ~15;
    s.rk = s.rows = s.per;  // the whole share resident: one round
    if (s.per > kCap || draft_smem_bytes(D, G, s) > kSmemLimit) {
        s.rk = kRound;  // several rounds through two buffers
        s.rows = 2 * kRound;
    }
    return s;
}

// Clusters of `cs` CTAs with `smem` bytes each that fit on the GPU at once (cached per size).
template <int D>
int max_active_clusters(int cs, size_t smem)
{
    static int cached[kMaxCluster + 1];
    static size_t cached_smem[kMaxCluster + 1];
    if (cached_smem[cs] == smem && cached[cs] > 0) return cached[cs];
    cudaLaunchConfig_t q = {};
    q.gridDim = dim3(cs, 1, sm_count());
    q.blockDim = dim3(kThreads);
    q.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = cs;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    q.attrs = at;
    q.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, draft_cluster_kernel<D>, &q) != cudaSuccess) {
        cudaGetLastError();
        n = sm_count() / cs;
    }
    cached[cs] = n;
    cached_smem[cs] = smem;
    return n;
}

template <int D>
bool set_smem_limit(size_t smem)
{
    static size_t configured = 0;  // per template instance: largest size opted in so far
    if (smem <= configured) return true;
    if (cudaFuncSetAttribute(draft_cluster_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return false;
    configured = smem;
    return true;
}

// Split of a call.  The cluster grows (1, 2, 4, 8 CTAs) while all CTAs still fit the SMs in one wave
// (a second wave could not start its gather under the first) and a CTA keeps about a round of keys.  A call that fits the GPU in one wave wants the
// next call's gather to run beside it (programmatic dependent launch), which needs both calls'
// clusters resident together; a GPC holds at most two clusters of eight and not every GPC
// does, so where 2 x clusters-per-call does not fit, clusters of six (which pack better) are
// used if the larger share still fits shared memory in one round.
template <int D>
bool draft_plan(const KvView& kv, int n_keys_max, DraftShape* out)
{
    const long probs = (long)kv.n_layers * kv.batch * kv.n_kv_heads;
    const int G = kv.n_q_heads / kv.n_kv_heads;
    const int keys = n_keys_max > 0 ? n_keys_max : 1;
    const int rounds = (keys + kRound - 1) / kRound;
    int cs = 1;
    while (cs < kMaxCluster && probs * cs * 2 <= sm_count() && cs < rounds) cs *= 2;  // one wave of CTAs at most
    DraftShape s = make_shape(D, G, keys, cs);
    if (!set_smem_limit<D>(kSmemLimit)) return false;
    if (cs == kMaxCluster && probs * cs <= sm_count() &&
        2 * probs > max_active_clusters<D>(cs, draft_smem_bytes(D, G, s))) {
        const DraftShape t = make_shape(D, G, keys, 6);
        if (t.rk == t.per && 2 * probs <= max_active_clusters<D>(6, draft_smem_bytes(D, G, t))) s = t;
    }
    *out = s;
    return true;
}

template <int D>
int launch_d(const DraftArgs& a, cudaStream_t stream)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    DraftShape shp;
    if (!draft_plan<D>(a.kv, a.k_total + a.max_tail, &shp)) return SPEC_ERR_CUDA;
#ifdef SPEC_TRACE
    if (const char* e = getenv("SPEC_DRAFT_CS")) shp = make_shape(D, G, a.k_total + a.max_tail, atoi(e));
    if (getenv("SPEC_DRAFT_UNPACKED")) shp.packed = 0;
#endif
    const size_t smem = draft_smem_bytes(D, G, shp);
    if (smem > kSmemLimit) return SPEC_ERR_UNSUPPORTED_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(shp.cs, a.kv.n_kv_heads, a.kv.n_layers * a.kv.batch);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = shp.cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see the kernel's prologue
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    if (cudaLaunchKernelEx(&cfg, draft_cluster_kernel<D>, a, shp, static_cast<int*>(a.workspace)) != cudaSuccess) {
        cudaGetLastError();
        return SPEC_ERR_CUDA;
    }
    count_launch(1);
    return SPEC_OK;
}

}  // namespace

size_t draft_workspace(const KvView&, int) { return kStatusBytes; }

int draft_launch(const DraftArgs& a, cudaStream_t stream)
{
    const int G = a.kv.n_q_heads / a.kv.n_kv_heads;
    if (G > kMaxGroup) return SPEC_ERR_UNSUPPORTED_SHAPE;
    if (a.workspace_bytes < kStatusBytes) return SPEC_ERR_WORKSPACE_TOO_SMALL;
    if (a.kv.head_dim == 128) return launch_d<128>(a, stream);
    if (a.kv.head_dim == 64) return launch_d<64>(a, stream);
    return SPEC_ERR_UNSUPPORTED_SHAPE;
}

}  // namespace spec
