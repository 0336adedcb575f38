// Recall selection of Eq. 4: sink + TopK over the middle span + recent, per (layer, sequence,
// KV head).  One CTA per problem.  The scores are sums of probabilities (finite, >= 0), so the
// fp32 bit pattern orders like the value and the K_mid-th largest is found by a three-pass
// radix select (11 + 11 + 10 bits) on the bit patterns; an ordered compaction then emits, in
// ascending position, everything above the threshold plus the lowest-position ties.
// The scores are swept twice when the threshold's first-digit bin fits in shared memory (the usual
// case): the second sweep marks every candidate above that bin in a position bitmap and keeps the
// bin's own candidates (score, position) in a list; the last two digits are decided on the list and
// the index set is read off the bitmap in position order.  Flat scores (a bin too full for the list)
// and contexts too long for the bitmap fall back to one sweep per digit plus one for an ordered
// compaction.
// The first pass's histogram (top 11 bits) may arrive from the verification kernel, which counts
// every score it writes: the positions outside the candidate span are taken out again here, the
// sweep over the scores is skipped, and the counts are cleared for the next round.
#include "spec_common.cuh"

namespace spec {

namespace {

constexpr int kThreads = 1024;
constexpr int kBins = kScoreBins;
static_assert(kBins == 2 * kThreads, "two bins per thread");
constexpr int kItems = 8;  // consecutive candidates per thread in the compaction sweep
constexpr int kCap = 6144; // candidates (score, position) kept in shared memory
constexpr int kMapWords = 4096;  // position bitmap: contexts up to 128 K keys
static_assert(kMapWords == 4 * kThreads, "at most four bitmap words per thread");
constexpr size_t kDynSmem = (size_t)(2 * kCap + kMapWords) * 4;

// Exclusive block-wide prefix sum of one int per thread; `total` gets the block sum.
__device__ __forceinline__ int block_exclusive_scan(int x, int* warp_tmp, int& total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += y;
    }
    __syncthreads();  // warp_tmp may still be read from a previous scan
    if (lane == 31) warp_tmp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tmp[lane];
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += y;
        }
        warp_tmp[lane] = winc - w;          // exclusive offset of each warp
        if (lane == 31) warp_tmp[32] = winc;  // block total
    }
    __syncthreads();
    total = warp_tmp[32];
    return warp_tmp[warp] + inc - x;
}

// Calls f(bits, position) for every candidate of [lo, hi): eight loads per thread are in flight before the first
// is used (a loop of one load and one atomic per trip would pay the memory latency on every trip).
template <typename F>
__device__ __forceinline__ void sweep(const uint32_t* __restrict__ st, int lo, int hi, F f)
{
    for (int base = lo + threadIdx.x; base < hi; base += 8 * kThreads) {
        uint32_t u[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) u[k] = base + k * kThreads < hi ? __ldg(st + base + k * kThreads) : 0u;
#pragma unroll
        for (int k = 0; k < 8; ++k)
            if (base + k * kThreads < hi) f(u[k], base + k * kThreads);
    }
}

__global__ void __launch_bounds__(kThreads, 2)  // two CTAs per SM: 32 registers per thread
select_recall_kernel(const float* __restrict__ stats, int64_t stat_stride, int batch, int n_kv_heads,
                     const int32_t* __restrict__ sel_len, int k_sink, int k_recent, int k_total,
                     int32_t* __restrict__ indices, int32_t* __restrict__ n_indices,
                     uint32_t* __restrict__ hist_g, const int32_t* __restrict__ hist_len)
{
    __shared__ int hist[kBins];
    __shared__ int warp_tmp[33];
    __shared__ int sh_bucket, sh_above, sh_count, list_n;
    extern __shared__ uint32_t dyn_smem[];
    uint32_t* list = dyn_smem;                                // [kCap] score bit patterns
    int* lpos = reinterpret_cast<int*>(dyn_smem + kCap);      // [kCap] their positions
    uint32_t* bitmap = dyn_smem + 2 * kCap;                   // [kMapWords] chosen positions

    const int64_t prob = blockIdx.x;
    const int b = (int)((prob / n_kv_heads) % batch);
    const int tid = threadIdx.x;
    // counts handed over by the verification kernel: requested first (two bins per thread), taken and
    // cleared whatever happens below
    uint32_t h0 = 0, h1 = 0;
    uint32_t* hg = hist_g ? hist_g + prob * kBins : nullptr;
    if (hg) {
        h0 = hg[tid];
        h1 = hg[tid + kThreads];
    }
    const int T = sel_len[b];
    const int HL = hg ? hist_len[b] : 0;
    int32_t* out = indices + prob * k_total;
    const uint32_t* st = reinterpret_cast<const uint32_t*>(stats + prob * stat_stride);
    // they cover positions [0, hist_len): usable if the candidate span lies inside.  The positions outside
    // the span that were counted (sink, recent window, rows beyond the committed length: a few dozen)
    // are fetched now and taken out of the counts below.
    const bool have_hist = hg && T <= HL && T > k_total;
    uint32_t excl = 0xffffffffu;
    if (have_hist && tid < k_sink + (HL - (T - k_recent)))
        excl = __ldg(st + (tid < k_sink ? tid : T - k_recent + (tid - k_sink))) >> 21;
    if (hg) {
        hist[tid] = (int)h0;
        hist[tid + kThreads] = (int)h1;
        hg[tid] = 0u;
        hg[tid + kThreads] = 0u;
        __syncthreads();
    }

    if (T <= k_total) {  // everything fits: keep every position
        for (int i = tid; i < k_total; i += kThreads) out[i] = i < T ? i : -1;
        if (tid == 0) n_indices[prob] = T > 0 ? T : 0;
        return;
    }
    const int lo = k_sink, hi = T - k_recent;  // candidate span [lo, hi), holds > k_mid entries
    const int k_mid = k_total - k_sink - k_recent;
    for (int i = tid; i < k_sink; i += kThreads) out[i] = i;
    for (int i = tid; i < k_recent; i += kThreads) out[k_sink + k_mid + i] = hi + i;
    if (tid == 0) n_indices[prob] = k_total;
    if (k_mid == 0) return;

    // ---- radix select: bit pattern `thr` of the k_mid-th largest candidate ----
    uint32_t prefix = 0, mask = 0;
    int need = k_mid;  // how many to take among candidates matching the decided prefix
    int n_list = 0;
    bool use_list = false;
    const bool map_ok = hi <= kMapWords * 32;
    const int map_words = map_ok ? (hi + 31) >> 5 : 0;
    const int wpt = (map_words + kThreads - 1) / kThreads;  // bitmap words per thread (consecutive ones)
    // walks the buckets of `hist` from the largest digit down (thread t owns reversed bins 2t, 2t+1) and
    // leaves the one in which the running count reaches `want`; false if the counts do not reach it
    auto find_bucket = [&](int nb, int want) -> bool {
        const int j0 = 2 * tid, j1 = 2 * tid + 1;
        const int c0 = j0 < nb ? hist[nb - 1 - j0] : 0;
        const int c1 = j1 < nb ? hist[nb - 1 - j1] : 0;
        int total;
        const int ex = block_exclusive_scan(c0 + c1, warp_tmp, total);
        if (ex < want && want <= ex + c0) {
            sh_bucket = nb - 1 - j0;
            sh_above = ex;
            sh_count = c0;
        } else if (ex + c0 < want && want <= ex + c0 + c1) {
            sh_bucket = nb - 1 - j1;
            sh_above = ex + c0;
            sh_count = c1;
        }
        __syncthreads();
        return total >= want;
    };
    for (int pass = 0; pass < 3; ++pass) {
        const int shift = pass == 0 ? 21 : (pass == 1 ? 10 : 0);
        const int nb = pass == 2 ? 1024 : 2048;
        if (pass == 0 && have_hist) {
            if (excl != 0xffffffffu) atomicSub(&hist[excl], 1);
            for (int i = tid + kThreads; i < lo + (HL - hi); i += kThreads) {  // (more than 1024 positions outside)
                const int pos = i < lo ? i : hi + (i - lo);
                atomicSub(&hist[__ldg(st + pos) >> 21], 1);
            }
        } else {
            for (int i = tid; i < kBins; i += kThreads) hist[i] = 0;
            __syncthreads();
            if (pass > 0 && use_list) {  // the candidates that share the first digit sit in shared memory
                for (int i = tid; i < n_list; i += kThreads) {
                    const uint32_t u = list[i];
                    if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & (nb - 1)], 1);
                }
            } else if (pass == 0) {
                // The first trip (8 K candidates) is counted in full; the bin in which ITS count reaches
                // k_mid bounds the threshold's bin from below, so the remaining trips count only what
                // lies at or above it: a few percent of the candidates instead of all of them (the
                // counts below the threshold's bin are never looked at).
                const int mid = min(hi, lo + 8 * kThreads);
                sweep(st, lo, mid, [&](uint32_t u, int) { atomicAdd(&hist[u >> 21], 1); });
                if (mid < hi) {
                    __syncthreads();
                    const uint32_t floor_bin = find_bucket(nb, need) ? (uint32_t)sh_bucket : 0u;
                    sweep(st, mid, hi, [&](uint32_t u, int) {
                        if ((u >> 21) >= floor_bin) atomicAdd(&hist[u >> 21], 1);
                    });
                }
            } else {
                sweep(st, lo, hi, [&](uint32_t u, int) {
                    if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & (nb - 1)], 1);
                });
            }
        }
        __syncthreads();
        find_bucket(nb, need);
        prefix |= (uint32_t)sh_bucket << shift;
        mask |= (uint32_t)(nb - 1) << shift;
        need -= sh_above;
        const int in_bucket = sh_count;
        __syncthreads();
        if (pass == 0 && in_bucket <= kCap) {
            // One sweep collects the candidates of the threshold's bin (usually a few hundred of the tens
            // of thousands) with their positions and marks everything above that bin in the position
            // bitmap; the two remaining digits are then decided on the list instead of by two more
            // sweeps over all scores.  A bin too full for the list (flat scores) keeps the sweeps.
            if (tid == 0) list_n = 0;
            for (int i = tid; i < map_words; i += kThreads) bitmap[i] = 0u;
            __syncthreads();
            const uint32_t bucket = prefix >> 21;
            sweep(st, lo, hi, [&](uint32_t u, int pos) {
                const uint32_t bin = u >> 21;
                if (bin == bucket) {
                    const int at = atomicAdd(&list_n, 1);
                    if (at < kCap) {
                        list[at] = u;
                        lpos[at] = pos;
                    }
                } else if (bin > bucket && map_ok) {
                    atomicOr(&bitmap[pos >> 5], 1u << (pos & 31));
                }
            });
            __syncthreads();
            n_list = list_n;
            use_list = n_list <= kCap;
        }
    }
    const uint32_t thr = prefix;  // take every candidate > thr and the first `need` equal to it

    bool off_map = use_list && map_ok;
    int n_eq = 0;
    int* eqpos = hist;  // the tie positions reuse the histogram's storage
    if (off_map) {
        // list entries above the threshold join the bitmap; the ties (bit pattern equal to the
        // threshold) are set aside
        if (tid == 0) list_n = 0;
        __syncthreads();
        for (int i = tid; i < n_list; i += kThreads) {
            const uint32_t u = list[i];
            const int pos = lpos[i];
            if (u > thr) {
                atomicOr(&bitmap[pos >> 5], 1u << (pos & 31));
            } else if (u == thr) {
                const int at = atomicAdd(&list_n, 1);
                if (at < kBins) eqpos[at] = pos;
            }
        }
        __syncthreads();
        n_eq = list_n;
        off_map = n_eq <= kBins;  // (thousands of equal scores: the ordered compaction below handles them)
    }
    if (off_map) {
        // ---- the index set off the bitmap ----
        // the ties are ranked by position among themselves and the lowest `need` join
        for (int i = tid; i < n_eq; i += kThreads) {
            const int pos = eqpos[i];
            int rank = 0;
            if (n_eq > need)
                for (int j = 0; j < n_eq; ++j) rank += eqpos[j] < pos ? 1 : 0;
            if (rank < need) atomicOr(&bitmap[pos >> 5], 1u << (pos & 31));
        }
        __syncthreads();
        uint32_t w[4];
        int cnt = 0;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            w[k] = (k < wpt && wpt * tid + k < map_words) ? bitmap[wpt * tid + k] : 0u;
            cnt += __popc(w[k]);
        }
        int total;
        int at = k_sink + block_exclusive_scan(cnt, warp_tmp, total);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t m = w[k];
            while (m) {
                const int bit = __ffs(m) - 1;
                m &= m - 1;
                out[at++] = (wpt * tid + k) * 32 + bit;
            }
        }
        return;
    }

    // ---- ordered compaction over the candidate span (flat scores or very long contexts) ----
    // One block scan per trip: the counts of "above the threshold" (high half) and "equal to it" (low
    // half) travel in one word; a candidate's slot is (candidates above it so far) + (equal ones so far,
    // capped at the number still needed).
    int gt_seen = 0, eq_seen = 0;
    for (int base = lo; base < hi; base += kThreads * kItems) {
        const int i0 = base + tid * kItems;
        uint32_t u[kItems];
        int packed = 0;
#pragma unroll
        for (int k = 0; k < kItems; ++k) {
            u[k] = (i0 + k < hi) ? __ldg(st + i0 + k) : 0u;
            if (i0 + k < hi) packed += u[k] > thr ? (1 << 16) : (u[k] == thr ? 1 : 0);
        }
        int total;
        const int ex = block_exclusive_scan(packed, warp_tmp, total);
        int gt = gt_seen + (ex >> 16), eq = eq_seen + (ex & 0xffff);
#pragma unroll
        for (int k = 0; k < kItems; ++k) {
            if (i0 + k < hi) {
                if (u[k] > thr) {
                    out[k_sink + gt + min(eq, need)] = i0 + k;
                    ++gt;
                } else if (u[k] == thr) {
                    if (eq < need) out[k_sink + gt + eq] = i0 + k;
                    ++eq;
                }
            }
        }
        gt_seen += total >> 16;
        eq_seen += total & 0xffff;
    }
}

// Top-11-bit counts of stats[prob][0 : len[b]) for the verification kernels that do not count while
// they write the statistic.
__global__ void __launch_bounds__(256)
score_hist_kernel(const float* __restrict__ stats, int64_t stat_stride, int batch, int heads,
                  const int32_t* __restrict__ len, int max_len, uint32_t* __restrict__ hist)
{
    const int64_t prob = blockIdx.y;
    const int b = (int)((prob / heads) % batch);
    const int T = min(max(len[b], 0), max_len);
    const uint32_t* st = reinterpret_cast<const uint32_t*>(stats + prob * stat_stride);
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < T; i += gridDim.x * blockDim.x)
        atomicAdd(hist + prob * kBins + (__ldg(st + i) >> 21), 1u);
}

}  // namespace

int select_launch(const float* stats, int64_t stat_stride, int n_layers, int batch, int n_kv_heads,
                  const int32_t* sel_len, int k_sink, int k_recent, int k_total, int32_t* indices,
                  int32_t* n_indices, uint32_t* hist, const int32_t* hist_len, cudaStream_t stream)
{
    const long probs = (long)n_layers * batch * n_kv_heads;
    static bool opted_in[64] = {};  // per device: the kernel's dynamic shared memory exceeds the default limit
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SPEC_ERR_CUDA;
    if (!opted_in[dev]) {
        if (cudaFuncSetAttribute(select_recall_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem) !=
            cudaSuccess)
            return SPEC_ERR_CUDA;
        opted_in[dev] = true;
    }
    select_recall_kernel<<<(unsigned)probs, kThreads, kDynSmem, stream>>>(
        stats, stat_stride, batch, n_kv_heads, sel_len, k_sink, k_recent, k_total, indices, n_indices, hist, hist_len);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

int score_hist_launch(const float* stats, int64_t stat_stride, long probs, int batch, int heads, const int32_t* len,
                      int max_len, uint32_t* hist, cudaStream_t stream)
{
    if (probs > 65535) return SPEC_ERR_UNSUPPORTED_SHAPE;
    const int bx = max_len > 256 * 16 ? 16 : (max_len + 255) / 256;
    score_hist_kernel<<<dim3(bx > 0 ? bx : 1, (unsigned)probs), 256, 0, stream>>>(stats, stat_stride, batch, heads, len,
                                                                                 max_len, hist);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

}  // namespace spec
