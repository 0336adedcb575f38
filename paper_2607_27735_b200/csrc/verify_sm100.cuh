// Interface of the sm_100a (tcgen05 / TMA) verification path (verify_sm100.cu).
#pragma once
#include "spec_common.cuh"

namespace spec {
// variant: 0 = automatic (score-cache kernel when a CTA's share of keys fits tensor memory,
// else the two-sweep kernel), 1 = two-sweep only, 2 = score-cache only
bool verify_sm100_supported(const KvView& kv, int n_q, int variant);
size_t verify_sm100_workspace(const KvView& kv, int n_q, int max_ctx_len);
// Clears the status word itself; *used_variant gets 1 (two-sweep) or 2 (score-cache).
int verify_sm100_launch(const VerifyArgs& a, int variant, cudaStream_t stream, int* used_variant);
// whether that call would accept the arguments (nothing is launched)
bool verify_sm100_can_run(const VerifyArgs& a, int variant);
// What AUTO would launch for this shape: out = {kernel (0 none, 1 two-sweep, 2 score-cache, 3 score-cache on two
// halves of the rows), KV heads per unit, CTAs per head, units, score columns, cached tiles, K/V slots, P buffers}.
void verify_sm100_describe(const KvView& kv, int n_q, int max_ctx_len, int32_t out[8]);

}  // namespace spec
