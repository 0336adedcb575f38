// Interface of the tcgen05 / TMA verification kernel (verify_sm100.cu).
#pragma once
#include "spec_common.cuh"

namespace spec {
bool verify_sm100_supported(const KvView& kv, int n_q);
size_t verify_sm100_workspace(const KvView& kv, int n_q, int max_ctx_len);
int verify_sm100_launch(const VerifyArgs& a, cudaStream_t stream);
}  // namespace spec
