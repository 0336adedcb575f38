// tcgen05 / TMA verification kernel (placeholder until the fast path lands).
#include "verify_sm100.cuh"

namespace spec {
bool verify_sm100_supported(const KvView&, int) { return false; }
size_t verify_sm100_workspace(const KvView&, int, int) { return 0; }
int verify_sm100_launch(const VerifyArgs&, cudaStream_t) { return SPEC_ERR_UNSUPPORTED_SHAPE; }
}  // namespace spec
