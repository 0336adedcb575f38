// spec_verify_attn_noalloc: verification attention for callers that cannot provide a workspace.
//
// Some hosts of this library never get to call cudaMalloc themselves: a plugin that is handed
// its input and output buffers by a runtime that owns all device memory, or code that runs
// after the framework's memory pool has taken the whole GPU.  For them the scratch that
// spec_verify_attn needs (cross-CTA counters, per-CTA partial outputs) lives in a fixed array
// inside the library image, kStaticScratchBytes per GPU, present on every device that loads the
// library until the process exits.
#include <mutex>

#include "spec_common.cuh"

namespace {

constexpr size_t kStaticScratchBytes = 16u << 20;  // 16 MiB: one layer of the 8B shape at 32K context needs 11 MiB
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress: it is not a device address.
static __device__ __align__(256) unsigned char g_scratch[kStaticScratchBytes];

std::mutex g_mutex;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up once per device).
int scratch_address(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return SPEC_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return SPEC_ERR_CUDA;
        }
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return SPEC_OK;
}

}  // namespace

extern "C" {

size_t spec_noalloc_scratch_bytes(void) { return kStaticScratchBytes; }

int spec_verify_attn_noalloc(const spec_kv_t* kv, const void* q, int32_t n_q, const int32_t* ctx_len,
                             int32_t max_ctx_len, int32_t stat_window, float* out, float* lse, float* stats,
                             int64_t stat_stride, void* cuda_stream)
{
    const size_t need = spec_workspace_bytes(SPEC_WS_VERIFY, kv, n_q, max_ctx_len, 1);
    if (need == 0) return SPEC_ERR_INVALID_ARG;
    if (need > kStaticScratchBytes) return SPEC_ERR_WORKSPACE_TOO_SMALL;  // shape too large for the built-in scratch
    void* scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != SPEC_OK) return rc;
    // The array keeps whatever the previous call left (possibly laid out for another shape): the
    // cross-CTA counters behind the status block (at most two per (layer, sequence, KV head) plus
    // one) must start at zero.  The status word itself is left alone, so that an error nobody has
    // read yet survives until spec_noalloc_read_status(), as with a caller's workspace.
    size_t head = (2 * (size_t)kv->n_layers * kv->batch * kv->n_kv_heads + 1) * sizeof(int) + 256;
    if (spec::kStatusBytes + head > need) head = need > spec::kStatusBytes ? need - spec::kStatusBytes : 0;
    if (head > 0 && cudaMemsetAsync(static_cast<char*>(scratch) + spec::kStatusBytes, 0, head,
                                    static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return SPEC_ERR_CUDA;
    return spec_verify_attn(kv, q, n_q, ctx_len, max_ctx_len, stat_window, out, lse, stats, stat_stride, scratch,
                            kStaticScratchBytes, cuda_stream);
}

int spec_noalloc_read_status(void* cuda_stream)
{
    void* scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != SPEC_OK) return rc;
    return spec_read_status(scratch, cuda_stream);
}

}  // extern "C"
