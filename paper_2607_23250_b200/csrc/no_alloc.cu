// Backward entry point for callers that must not allocate device memory.
//
// Some callers cannot call cudaMalloc (or have torch do it) at the moment they need a backward
// pass: code running while a CUDA stream is being captured, code inside a memory-pool callback
// or under an allocator lock, and services that size all of their device memory at start-up and
// forbid later growth.  For them the row-statistics scratch that libra_attn_pool_bwd takes from
// the caller lives here, in a fixed array inside the library's device image.
#include <mutex>

#include "common.h"

namespace {

// Scratch for the two row statistics, D_i and LSE in log2 units: 2 x hq x round_up(T, 128) floats.
// 4 Mi floats = 16 MiB, enough for e.g. 32 query heads x 65536 tokens.  Every GPU whose context
// loads this library holds the array until the process exits.
constexpr size_t kMaxScratchFloats = size_t(4) << 20;
static __device__ __align__(256) float g_bwd_scratch[kMaxScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};

// The array's name is only a host-side handle; kernels need its device address, which is looked
// up once per device with that device current.
int scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return LIBRA_ERR_NO_DEVICE;
    if (dev < 0 || dev >= kMaxDevices) return LIBRA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_bwd_scratch) != cudaSuccess || !ptr) return LIBRA_ERR_CUDA;
        g_scratch_addr[dev] = ptr;
    }
    *out = g_scratch_addr[dev];
    return LIBRA_OK;
}

}  // namespace

extern "C" size_t libra_attn_pool_bwd_noalloc_max_bytes(void) { return kMaxScratchFloats * sizeof(float); }

extern "C" int libra_attn_pool_bwd_noalloc(const void* q_dev, const void* k_dev, const void* v_dev,
                                           const void* out_dev, const float* lse_dev, const void* dout_dev,
                                           const int32_t* cu_seqlens_dev, const libra_plan_t* plan, void* dq_dev,
                                           void* dk_dev, void* dv_dev, const libra_dims* dims, void* stream) {
    if (!plan || !dims) return LIBRA_ERR_INVALID_ARG;
    // the same verdicts, in the same order, as the regular entry point gives for bad dimensions
    if (dims->hq <= 0 || dims->hkv <= 0 || dims->hq % dims->hkv) return LIBRA_ERR_INVALID_ARG;
    if (dims->head_dim != 64 && dims->head_dim != 128 && dims->head_dim != 256) return LIBRA_ERR_UNSUPPORTED;
    const size_t need = libra_attn_pool_bwd_workspace_bytes(plan, dims);
    if (need == 0) return LIBRA_ERR_INVALID_ARG;
    if (need > kMaxScratchFloats * sizeof(float)) return LIBRA_ERR_SCRATCH_TOO_SMALL;
    void* scratch = nullptr;
    const int rc = scratch_address(&scratch);
    if (rc != LIBRA_OK) return rc;
    // Nothing in the scratch has to start at zero: the row-statistics kernel writes every element the
    // later kernels read, so whatever the previous call left behind is simply overwritten.
    return libra_attn_pool_bwd(q_dev, k_dev, v_dev, out_dev, lse_dev, dout_dev, cu_seqlens_dev, plan, dq_dev, dk_dev,
                               dv_dev, scratch, dims, stream);
}
