// Backward entry point for callers that cannot allocate device memory.  See include/bpt.h.
#include <mutex>

#include "bpt_internal.cuh"

namespace {

constexpr size_t kStaticScratchBytes = (size_t)32 << 20;  // 32 MiB per device that loads the library
constexpr int kMaxDevices = 64;

// The scratch itself.  In host code this name is only a handle for the runtime's symbol
// calls, never an address a kernel may be given; device_scratch() below asks the runtime
// for the real device address once per device.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices];
bool g_scratch_ready[kMaxDevices];

// Device address of the array on the current device (set-up on the first call per device).
bpt_status device_scratch(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BPT_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_ready[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return BPT_ERR_CUDA;
        g_scratch_addr[dev] = p;
        g_scratch_ready[dev] = true;
    }
    *out = g_scratch_addr[dev];
    return BPT_OK;
}

}  // namespace

extern "C" size_t bpt_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" bpt_status bpt_attn_bwd_static_scratch(const bpt_graph* g, int32_t B, int32_t H, int32_t d, bpt_dtype dtype,
                                                  const void* q, const void* k, const void* v, const void* rel_emb,
                                                  float scale, const void* out, const float* lse, const void* d_out,
                                                  void* dq, void* dk, void* dv, float* d_rel, void* cuda_stream) {
    if (!g) return BPT_ERR_INVALID_ARG;
    // The tiled backward works through the (batch entry, head) pairs in as many passes as the array's size
    // dictates; only a problem whose single pair does not fit is refused.
    const size_t need = bpt_attn_bwd_min_workspace_bytes(g, B, H, d, dtype);
    if (need > kStaticScratchBytes) return BPT_ERR_SCRATCH_LIMIT;
    void* scratch = nullptr;
    const bpt_status s = device_scratch(&scratch);
    if (s != BPT_OK) return s;
    // Every byte of the scratch that the backward reads it has written earlier in the same
    // call, so nothing has to be cleared although the previous call's contents are still there.
    return bpt_attn_bwd(g, B, H, d, dtype, q, k, v, rel_emb, scale, out, lse, d_out, dq, dk, dv, d_rel,
                        scratch, kStaticScratchBytes, cuda_stream);
}
