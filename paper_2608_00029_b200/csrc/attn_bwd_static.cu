// nova_attn_bwd_static_scratch: the backward pass for callers that cannot allocate device memory.
//
// nova_attn_bwd needs an fp32 dQ accumulator that the caller normally allocates.  Some callers have
// no allocator to ask: code running inside a framework's static memory plan, a plugin that is handed
// only its input and output buffers, a real-time loop that must not call cudaMalloc after start-up.
// For them the accumulator lives in the fixed array below, which is part of the library image: every
// GPU on which the library's device code has been loaded holds these 32 MiB until the process exits.
// (The CUDA runtime loads device code lazily by default: the array is then materialised by the first
// call of this entry point on a device, not when the shared object is opened.)
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/nova_attn.h"
#include "kernels.h"

namespace {

constexpr size_t kStaticScratchFloats = size_t(8) << 20;  // 8 Mi floats = 32 MiB
constexpr size_t kStaticScratchBytes = kStaticScratchFloats * sizeof(float);

// In host code this name is only a handle for the runtime, not a device address: it must never be
// passed to a kernel or a memset.  The address the GPU sees comes from cudaGetSymbolAddress below.
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
float* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of the array on the current device, looked up once per device.
cudaError_t static_scratch_address(float** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (g_scratch_addr[dev] == nullptr) {
        float* p = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" {

size_t nova_attn_static_scratch_bytes(void) { return kStaticScratchBytes; }

int nova_attn_bwd_static_scratch(const void* Q, const void* K, const void* V, const void* O, const void* dO,
                                 const float* LSE, const float* Delta, void* dQ, void* dK, void* dV, int B, int H,
                                 int T, int D, float scale, int causal, void* stream) {
    // Same order of checks as nova_attn_bwd: the arguments first, then the size of the accumulator.
    if (int rc = nova::validate_bwd_args(Q, K, V, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, scale)) return rc;
    if (nova_attn_bwd_workspace_bytes(B, H, T, D) > kStaticScratchBytes) return NOVA_ATTN_ERR_WORKSPACE;
    float* scratch = nullptr;
    const cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return nova::record_cuda_error(static_cast<int>(e));
    // Same kernels as nova_attn_bwd; it clears the part of the accumulator it uses on `stream` first,
    // so whatever the previous call left in the array does not matter.
    return nova_attn_bwd(Q, K, V, O, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, scale, causal, scratch,
                         kStaticScratchBytes, stream);
}

}  // extern "C"
