// C ABI of libnova_attn (see include/nova_attn.h): argument validation, TMA tensor-map encoding and
// caching, per-device set-up, kernel launches on the caller's stream.  No device allocation, no sync.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>

#include "../../include/nova_attn.h"
#include "kernels.h"

namespace nova {

__device__ int g_dev_status = 0;

namespace {

thread_local int t_last_cuda_error = 0;

int fail_cuda(int code) {
    t_last_cuda_error = code;
    return NOVA_ATTN_ERR_CUDA;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxDevices = 64;
struct DeviceState {
    bool ready = false;
    int status = NOVA_ATTN_OK;  // sticky result of the one-time set-up
    int num_sms = 0;
    int* dev_status = nullptr;
};
std::mutex g_mutex;
DeviceState g_devices[kMaxDevices];
EncodeTiledFn g_encode = nullptr;

// One-time set-up of the current device: capability check, opt-in shared memory sizes, address of
// the device status word, tensor-map encoder entry point.
int device_state(DeviceState** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail_cuda(e);
    if (dev < 0 || dev >= kMaxDevices) return NOVA_ATTN_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mutex);
    DeviceState& st = g_devices[dev];
    if (!st.ready) {
        st.ready = true;
        int major = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) { st.status = fail_cuda(e); return st.status; }
        if (major != 10) { st.status = NOVA_ATTN_ERR_UNSUPPORTED; return st.status; }
        e = cudaDeviceGetAttribute(&st.num_sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) { st.status = fail_cuda(e); return st.status; }
        if (g_encode == nullptr) {
            void* fn = nullptr;
            cudaDriverEntryPointQueryResult qres;
            e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
            if (e != cudaSuccess || fn == nullptr || qres != cudaDriverEntryPointSuccess) {
                st.status = fail_cuda(e != cudaSuccess ? e : cudaErrorSymbolNotFound);
                return st.status;
            }
            g_encode = reinterpret_cast<EncodeTiledFn>(fn);
        }
        e = configure_attn_fwd();
        if (e == cudaSuccess) e = configure_attn_bwd();
        if (e == cudaSuccess) e = configure_attn_delta();
        if (e == cudaSuccess) e = cudaGetSymbolAddress(reinterpret_cast<void**>(&st.dev_status), g_dev_status);
        if (e != cudaSuccess) { st.status = fail_cuda(e); return st.status; }
    }
    if (st.status != NOVA_ATTN_OK) return st.status;
    *out = &st;
    return NOVA_ATTN_OK;
}

// Tensor maps are pure functions of (pointer, D, T, B*H); a small cache keeps the host cost of a
// call to a lookup when the same buffers are used step after step.
struct MapKey {
    const void* ptr;
    int D, T, BH, dev, elem_bytes;
};
struct MapEntry {
    MapKey key{};
    bool valid = false;
    CUtensorMap map;
};
constexpr int kMapCache = 128;
MapEntry g_maps[kMapCache];

// elem_bytes 2: bf16 tensor, box [64, 128, 1]; elem_bytes 4: fp32 tensor, box [32, 128, 1].
int get_tensor_map(const void* ptr, int D, long long T, long long BH, CUtensorMap* out, int elem_bytes = 2) {
    int dev = 0;
    cudaGetDevice(&dev);
    const MapKey key{ptr, D, static_cast<int>(T), static_cast<int>(BH), dev, elem_bytes};
    const uint64_t h = (reinterpret_cast<uint64_t>(ptr) >> 8) * 0x9E3779B97F4A7C15ull + uint64_t(T) * 31 + uint64_t(BH) * 131 + D;
    std::lock_guard<std::mutex> lock(g_mutex);
    MapEntry& e = g_maps[(h >> 32) % kMapCache];
    if (e.valid && e.key.ptr == key.ptr && e.key.D == key.D && e.key.T == key.T && e.key.BH == key.BH &&
        e.key.dev == key.dev && e.key.elem_bytes == key.elem_bytes) {
        *out = e.map;
        return NOVA_ATTN_OK;
    }
    // [D, T, B*H], D contiguous; 128-byte box rows; rows past T read as zero and are clipped on writes.
    const cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(T), cuuint64_t(BH)};
    const cuuint64_t strides[2] = {cuuint64_t(D) * elem_bytes, cuuint64_t(T) * cuuint64_t(D) * elem_bytes};
    const cuuint32_t box[3] = {cuuint32_t(128 / elem_bytes), cuuint32_t(kBlockQ), 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUtensorMap m;
    const CUresult r = g_encode(&m, elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                                3, const_cast<void*>(ptr), dims, strides, box,
                                estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
    e.key = key;
    e.map = m;
    e.valid = true;
    *out = m;
    return NOVA_ATTN_OK;
}

// Workspace of the backward: the fp32 dQ accumulator [B,H,T,D], rounded up to 256 bytes.
size_t acc_bytes(int B, int H, int T, int D) {
    const size_t n = static_cast<size_t>(B) * H * T * D * sizeof(float);
    return (n + 255) & ~size_t(255);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_shape(int B, int H, int T, int D) {
    if (B <= 0 || H <= 0 || T <= 0) return NOVA_ATTN_ERR_SHAPE;
    if (D != 64 && D != 128) return NOVA_ATTN_ERR_UNSUPPORTED;
    const long long bh = static_cast<long long>(B) * H;
    // grid = tiles * B*H must fit a 1-D grid; rows must fit 32-bit tile arithmetic
    const long long tiles = (static_cast<long long>(T) + kBlockQ - 1) / kBlockQ;
    if (bh > (1ll << 30) || bh * tiles > 2147483647ll || static_cast<long long>(T) > (1ll << 30)) return NOVA_ATTN_ERR_SHAPE;
    return NOVA_ATTN_OK;
}

}  // namespace
}  // namespace nova

using namespace nova;

extern "C" {

int nova_attn_fwd(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int H, int T, int D,
                  float scale, int causal, void* stream) {
    if (!Q || !K || !V || !O || !LSE) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_shape(B, H, T, D)) return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE)) return NOVA_ATTN_ERR_ALIGNMENT;
    if (!std::isfinite(scale) || !(scale > 0.f)) return NOVA_ATTN_ERR_SCALE;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const long long BH = static_cast<long long>(B) * H;
    CUtensorMap tmQ, tmK, tmV, tmO;
    if (int rc = get_tensor_map(Q, D, T, BH, &tmQ)) return rc;
    if (int rc = get_tensor_map(K, D, T, BH, &tmK)) return rc;
    if (int rc = get_tensor_map(V, D, T, BH, &tmV)) return rc;
    if (int rc = get_tensor_map(O, D, T, BH, &tmO)) return rc;
    const AttnShape s{B, H, T, D, causal != 0, scale};
    const cudaError_t e = launch_attn_fwd(tmQ, tmK, tmV, tmO, LSE, s, st->num_sms, st->dev_status,
                                          static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NOVA_ATTN_OK : fail_cuda(e);
}

int nova_attn_bwd_preprocess(const void* O, const void* dO, float* Delta, int B, int H, int T, int D, void* stream) {
    if (!O || !dO || !Delta) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_shape(B, H, T, D)) return rc;
    if (!aligned16(O) || !aligned16(dO) || !aligned16(Delta)) return NOVA_ATTN_ERR_ALIGNMENT;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const long long rows = static_cast<long long>(B) * H * T;
    const cudaError_t e =
        launch_attn_bwd_preprocess(static_cast<const __nv_bfloat16*>(O), static_cast<const __nv_bfloat16*>(dO), Delta,
                                   rows, D, st->num_sms, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NOVA_ATTN_OK : fail_cuda(e);
}

int nova_attn_bwd_preprocess_exact(const void* Q, const void* K, const void* V, const void* dO, const float* LSE,
                                   float* Delta, int B, int H, int T, int D, float scale, int causal, void* stream) {
    if (!Q || !K || !V || !dO || !LSE || !Delta) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_shape(B, H, T, D)) return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(LSE) || !aligned16(Delta))
        return NOVA_ATTN_ERR_ALIGNMENT;
    if (!std::isfinite(scale) || !(scale > 0.f)) return NOVA_ATTN_ERR_SCALE;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const long long BH = static_cast<long long>(B) * H;
    CUtensorMap tmQ, tmK, tmV, tmdO;
    if (int rc = get_tensor_map(Q, D, T, BH, &tmQ)) return rc;
    if (int rc = get_tensor_map(K, D, T, BH, &tmK)) return rc;
    if (int rc = get_tensor_map(V, D, T, BH, &tmV)) return rc;
    if (int rc = get_tensor_map(dO, D, T, BH, &tmdO)) return rc;
    const AttnShape s{B, H, T, D, causal != 0, scale};
    const cudaError_t e =
        launch_attn_delta(tmQ, tmK, tmV, tmdO, LSE, Delta, s, st->dev_status, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NOVA_ATTN_OK : fail_cuda(e);
}

size_t nova_attn_bwd_workspace_bytes(int B, int H, int T, int D) {
    if (check_shape(B, H, T, D) != NOVA_ATTN_OK) return 0;
    return acc_bytes(B, H, T, D);
}

int nova_attn_bwd_steps(const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* LSE,
                        const float* Delta, void* dQ, void* dK, void* dV, int B, int H, int T, int D, float scale,
                        int causal, void* workspace, size_t workspace_bytes, void* stream, int steps) {
    (void)O;  // Delta already carries rowsum(dO * O)
    if (!Q || !K || !V || !dO || !LSE || !Delta || !dQ || !dK || !dV) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_shape(B, H, T, D)) return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(LSE) || !aligned16(Delta) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
        return NOVA_ATTN_ERR_ALIGNMENT;
    if (!std::isfinite(scale) || !(scale > 0.f)) return NOVA_ATTN_ERR_SCALE;
    const size_t need = nova_attn_bwd_workspace_bytes(B, H, T, D);
    if (!workspace || workspace_bytes < need) return NOVA_ATTN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return NOVA_ATTN_ERR_ALIGNMENT;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const long long BH = static_cast<long long>(B) * H;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    float* acc = static_cast<float*>(workspace);
    cudaError_t e = cudaSuccess;
    if (steps & NOVA_ATTN_BWD_STEP_ZERO) {
        e = launch_zero(acc, need, st->num_sms, cs);
        if (e != cudaSuccess) return fail_cuda(e);
    }
    if (steps & NOVA_ATTN_BWD_STEP_MAIN) {
        CUtensorMap tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV;
        if (int rc = get_tensor_map(Q, D, T, BH, &tmQ)) return rc;
        if (int rc = get_tensor_map(K, D, T, BH, &tmK)) return rc;
        if (int rc = get_tensor_map(V, D, T, BH, &tmV)) return rc;
        if (int rc = get_tensor_map(dO, D, T, BH, &tmdO)) return rc;
        if (int rc = get_tensor_map(acc, D, T, BH, &tmAcc, 4)) return rc;
        if (int rc = get_tensor_map(dK, D, T, BH, &tmdK)) return rc;
        if (int rc = get_tensor_map(dV, D, T, BH, &tmdV)) return rc;
        const AttnShape s{B, H, T, D, causal != 0, scale};
        e = launch_attn_bwd(tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, LSE, Delta, static_cast<__nv_bfloat16*>(dK),
                            static_cast<__nv_bfloat16*>(dV), s, st->num_sms, st->dev_status, cs);
        if (e != cudaSuccess) return fail_cuda(e);
    }
    if (steps & NOVA_ATTN_BWD_STEP_CONVERT) {
        e = launch_dq_convert(acc, static_cast<__nv_bfloat16*>(dQ), static_cast<long long>(B) * H * T * D, scale,
                              st->num_sms, cs);
        if (e != cudaSuccess) return fail_cuda(e);
    }
    return NOVA_ATTN_OK;
}

int nova_attn_bwd(const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* LSE,
                  const float* Delta, void* dQ, void* dK, void* dV, int B, int H, int T, int D, float scale,
                  int causal, void* workspace, size_t workspace_bytes, void* stream) {
    return nova_attn_bwd_steps(Q, K, V, O, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, scale, causal, workspace,
                               workspace_bytes, stream,
                               NOVA_ATTN_BWD_STEP_ZERO | NOVA_ATTN_BWD_STEP_MAIN | NOVA_ATTN_BWD_STEP_CONVERT);
}

const char* nova_attn_status_string(int status) {
    switch (status) {
        case NOVA_ATTN_OK: return "ok";
        case NOVA_ATTN_ERR_NULL: return "a required pointer is NULL";
        case NOVA_ATTN_ERR_SHAPE: return "B, H, T must be positive and within the supported range";
        case NOVA_ATTN_ERR_UNSUPPORTED: return "unsupported head dimension (need 64 or 128) or device (need sm_100)";
        case NOVA_ATTN_ERR_ALIGNMENT: return "a tensor pointer is not 16-byte aligned";
        case NOVA_ATTN_ERR_SCALE: return "scale must be finite and > 0";
        case NOVA_ATTN_ERR_WORKSPACE: return "workspace is NULL or too small";
        case NOVA_ATTN_ERR_CUDA: return "a CUDA call failed (see nova_attn_last_cuda_error)";
        case NOVA_ATTN_ERR_TIMEOUT: return "a bounded device-side wait expired; outputs are invalid";
        default: return "unknown status";
    }
}

int nova_attn_last_cuda_error(void) { return t_last_cuda_error; }

int nova_attn_poll_device_status(void* stream) {
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaStreamSynchronize(cs);
    if (e != cudaSuccess) return fail_cuda(e);
    int word = 0;
    e = cudaMemcpy(&word, st->dev_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return fail_cuda(e);
    if (word != 0) {
        const int zero = 0;
        e = cudaMemcpy(st->dev_status, &zero, sizeof(int), cudaMemcpyHostToDevice);
        if (e != cudaSuccess) return fail_cuda(e);
        return NOVA_ATTN_ERR_TIMEOUT;
    }
    return NOVA_ATTN_OK;
}

}  // extern "C"
