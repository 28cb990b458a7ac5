// C ABI of libnova_attn (see include/nova_attn.h): argument validation, TMA tensor-map encoding and
// caching, per-device set-up, kernel launches on the caller's stream.  No device allocation, no sync.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>

#include "../../include/nova_attn.h"
#include "../../include/nova_lmhead.h"
#include "kernels.h"
#include "work_plan.h"

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
// Test aid (nova_attn_test_configure_waits): cycle limit of the device-side waits and the fault to inject.
constexpr long long kDefaultWaitLimit = 1ll << 29;
std::atomic<long long> g_wait_limit{kDefaultWaitLimit};
std::atomic<int> g_inject{0};
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
        if (e == cudaSuccess) e = configure_attn_dq();
        if (e == cudaSuccess) e = configure_lmhead();
        if (e == cudaSuccess) e = cudaGetSymbolAddress(reinterpret_cast<void**>(&st.dev_status), g_dev_status);
        if (e != cudaSuccess) { st.status = fail_cuda(e); return st.status; }
    }
    if (st.status != NOVA_ATTN_OK) return st.status;
    *out = &st;
    return NOVA_ATTN_OK;
}

// Tensor maps are pure functions of (pointer, shape, strides); a small cache keeps the host cost of a
// call to a lookup when the same buffers are used step after step.
struct MapKey {
    const void* ptr;
    int D, T, BH, dev, elem_bytes;
    long long st, sh;
};
struct MapEntry {
    MapKey key{};
    bool valid = false;
    CUtensorMap map;
};
constexpr int kMapCache = 128;
MapEntry g_maps[kMapCache];

// 3-D map [D, T, B*H] of a tensor whose heads and batches merge into one dimension of stride `sh`
// elements (0: contiguous, sh = T*D) with token stride `st` (0: D).
// elem_bytes 2: bf16 tensor, box [64, 128, 1]; elem_bytes 4: fp32 tensor, box [32, 128, 1].
int get_tensor_map(const void* ptr, int D, long long T, long long BH, CUtensorMap* out, int elem_bytes = 2,
                   long long st = 0, long long sh = 0) {
    int dev = 0;
    cudaGetDevice(&dev);
    if (st == 0) st = D;
    if (sh == 0) sh = T * D;
    const MapKey key{ptr, D, static_cast<int>(T), static_cast<int>(BH), dev, elem_bytes, st, sh};
    const uint64_t h = (reinterpret_cast<uint64_t>(ptr) >> 8) * 0x9E3779B97F4A7C15ull + uint64_t(T) * 31 + uint64_t(BH) * 131 + D;
    std::lock_guard<std::mutex> lock(g_mutex);
    MapEntry& e = g_maps[(h >> 32) % kMapCache];
    if (e.valid && e.key.ptr == key.ptr && e.key.D == key.D && e.key.T == key.T && e.key.BH == key.BH &&
        e.key.dev == key.dev && e.key.elem_bytes == key.elem_bytes && e.key.st == key.st && e.key.sh == key.sh) {
        *out = e.map;
        return NOVA_ATTN_OK;
    }
    // [D, T, B*H], D contiguous; 128-byte box rows; rows past T read as zero and are clipped on writes.
    const cuuint64_t dims[3] = {cuuint64_t(D), cuuint64_t(T), cuuint64_t(BH)};
    const cuuint64_t strides[2] = {cuuint64_t(st) * elem_bytes, cuuint64_t(sh) * elem_bytes};
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

// 4-D map of a bf16 tensor indexed [b, h, t, d] with strides `st` (elements): dimensions [D, x, y, z] where
// x, y, z are token / head / batch in order of increasing stride (the encoder wants that), box 64 x 128
// tokens.  `*order` receives which of the three sits where (the code tma_order_coords understands).
struct Map4Key {
    const void* ptr;
    int D, T, H, B, dev;
    long long sb, sh, st;
};
struct Map4Entry {
    Map4Key key{};
    bool valid = false;
    int order = 0;
    CUtensorMap map;
};
Map4Entry g_maps4[kMapCache];

int get_tensor_map4(const void* ptr, const AttnShape& s, const TensorStrides& st, CUtensorMap* out, uint32_t* order) {
    int dev = 0;
    cudaGetDevice(&dev);
    const Map4Key key{ptr, s.D, s.T, s.H, s.B, dev, st.b, st.h, st.t};
    const uint64_t h = (reinterpret_cast<uint64_t>(ptr) >> 8) * 0x9E3779B97F4A7C15ull + uint64_t(s.T) * 31 +
                       uint64_t(s.B) * 131 + uint64_t(s.H) * 17 + uint64_t(st.t) * 7 + s.D;
    std::lock_guard<std::mutex> lock(g_mutex);
    Map4Entry& e = g_maps4[(h >> 32) % kMapCache];
    if (e.valid && e.key.ptr == key.ptr && e.key.D == key.D && e.key.T == key.T && e.key.H == key.H &&
        e.key.B == key.B && e.key.dev == key.dev && e.key.sb == key.sb && e.key.sh == key.sh && e.key.st == key.st) {
        *out = e.map;
        *order = static_cast<uint32_t>(e.order);
        return NOVA_ATTN_OK;
    }
    // which: 0 = token, 1 = head, 2 = batch; sorted by stride (ties keep token < head < batch)
    int which[3] = {0, 1, 2};
    const long long stride_of[3] = {st.t, st.h, st.b};
    const int extent_of[3] = {s.T, s.H, s.B};
    for (int i = 1; i < 3; ++i)
        for (int j = i; j > 0 && stride_of[which[j]] < stride_of[which[j - 1]]; --j) {
            const int tmp = which[j];
            which[j] = which[j - 1];
            which[j - 1] = tmp;
        }
    static const int kCodes[3][3] = {{-1, 0, 2}, {1, -1, 4}, {3, 5, -1}};  // [which[0]][which[1]] -> order code
    const int code = kCodes[which[0]][which[1]];
    cuuint64_t dims[4] = {cuuint64_t(s.D), 0, 0, 0};
    cuuint64_t strides[3];
    cuuint32_t box[4] = {cuuint32_t(kBoxCols), 1, 1, 1};
    for (int i = 0; i < 3; ++i) {
        dims[1 + i] = cuuint64_t(extent_of[which[i]]);
        strides[i] = cuuint64_t(stride_of[which[i]]) * sizeof(__nv_bfloat16);
        if (which[i] == 0) box[1 + i] = cuuint32_t(kBlockQ);
    }
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMap m;
    const CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail_cuda(static_cast<int>(r));
    e.key = key;
    e.map = m;
    e.order = code;
    e.valid = true;
    *out = m;
    *order = static_cast<uint32_t>(code);
    return NOVA_ATTN_OK;
}

// 2-D map of a row-major bf16 matrix [rows, cols] (cols contiguous): dimensions [cols, rows], box
// [box_cols, box_rows], 128-byte swizzle; elements outside the matrix read as zeros.
int encode_matrix_map(const void* ptr, long long rows, long long cols, int box_rows, int box_cols, CUtensorMap* out) {
    const cuuint64_t dims[2] = {cuuint64_t(cols), cuuint64_t(rows)};
    const cuuint64_t strides[1] = {cuuint64_t(cols) * sizeof(__nv_bfloat16)};
    const cuuint32_t box[2] = {cuuint32_t(box_cols), cuuint32_t(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = g_encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? NOVA_ATTN_OK : fail_cuda(static_cast<int>(r));
}

int check_lmhead_shape(int M, int N, int K) {
    if (M <= 0 || N <= 0 || K <= 0 || (K & 7) || (N & 7)) return NOVA_ATTN_ERR_SHAPE;
    if (M > (1 << 28) || N > (1 << 28) || K > (1 << 20)) return NOVA_ATTN_ERR_SHAPE;
    return NOVA_ATTN_OK;
}

// Heads and batches of the tensor merge into one dimension (the [B,H,T,D] family): 3-D maps, plain kernels.
bool merges(const AttnShape& s, const TensorStrides& st) {
    return st.b == static_cast<long long>(s.H) * st.h && st.t <= st.h;
}

// The map of a bf16 tensor for the plain (3-D) or the strided (4-D) build of the kernels.
int get_bf16_map(const void* ptr, const AttnShape& s, const TensorStrides& st, bool strided, CUtensorMap* out,
                 uint32_t* order) {
    if (strided) return get_tensor_map4(ptr, s, st, out, order);
    *order = 0;
    return get_tensor_map(ptr, s.D, s.T, static_cast<long long>(s.B) * s.H, out, 2, st.t, st.h);
}

TensorStrides contiguous_strides(int H, int T, int D) {
    return TensorStrides{static_cast<long long>(H) * T * D, static_cast<long long>(T) * D, static_cast<long long>(D)};
}

// Strides are in elements; every one a multiple of 8 (16 bytes, which TMA and the 16-byte accesses of the
// helper kernels need), the token stride at least D, none so large that a byte offset leaves 2^40.
int check_strides(const nova_attn_strides* p, int D, TensorStrides* out) {
    if (!p) return NOVA_ATTN_ERR_NULL;
    if ((p->batch & 7) || (p->head & 7) || (p->token & 7)) return NOVA_ATTN_ERR_ALIGNMENT;
    if (p->token < D || p->head < 8 || p->batch < 8) return NOVA_ATTN_ERR_SHAPE;
    const long long lim = (1ll << 39);
    if (p->token >= lim || p->head >= lim || p->batch >= lim) return NOVA_ATTN_ERR_SHAPE;
    *out = TensorStrides{p->batch, p->head, p->token};
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

int record_cuda_error(int code) { return fail_cuda(code); }

int validate_bwd_args(const void* Q, const void* K, const void* V, const void* dO, const float* LSE,
                      const float* Delta, const void* dQ, const void* dK, const void* dV, int B, int H, int T, int D,
                      float scale) {
    if (!Q || !K || !V || !dO || !LSE || !Delta || !dQ || !dK || !dV) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_shape(B, H, T, D)) return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(dO) || !aligned16(LSE) || !aligned16(Delta) ||
        !aligned16(dQ) || !aligned16(dK) || !aligned16(dV))
        return NOVA_ATTN_ERR_ALIGNMENT;
    if (!std::isfinite(scale) || !(scale > 0.f)) return NOVA_ATTN_ERR_SCALE;
    return NOVA_ATTN_OK;
}

}  // namespace nova

using namespace nova;

extern "C" {

int nova_attn_fwd_strided(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int H, int T, int D,
                          const nova_attn_strides* q_strides, const nova_attn_strides* k_strides,
                          const nova_attn_strides* v_strides, const nova_attn_strides* o_strides, float scale,
                          int causal, void* stream) {
    if (!Q || !K || !V || !O || !LSE) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_shape(B, H, T, D)) return rc;
    if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O) || !aligned16(LSE)) return NOVA_ATTN_ERR_ALIGNMENT;
    if (!std::isfinite(scale) || !(scale > 0.f)) return NOVA_ATTN_ERR_SCALE;
    TensorStrides sq, sk, sv, so;
    if (int rc = check_strides(q_strides, D, &sq)) return rc;
    if (int rc = check_strides(k_strides, D, &sk)) return rc;
    if (int rc = check_strides(v_strides, D, &sv)) return rc;
    if (int rc = check_strides(o_strides, D, &so)) return rc;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const AttnShape s{B, H, T, D, causal != 0, scale};
    CUtensorMap tmQ, tmK, tmV, tmO;
    uint32_t oq, ok, ov, oo;
    const bool strided = !(merges(s, sq) && merges(s, sk) && merges(s, sv) && merges(s, so));
    if (int rc = get_bf16_map(Q, s, sq, strided, &tmQ, &oq)) return rc;
    if (int rc = get_bf16_map(K, s, sk, strided, &tmK, &ok)) return rc;
    if (int rc = get_bf16_map(V, s, sv, strided, &tmV, &ov)) return rc;
    if (int rc = get_bf16_map(O, s, so, strided, &tmO, &oo)) return rc;
    const uint32_t orders = oq | (ok << 4) | (ov << 8) | (oo << 12);
    const cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const cudaError_t e = launch_attn_fwd(tmQ, tmK, tmV, tmO, strided, orders, LSE, s, st->num_sms,
                                          g_wait_limit.load(std::memory_order_relaxed),
                                          g_inject.load(std::memory_order_relaxed), st->dev_status, cs);
    return e == cudaSuccess ? NOVA_ATTN_OK : fail_cuda(e);
}

int nova_attn_fwd(const void* Q, const void* K, const void* V, void* O, float* LSE, int B, int H, int T, int D,
                  float scale, int causal, void* stream) {
    if (int rc = check_shape(B, H, T, D)) return rc;
    const TensorStrides c = contiguous_strides(H, T, D);
    const nova_attn_strides n{c.b, c.h, c.t};
    return nova_attn_fwd_strided(Q, K, V, O, LSE, B, H, T, D, &n, &n, &n, &n, scale, causal, stream);
}

int nova_attn_bwd_preprocess_strided(const void* O, const void* dO, float* Delta, int B, int H, int T, int D,
                                     const nova_attn_strides* o_strides, const nova_attn_strides* do_strides,
                                     void* stream) {
    if (!O || !dO || !Delta) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_shape(B, H, T, D)) return rc;
    if (!aligned16(O) || !aligned16(dO) || !aligned16(Delta)) return NOVA_ATTN_ERR_ALIGNMENT;
    TensorStrides so, sdo;
    if (int rc = check_strides(o_strides, D, &so)) return rc;
    if (int rc = check_strides(do_strides, D, &sdo)) return rc;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const AttnShape s{B, H, T, D, 1, 1.f};
    const cudaError_t e =
        launch_attn_bwd_preprocess(static_cast<const __nv_bfloat16*>(O), static_cast<const __nv_bfloat16*>(dO), Delta, s,
                                   so, sdo, st->num_sms, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NOVA_ATTN_OK : fail_cuda(e);
}

int nova_attn_bwd_preprocess(const void* O, const void* dO, float* Delta, int B, int H, int T, int D, void* stream) {
    if (int rc = check_shape(B, H, T, D)) return rc;
    const TensorStrides c = contiguous_strides(H, T, D);
    const nova_attn_strides n{c.b, c.h, c.t};
    return nova_attn_bwd_preprocess_strided(O, dO, Delta, B, H, T, D, &n, &n, stream);
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

namespace {
// The three steps of the backward on strided bf16 tensors; `steps` as in nova_attn_bwd_steps.
int bwd_impl(const void* Q, const void* K, const void* V, const void* dO, const float* LSE, const float* Delta, void* dQ,
             void* dK, void* dV, int B, int H, int T, int D, const TensorStrides& sq, const TensorStrides& sk,
             const TensorStrides& sv, const TensorStrides& sdo, const TensorStrides& sdq, const TensorStrides& sdk,
             const TensorStrides& sdv, float scale, int causal, void* workspace, size_t workspace_bytes, void* stream,
             int steps) {
    if (int rc = validate_bwd_args(Q, K, V, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, scale)) return rc;
    const size_t need = nova_attn_bwd_workspace_bytes(B, H, T, D);
    if (!workspace || workspace_bytes < need) return NOVA_ATTN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return NOVA_ATTN_ERR_ALIGNMENT;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const long long BH = static_cast<long long>(B) * H;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    float* acc = static_cast<float*>(workspace);
    const AttnShape s{B, H, T, D, causal != 0, scale};
    cudaError_t e = cudaSuccess;
    if (steps & NOVA_ATTN_BWD_STEP_ZERO) {
        e = launch_zero(acc, need, st->num_sms, cs);
        if (e != cudaSuccess) return fail_cuda(e);
    }
    if (steps & NOVA_ATTN_BWD_STEP_MAIN) {
        CUtensorMap tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV;
        uint32_t oq, ok, ov, odo, odk, odv;
        const bool strided = !(merges(s, sq) && merges(s, sk) && merges(s, sv) && merges(s, sdo) && merges(s, sdk) &&
                               merges(s, sdv));
        if (int rc = get_bf16_map(Q, s, sq, strided, &tmQ, &oq)) return rc;
        if (int rc = get_bf16_map(K, s, sk, strided, &tmK, &ok)) return rc;
        if (int rc = get_bf16_map(V, s, sv, strided, &tmV, &ov)) return rc;
        if (int rc = get_bf16_map(dO, s, sdo, strided, &tmdO, &odo)) return rc;
        if (int rc = get_tensor_map(acc, D, T, BH, &tmAcc, 4)) return rc;
        if (int rc = get_bf16_map(dK, s, sdk, strided, &tmdK, &odk)) return rc;
        if (int rc = get_bf16_map(dV, s, sdv, strided, &tmdV, &odv)) return rc;
        const uint32_t orders = oq | (ok << 4) | (ov << 8) | (odo << 12) | (odk << 16) | (odv << 20);
        e = launch_attn_bwd(tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, strided, orders, false, LSE, Delta, static_cast<__nv_bfloat16*>(dK),
                            static_cast<__nv_bfloat16*>(dV), sdk, sdv, s, st->num_sms, st->dev_status, cs);
        if (e != cudaSuccess) return fail_cuda(e);
    }
    if (steps & NOVA_ATTN_BWD_STEP_CONVERT) {
        e = launch_dq_convert(acc, static_cast<__nv_bfloat16*>(dQ), s, sdq, scale, st->num_sms, cs);
        if (e != cudaSuccess) return fail_cuda(e);
    }
    return NOVA_ATTN_OK;
}
}  // namespace

int nova_attn_bwd_steps(const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* LSE,
                        const float* Delta, void* dQ, void* dK, void* dV, int B, int H, int T, int D, float scale,
                        int causal, void* workspace, size_t workspace_bytes, void* stream, int steps) {
    (void)O;  // Delta already carries rowsum(dO * O)
    if (int rc = validate_bwd_args(Q, K, V, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, scale)) return rc;
    const TensorStrides c = contiguous_strides(H, T, D);
    return bwd_impl(Q, K, V, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, c, c, c, c, c, c, c, scale, causal, workspace,
                    workspace_bytes, stream, steps);
}

int nova_attn_bwd(const void* Q, const void* K, const void* V, const void* O, const void* dO, const float* LSE,
                  const float* Delta, void* dQ, void* dK, void* dV, int B, int H, int T, int D, float scale,
                  int causal, void* workspace, size_t workspace_bytes, void* stream) {
    return nova_attn_bwd_steps(Q, K, V, O, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, scale, causal, workspace,
                               workspace_bytes, stream,
                               NOVA_ATTN_BWD_STEP_ZERO | NOVA_ATTN_BWD_STEP_MAIN | NOVA_ATTN_BWD_STEP_CONVERT);
}

int nova_attn_bwd_deterministic(const void* Q, const void* K, const void* V, const void* dO, const float* LSE,
                                const float* Delta, void* dQ, void* dK, void* dV, int B, int H, int T, int D,
                                float scale, int causal, void* stream) {
    if (int rc = validate_bwd_args(Q, K, V, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, scale)) return rc;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    const long long BH = static_cast<long long>(B) * H;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    const AttnShape s{B, H, T, D, causal != 0, scale};
    const TensorStrides c = contiguous_strides(H, T, D);
    CUtensorMap tmQ, tmK, tmV, tmdO, tmdK, tmdV;
    if (int rc = get_tensor_map(Q, D, T, BH, &tmQ)) return rc;
    if (int rc = get_tensor_map(K, D, T, BH, &tmK)) return rc;
    if (int rc = get_tensor_map(V, D, T, BH, &tmV)) return rc;
    if (int rc = get_tensor_map(dO, D, T, BH, &tmdO)) return rc;
    if (int rc = get_tensor_map(dK, D, T, BH, &tmdK)) return rc;
    if (int rc = get_tensor_map(dV, D, T, BH, &tmdV)) return rc;
    cudaError_t e = launch_attn_dq(tmQ, tmK, tmV, tmdO, LSE, Delta, static_cast<__nv_bfloat16*>(dQ), s, st->dev_status, cs);
    if (e != cudaSuccess) return fail_cuda(e);
    // the dK/dV half: the fused kernel without its dQ product (the accumulator map is never used: any map will do)
    e = launch_attn_bwd(tmQ, tmK, tmV, tmdO, tmQ, tmdK, tmdV, false, 0u, true, LSE, Delta, static_cast<__nv_bfloat16*>(dK),
                        static_cast<__nv_bfloat16*>(dV), c, c, s, st->num_sms, st->dev_status, cs);
    return e == cudaSuccess ? NOVA_ATTN_OK : fail_cuda(e);
}

int nova_attn_bwd_strided(const void* Q, const void* K, const void* V, const void* dO, const float* LSE,
                          const float* Delta, void* dQ, void* dK, void* dV, int B, int H, int T, int D,
                          const nova_attn_strides* q_strides, const nova_attn_strides* k_strides,
                          const nova_attn_strides* v_strides, const nova_attn_strides* do_strides,
                          const nova_attn_strides* dq_strides, const nova_attn_strides* dk_strides,
                          const nova_attn_strides* dv_strides, float scale, int causal, void* workspace,
                          size_t workspace_bytes, void* stream) {
    if (int rc = check_shape(B, H, T, D)) return rc;
    TensorStrides sq, sk, sv, sdo, sdq, sdk, sdv;
    if (int rc = check_strides(q_strides, D, &sq)) return rc;
    if (int rc = check_strides(k_strides, D, &sk)) return rc;
    if (int rc = check_strides(v_strides, D, &sv)) return rc;
    if (int rc = check_strides(do_strides, D, &sdo)) return rc;
    if (int rc = check_strides(dq_strides, D, &sdq)) return rc;
    if (int rc = check_strides(dk_strides, D, &sdk)) return rc;
    if (int rc = check_strides(dv_strides, D, &sdv)) return rc;
    return bwd_impl(Q, K, V, dO, LSE, Delta, dQ, dK, dV, B, H, T, D, sq, sk, sv, sdo, sdq, sdk, sdv, scale, causal,
                    workspace, workspace_bytes, stream,
                    NOVA_ATTN_BWD_STEP_ZERO | NOVA_ATTN_BWD_STEP_MAIN | NOVA_ATTN_BWD_STEP_CONVERT);
}

size_t nova_lmhead_workspace_bytes(int M, int N, int K) {
    if (check_lmhead_shape(M, N, K) != NOVA_ATTN_OK) return 0;
    return lmhead_workspace_bytes(M, N);
}

int nova_lmhead_fwd(const void* X, const void* W, const int* targets, void* logits, float* lse, float* loss, int M,
                    int N, int K, void* workspace, size_t workspace_bytes, void* stream) {
    if (!X || !W || !targets || !lse || !loss) return NOVA_ATTN_ERR_NULL;
    if (int rc = check_lmhead_shape(M, N, K)) return rc;
    if (!aligned16(X) || !aligned16(W) || !aligned16(logits)) return NOVA_ATTN_ERR_ALIGNMENT;
    if ((reinterpret_cast<uintptr_t>(targets) & 3u) || (reinterpret_cast<uintptr_t>(lse) & 3u) ||
        (reinterpret_cast<uintptr_t>(loss) & 3u))
        return NOVA_ATTN_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < lmhead_workspace_bytes(M, N)) return NOVA_ATTN_ERR_WORKSPACE;
    if (!aligned16(workspace)) return NOVA_ATTN_ERR_ALIGNMENT;
    DeviceState* st = nullptr;
    if (int rc = device_state(&st)) return rc;
    int rows_x = 0, rows_w = 0;
    const int box_k = lmhead_boxes(&rows_x, &rows_w);
    CUtensorMap tmX, tmW, tmWh, tmL;
    if (int rc = encode_matrix_map(X, M, K, rows_x, box_k, &tmX)) return rc;
    if (int rc = encode_matrix_map(W, N, K, rows_w, box_k, &tmW)) return rc;
    if (int rc = encode_matrix_map(W, N, K, rows_w / 2, box_k, &tmWh)) return rc;  // half a W tile per CTA of a pair
    if (logits) {
        if (int rc = encode_matrix_map(logits, M, N, 32, 64, &tmL)) return rc;
    } else {
        tmL = tmX;  // never used
    }
    const cudaError_t e = launch_lmhead(tmX, tmW, tmWh, tmL, logits != nullptr, targets, lse, loss, M, N, K, workspace,
                                        st->num_sms, st->dev_status, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? NOVA_ATTN_OK : fail_cuda(e);
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

int nova_attn_test_configure_waits(long long limit_cycles, int inject) {
    if (limit_cycles < 0 || inject < 0 || inject > 1) return NOVA_ATTN_ERR_SHAPE;
    g_wait_limit.store(limit_cycles == 0 ? kDefaultWaitLimit : limit_cycles, std::memory_order_relaxed);
    g_inject.store(inject, std::memory_order_relaxed);
    return NOVA_ATTN_OK;
}

int nova_attn_bwd_work_list(int BH, long long T, int D, int causal, int n_ctas, int cta, int* items, int capacity,
                            int* plan4) {
    if (BH < 1 || T < 1 || (D != 64 && D != 128) || n_ctas < 1 || cta < 0 || cta >= n_ctas || capacity < 0 ||
        (capacity > 0 && items == nullptr))
        return NOVA_ATTN_ERR_SHAPE;
    int n_tiles = 0, grid = 0;
    const WorkPlan plan = bwd_work_plan(BH, T, D, causal != 0, n_ctas, &n_tiles, &grid);
    if (plan4 != nullptr) {
        plan4[0] = plan.chunk;
        plan4[1] = plan.n_chunks;
        plan4[2] = plan.passes_per_chunk;
        plan4[3] = plan.passes_last;
    }
    if (cta >= grid) return 0;  // fewer items than CTAs: the grid is that much smaller
    const WorkArgs wa{BH, n_tiles, 1, 0u, 0, plan};
    const WorkList wl{wa, causal != 0};
    int n = 0;
    for (WorkCursor cur; !wl.done(cur); wl.advance(cur)) {
        int kt, bh, i0, n_it;
        if (!wl.get_for(cur, grid, cta, &kt, &bh, &i0, &n_it)) continue;
        if (n < capacity) {
            items[2 * n] = kt;
            items[2 * n + 1] = bh;
        }
        ++n;
    }
    return n;
}

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
