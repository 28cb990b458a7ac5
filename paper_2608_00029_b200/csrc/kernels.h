// Internal launch interface between the C ABI (api.cu) and the kernels.  Not installed.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace nova {

constexpr int kBlockQ = 128;        // query rows per tile (UMMA M)
constexpr int kBlockK = 128;        // keys per tile
constexpr int kBoxCols = 64;        // bf16 elements per 128-byte swizzled row (TMA box inner extent)
constexpr int kHalfTileBytes = 128 * 128;  // one [128 rows x 64 bf16] box

struct AttnShape {
    int B, H, T, D;
    int causal;
    float scale;
};

// Strides, in elements, of a bf16 tensor indexed [b, h, t, d]; d is contiguous.  [B,H,T,D] storage has
// (H*T*D, T*D, D); the Q slice of a fused projection output [B, T, 3, H, D] has (T*3*H*D, D, 3*H*D).
struct TensorStrides {
    long long b, h, t;
};

// Records a CUDA error code for nova_attn_last_cuda_error() of the calling thread and returns
// NOVA_ATTN_ERR_CUDA; for the entry points that live outside api.cu.
int record_cuda_error(int code);

// The argument checks every backward entry point makes before anything else (NULL pointers, shape, 16-byte
// alignment of the tensors, scale); returns NOVA_ATTN_OK or the error nova_attn_bwd would report.
int validate_bwd_args(const void* Q, const void* K, const void* V, const void* dO, const float* LSE,
                      const float* Delta, const void* dQ, const void* dK, const void* dV, int B, int H, int T, int D,
                      float scale);

// Launches `kernel` allowing it to overlap the tail of the previous kernel in `stream` (programmatic
// dependent launch); the kernel must call griddep_wait() before it touches global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_overlapped(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem_bytes,
                                     cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// Forward.  Two builds of every kernel.  Plain (`strided` false): all bf16 tensors have batch stride =
// H * head stride, so their maps are 3-D [D, T, B*H]; box of 64 x 128 tokens, 128-byte swizzle.  Strided:
// the maps are 4-D [D, x, y, z] with token / head / batch in order of increasing stride, and `orders`
// holds, four bits per tensor in the order Q, K, V, O, which of the three sits where (see
// tma_load_tile).  `tmO` describes the output and is used for TMA stores.  Persistent: launches at most
// `num_sms` CTAs.  `wait_limit`: cycle limit of every device-side wait; `inject`: test aid, 1 makes the
// loader leave out its first K-tile request so that a wait runs out (0 in normal use).
cudaError_t launch_attn_fwd(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            const CUtensorMap& tmO, bool strided, uint32_t orders, float* LSE, const AttnShape& s,
                            int num_sms, long long wait_limit, int inject, int* dev_status, cudaStream_t stream);
cudaError_t configure_attn_fwd();

cudaError_t launch_attn_bwd_preprocess(const __nv_bfloat16* O, const __nv_bfloat16* dO, float* Delta,
                                       const AttnShape& s, const TensorStrides& so, const TensorStrides& sdo,
                                       int num_sms, cudaStream_t stream);

// Exact Delta_i = sum_j P_ij (dO_i . V_j) with P rebuilt from LSE (two contractions + exp2 per tile).
cudaError_t launch_attn_delta(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                              const CUtensorMap& tmdO, const float* LSE, float* Delta, const AttnShape& s,
                              int* dev_status, cudaStream_t stream);
cudaError_t configure_attn_delta();

// Deterministic dQ (the dQ half of the paper's two-kernel backward): one CTA per 128-row query tile walks
// the key tiles in order and writes dQ = bf16(scale * sum_j dS_j K_j).  3-D [D, T, B*H] maps; dQ contiguous.
cudaError_t launch_attn_dq(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                           const CUtensorMap& tmdO, const float* LSE, const float* Delta, __nv_bfloat16* dQ,
                           const AttnShape& s, int* dev_status, cudaStream_t stream);
cudaError_t configure_attn_dq();

// Backward main kernel: adds unscaled dQ partial tiles into the fp32 accumulator [B,H,T,D] (zero on
// entry) described by `tmAcc` (fp32 [D, T, B*H], box [32, 128, 1], 128-byte swizzle) and writes dK and dV
// (`tmdK`, `tmdV`: the bf16 maps of the outputs, used for TMA stores at D=64; at D=128 the rows go out
// with plain stores through `dK`, `dV` and their strides).  `strided`, `orders`: as in the forward, for
// Q, K, V, dO, dK, dV.  `no_dq`: write dK and dV only (the dK/dV half of the two-kernel backward); `tmAcc` is
// then never used.  Persistent: launches at most `num_sms` CTAs.
cudaError_t launch_attn_bwd(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            const CUtensorMap& tmdO, const CUtensorMap& tmAcc, const CUtensorMap& tmdK,
                            const CUtensorMap& tmdV, bool strided, uint32_t orders, bool no_dq, const float* LSE, const float* Delta,
                            __nv_bfloat16* dK, __nv_bfloat16* dV, const TensorStrides& sdk, const TensorStrides& sdv,
                            const AttnShape& s, int num_sms, int* dev_status, cudaStream_t stream);
cudaError_t configure_attn_bwd();

// Loss head (lmhead.cu): `tmX` is the 2-D map of X [K, M] with box [64, 128], `tmW` that of W [K, N] with box
// [64, 256], `tmL` that of the logits [N, M] with box [64, 32] (any valid map if `store_logits` is false), all
// bf16 with 128-byte swizzle.  Enqueues the fused contraction + statistics kernel and the merge.
cudaError_t launch_lmhead(const CUtensorMap& tmX, const CUtensorMap& tmW, const CUtensorMap& tmWh, const CUtensorMap& tmL,
                          bool store_logits, const int* targets, float* lse, float* loss, int M, int N, int K,
                          void* workspace, int num_sms, int* dev_status, cudaStream_t stream);
cudaError_t configure_lmhead();
size_t lmhead_workspace_bytes(int M, int N);
// Rows of the X and W boxes; returns the box width in k elements.
int lmhead_boxes(int* box_rows_x, int* box_rows_w);

// Clears `bytes` (a multiple of 16) at the 16-byte aligned `ptr`.
cudaError_t launch_zero(void* ptr, size_t bytes, int num_sms, cudaStream_t stream);

// dQ = bf16(scale * dq_acc); the accumulator is contiguous [B,H,T,D], dQ has strides `sdq`.
cudaError_t launch_dq_convert(const float* dq_acc, __nv_bfloat16* dQ, const AttnShape& s, const TensorStrides& sdq,
                              float scale, int num_sms, cudaStream_t stream);

}  // namespace nova
