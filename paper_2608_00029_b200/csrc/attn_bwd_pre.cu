// Memory-bound helpers of the backward pass.
//   bwd_preprocess_kernel: Delta_i = sum_d dO[i,d] * O[i,d]   (row term of the softmax Jacobian)
//   dq_convert_kernel:     dQ = bf16(scale * fp32 accumulator)
//   zero_kernel:           clears the fp32 accumulator before the backward kernel adds into it
// Both stream their inputs once with 16-byte loads; rows are split over D/8 lanes and reduced with
// xor-shuffles.  Grids are sized in multiples of the SM count.  The bf16 tensors may be strided
// (batch, head and token strides in elements, multiples of 8): a row index r = (b*H + h)*T + t is
// then split again; the contiguous case skips that arithmetic.
#include "kernels.h"
#include "ptx.cuh"

namespace nova {
namespace {

__device__ __forceinline__ float dot8_bf16(const uint4& a, const uint4& b) {
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float2 fa = __bfloat1622float2(pa[i]);
        const float2 fb = __bfloat1622float2(pb[i]);
        acc = fmaf(fa.x, fb.x, acc);
        acc = fmaf(fa.y, fb.y, acc);
    }
    return acc;
}

// Offset, in 16-byte units, of row r = (b*H + h)*T + t of a tensor with strides `s`.
__device__ __forceinline__ long long row_offset16(long long r, int H, int T, const TensorStrides& s) {
    const long long bh = r / T;
    const long long t = r - bh * T;
    const long long b = bh / H;
    const long long h = bh - b * H;
    return (b * s.b + h * s.h + t * s.t) >> 3;
}

// LPR = lanes per row = D/8 (8 for D=64, 16 for D=128); each lane owns 8 consecutive bf16.
template <int LPR, int UNROLL, bool kContiguous>
__global__ void __launch_bounds__(256) bwd_preprocess_kernel(const uint4* __restrict__ O, const uint4* __restrict__ dO,
                                                             float* __restrict__ Delta, long long rows, int H, int T,
                                                             const TensorStrides so, const TensorStrides sdo) {
    griddep_launch_dependents();
    griddep_wait();
    const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
    const long long rows_per_pass = nthreads / LPR;
    const int sub = static_cast<int>(tid % LPR);
    long long r = tid / LPR;
    for (; r < rows; r += rows_per_pass * UNROLL) {
        uint4 a[UNROLL], b[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const long long ru = r + u * rows_per_pass;
            if (ru < rows) {
                a[u] = __ldg(O + (kContiguous ? ru * LPR : row_offset16(ru, H, T, so)) + sub);
                b[u] = __ldg(dO + (kContiguous ? ru * LPR : row_offset16(ru, H, T, sdo)) + sub);
            } else {
                a[u] = make_uint4(0, 0, 0, 0);
                b[u] = make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            float acc = dot8_bf16(a[u], b[u]);
#pragma unroll
            for (int off = LPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            const long long ru = r + u * rows_per_pass;
            if (sub == 0 && ru < rows) Delta[ru] = acc;
        }
    }
}

// Each thread takes kConvertItems groups of 8 elements per pass and issues all their loads before the
// first store.
constexpr int kConvertItems = 4;

template <bool kContiguous>
__global__ void __launch_bounds__(256) dq_convert_kernel(const float4* __restrict__ acc, uint4* __restrict__ dQ,
                                                         long long n8, float scale, int lpr_shift, int H, int T,
                                                         const TensorStrides sdq) {
    griddep_launch_dependents();
    griddep_wait();
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x * kConvertItems;
    for (long long base = static_cast<long long>(blockIdx.x) * blockDim.x * kConvertItems + threadIdx.x; base < n8;
         base += stride) {
        float4 a[kConvertItems], b[kConvertItems];
#pragma unroll
        for (int k = 0; k < kConvertItems; ++k) {
            const long long i = base + static_cast<long long>(k) * blockDim.x;
            if (i < n8) {
                a[k] = __ldcs(acc + 2 * i);
                b[k] = __ldcs(acc + 2 * i + 1);
            }
        }
#pragma unroll
        for (int k = 0; k < kConvertItems; ++k) {
            const long long i = base + static_cast<long long>(k) * blockDim.x;
            if (i >= n8) continue;
            uint4 v;
            v.x = pack_bf16x2(a[k].x * scale, a[k].y * scale);
            v.y = pack_bf16x2(a[k].z * scale, a[k].w * scale);
            v.z = pack_bf16x2(b[k].x * scale, b[k].y * scale);
            v.w = pack_bf16x2(b[k].z * scale, b[k].w * scale);
            if (kContiguous) {
                dQ[i] = v;
            } else {
                const long long r = i >> lpr_shift;
                dQ[row_offset16(r, H, T, sdq) + (i - (r << lpr_shift))] = v;
            }
        }
    }
}

__global__ void __launch_bounds__(256) zero_kernel(uint4* __restrict__ p, long long n16) {
    griddep_launch_dependents();
    griddep_wait();
    const long long stride = static_cast<long long>(gridDim.x) * blockDim.x;
    for (long long i = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x; i < n16; i += stride)
        p[i] = make_uint4(0, 0, 0, 0);
}

}  // namespace

cudaError_t launch_zero(void* ptr, size_t bytes, int num_sms, cudaStream_t stream) {
    constexpr int kThreads = 256;
    const long long n16 = static_cast<long long>(bytes / 16);
    long long blocks = (n16 + kThreads - 1) / kThreads;
    const long long cap = static_cast<long long>(num_sms) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return launch_overlapped(zero_kernel, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), 0, stream,
                             static_cast<uint4*>(ptr), n16);
}

namespace {
bool is_contiguous(const AttnShape& s, const TensorStrides& st) {
    return st.t == s.D && st.h == static_cast<long long>(s.T) * s.D && st.b == static_cast<long long>(s.H) * s.T * s.D;
}
}  // namespace

cudaError_t launch_attn_bwd_preprocess(const __nv_bfloat16* O, const __nv_bfloat16* dO, float* Delta,
                                       const AttnShape& s, const TensorStrides& so, const TensorStrides& sdo,
                                       int num_sms, cudaStream_t stream) {
    constexpr int kThreads = 256, kUnroll = 4;
    const long long rows = static_cast<long long>(s.B) * s.H * s.T;
    const int lpr = s.D / 8;
    const long long rows_per_block = kThreads / lpr * kUnroll;
    long long blocks = (rows + rows_per_block - 1) / rows_per_block;
    const long long cap = static_cast<long long>(num_sms) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const uint4* o4 = reinterpret_cast<const uint4*>(O);
    const uint4* d4 = reinterpret_cast<const uint4*>(dO);
    const dim3 grid(static_cast<unsigned>(blocks));
    const bool contiguous = is_contiguous(s, so) && is_contiguous(s, sdo);
    auto go = [&](auto kernel) {
        return launch_overlapped(kernel, grid, dim3(kThreads), 0, stream, o4, d4, Delta, rows, s.H, s.T, so, sdo);
    };
    if (s.D == 64) return contiguous ? go(bwd_preprocess_kernel<8, kUnroll, true>) : go(bwd_preprocess_kernel<8, kUnroll, false>);
    return contiguous ? go(bwd_preprocess_kernel<16, kUnroll, true>) : go(bwd_preprocess_kernel<16, kUnroll, false>);
}

cudaError_t launch_dq_convert(const float* dq_acc, __nv_bfloat16* dQ, const AttnShape& s, const TensorStrides& sdq,
                              float scale, int num_sms, cudaStream_t stream) {
    constexpr int kThreads = 256;
    const long long n8 = static_cast<long long>(s.B) * s.H * s.T * s.D / 8;  // D is a multiple of 8
    long long blocks = (n8 + kThreads * kConvertItems - 1) / (kThreads * kConvertItems);
    const long long cap = static_cast<long long>(num_sms) * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const int lpr_shift = (s.D == 64) ? 3 : 4;
    const dim3 grid(static_cast<unsigned>(blocks));
    auto go = [&](auto kernel) {
        return launch_overlapped(kernel, grid, dim3(kThreads), 0, stream, reinterpret_cast<const float4*>(dq_acc),
                                 reinterpret_cast<uint4*>(dQ), n8, scale, lpr_shift, s.H, s.T, sdq);
    };
    return is_contiguous(s, sdq) ? go(dq_convert_kernel<true>) : go(dq_convert_kernel<false>);
}

}  // namespace nova
