// Exact softmax-Jacobian row term for the backward pass:  Delta_i = sum_j P_ij * (dO_i . V_j),
// with P recomputed from the saved log-sum-exp (paper Section 4.2, "The Backward Pass": the
// probability matrix is rebuilt inside the kernel, never stored).
//
// The cheap route to the same quantity, rowsum(dO * O), inherits the bf16 rounding of the stored O;
// with sharply peaked softmax rows (|O| ~ |V|) that error, multiplied by scale * (P K)_i, is the
// largest term in dQ and dK.  This kernel trades two extra contractions for an fp32-exact Delta.
//
// Same skeleton as the forward: one CTA per 128-row query tile, causal clamp of the key loop,
//   warp 0      TMA producer (Q and dO once, K and V tiles through a ring)
//   warp 1      UMMA issuer: S = Q K^T and dP = dO V^T into two TMEM accumulators
//   warps 2..5  one thread per query row: acc += exp2(S*c - LSE*log2e) * dP over the kept keys.
#include "kernels.h"
#include "ptx.cuh"

namespace nova {
namespace {

constexpr int kThreads = 192;
constexpr int kTmemCols = 256;

template <int D>
struct DeltaCfg {
    static constexpr int kHalves = D / kBoxCols;
    static constexpr int kTileBytes = kHalves * kHalfTileBytes;
    static constexpr int kStages = (D == 64) ? 2 : 1;
    static constexpr int kOffQ = 0;
    static constexpr int kOffdO = kTileBytes;
    static constexpr int kOffK = 2 * kTileBytes;
    static constexpr int kOffV = kOffK + kStages * kTileBytes;
    static constexpr int kOffBar = kOffV + kStages * kTileBytes;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;
};

struct DeltaBars {
    uint64_t q_full;
    uint64_t kv_full[2], kv_empty[2];
    uint64_t acc_full, acc_free, drain;
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__device__ __forceinline__ void delta_producer(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV,
                                               const CUtensorMap* tmdO, uint8_t* smem, DeltaBars* bars, int qt,
                                               int bh, int n_kv) {
    using Cfg = DeltaCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    int armed[2] = {-1, -1};
    mbar_expect_tx(&bars->q_full, 2 * Cfg::kTileBytes);
#pragma unroll
    for (int h = 0; h < Cfg::kHalves; ++h) {
        tma_load_3d(smem + Cfg::kOffQ + h * kHalfTileBytes, tmQ, &bars->q_full, h * kBoxCols, qt * kBlockQ, bh);
        tma_load_3d(smem + Cfg::kOffdO + h * kHalfTileBytes, tmdO, &bars->q_full, h * kBoxCols, qt * kBlockQ, bh);
    }
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
        const int st = j % Cfg::kStages;
        const uint32_t ph = (j / Cfg::kStages) & 1;
        ok = mbar_wait(&bars->kv_empty[st], ph ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(&bars->kv_full[st], 2 * Cfg::kTileBytes);
        armed[st] = ph;
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h) {
            tma_load_3d(smem + Cfg::kOffK + st * Cfg::kTileBytes + h * kHalfTileBytes, tmK, &bars->kv_full[st],
                        h * kBoxCols, j * kBlockK, bh);
            tma_load_3d(smem + Cfg::kOffV + st * Cfg::kTileBytes + h * kHalfTileBytes, tmV, &bars->kv_full[st],
                        h * kBoxCols, j * kBlockK, bh);
        }
    }
    if (!ok) {
        int none = 0;
        (void)mbar_wait(&bars->q_full, 0, &none);
        for (int st = 0; st < Cfg::kStages; ++st)
            if (armed[st] >= 0) (void)mbar_wait(&bars->kv_full[st], armed[st], &none);
    }
}

template <int D>
__device__ __forceinline__ void delta_mma(uint8_t* smem, DeltaBars* bars, uint32_t tmem_base, int n_kv) {
    using Cfg = DeltaCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    constexpr uint32_t kIdesc = umma_idesc_bf16(128, 128, 0, 0);
    const uint32_t sQ = smem_u32(smem + Cfg::kOffQ), sdO = smem_u32(smem + Cfg::kOffdO);
    bool ok = mbar_wait(&bars->q_full, 0, abort_flag);
    for (int j = 0; j < n_kv && ok; ++j) {
        const int st = j % Cfg::kStages;
        const uint32_t ph = (j / Cfg::kStages) & 1;
        ok = mbar_wait(&bars->kv_full[st], ph, abort_flag);
        if (!ok) break;
        ok = mbar_wait(&bars->acc_free, (j & 1) ^ 1, abort_flag);  // rows of tile j-1 have been read
        if (!ok) break;
        tc_fence_after();
        const uint32_t sK = smem_u32(smem + Cfg::kOffK + st * Cfg::kTileBytes);
        const uint32_t sV = smem_u32(smem + Cfg::kOffV + st * Cfg::kTileBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * kHalfTileBytes + (k % 4) * 32;
            umma_ss(tmem_base, umma_smem_desc_sw128(sQ + off, 16, 1024), umma_smem_desc_sw128(sK + off, 16, 1024),
                    kIdesc, k > 0 ? 1u : 0u);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * kHalfTileBytes + (k % 4) * 32;
            umma_ss(tmem_base + 128, umma_smem_desc_sw128(sdO + off, 16, 1024),
                    umma_smem_desc_sw128(sV + off, 16, 1024), kIdesc, k > 0 ? 1u : 0u);
        }
        tc_commit(&bars->kv_empty[st]);
        tc_commit(&bars->acc_full);
    }
    if (!ok) {
        int none = 0;
        tc_commit(&bars->drain);
        (void)mbar_wait(&bars->drain, 0, &none);
    }
}

template <int D, bool kCausal>
__device__ __forceinline__ void delta_rows(DeltaBars* bars, uint32_t tmem_base, const float* __restrict__ LSE,
                                           float* __restrict__ Delta, int T, int qt, int bh, int n_kv, float scale,
                                           int warp, int lane) {
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (warp & 3);
    const int row_local = lane_base + lane;
    const int row = qt * kBlockQ + row_local;
    const uint32_t t_s = tmem_addr(tmem_base, lane_base, 0);
    const uint32_t t_dp = tmem_addr(tmem_base, lane_base, 128);
    const float c = scale * kLog2e;
    const size_t idx = static_cast<size_t>(bh) * T + row;
    // Rows past the end of the sequence: LSE = +inf gives P = 0 everywhere.
    const float lse2 = (row < T) ? LSE[idx] * kLog2e : INFINITY;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
        ok = mbar_wait(&bars->acc_full, j & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const bool diag = kCausal && (j == qt);
        const int keys_left = T - j * kBlockK;
        const int lim = diag ? min(row_local, keys_left - 1) : min(keys_left, kBlockK) - 1;
#pragma unroll 1
        for (int cb = 0; cb < 128; cb += 32) {
            uint32_t sv[32], dv[32];
            tmem_ld_x32(t_s + cb, sv);
            tmem_ld_x32(t_dp + cb, dv);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                float p0 = ex2_approx(fmaf(__uint_as_float(sv[i + 0]), c, -lse2));
                float p1 = ex2_approx(fmaf(__uint_as_float(sv[i + 1]), c, -lse2));
                float p2 = ex2_approx(fmaf(__uint_as_float(sv[i + 2]), c, -lse2));
                float p3 = ex2_approx(fmaf(__uint_as_float(sv[i + 3]), c, -lse2));
                if (cb + i + 0 > lim) p0 = 0.f;
                if (cb + i + 1 > lim) p1 = 0.f;
                if (cb + i + 2 > lim) p2 = 0.f;
                if (cb + i + 3 > lim) p3 = 0.f;
                a0 = fmaf(p0, __uint_as_float(dv[i + 0]), a0);
                a1 = fmaf(p1, __uint_as_float(dv[i + 1]), a1);
                a2 = fmaf(p2, __uint_as_float(dv[i + 2]), a2);
                a3 = fmaf(p3, __uint_as_float(dv[i + 3]), a3);
            }
        }
        tc_fence_before();
        mbar_arrive(&bars->acc_free);
    }
    if (ok && row < T) Delta[idx] = (a0 + a1) + (a2 + a3);
}

template <int D, bool kCausal>
__global__ void __launch_bounds__(kThreads, 2)
attn_delta_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                  const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                  const float* __restrict__ LSE, float* __restrict__ Delta, int T, int BH, int n_q_tiles, float scale,
                  int* __restrict__ dev_status) {
    using Cfg = DeltaCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    DeltaBars* bars = reinterpret_cast<DeltaBars*>(smem + Cfg::kOffBar);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int qt = n_q_tiles - 1 - static_cast<int>(blockIdx.x) / BH;
    const int bh = static_cast<int>(blockIdx.x) % BH;
    const int n_kv_all = (T + kBlockK - 1) / kBlockK;
    const int n_kv = kCausal ? min(qt + 1, n_kv_all) : n_kv_all;

    if (threadIdx.x == 0) {
        mbar_init(&bars->q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->kv_full[s], 1);
            mbar_init(&bars->kv_empty[s], 1);
        }
        mbar_init(&bars->acc_full, 1);
        mbar_init(&bars->acc_free, 128);
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmdO);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        if (lane == 0) delta_producer<D>(&tmQ, &tmK, &tmV, &tmdO, smem, bars, qt, bh, n_kv);
    } else if (warp == 1) {
        if (lane == 0) delta_mma<D>(smem, bars, tmem_base, n_kv);
    } else {
        delta_rows<D, kCausal>(bars, tmem_base, LSE, Delta, T, qt, bh, n_kv, scale, warp, lane);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

template <int D, bool kCausal>
cudaError_t launch_one(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       const CUtensorMap& tmdO, const float* LSE, float* Delta, const AttnShape& s, int* dev_status,
                       cudaStream_t stream) {
    const int n_q_tiles = (s.T + kBlockQ - 1) / kBlockQ;
    const int BH = s.B * s.H;
    attn_delta_kernel<D, kCausal><<<dim3(static_cast<unsigned>(n_q_tiles) * BH), kThreads, DeltaCfg<D>::kSmemBytes,
                                   stream>>>(tmQ, tmK, tmV, tmdO, LSE, Delta, s.T, BH, n_q_tiles, s.scale, dev_status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t configure_attn_delta() {
    cudaError_t e;
    e = cudaFuncSetAttribute(attn_delta_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DeltaCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_delta_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, DeltaCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_delta_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, DeltaCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_delta_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, DeltaCfg<128>::kSmemBytes);
    return e;
}

cudaError_t launch_attn_delta(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                              const CUtensorMap& tmdO, const float* LSE, float* Delta, const AttnShape& s,
                              int* dev_status, cudaStream_t stream) {
    if (s.D == 64) {
        return s.causal ? launch_one<64, true>(tmQ, tmK, tmV, tmdO, LSE, Delta, s, dev_status, stream)
                        : launch_one<64, false>(tmQ, tmK, tmV, tmdO, LSE, Delta, s, dev_status, stream);
    }
    return s.causal ? launch_one<128, true>(tmQ, tmK, tmV, tmdO, LSE, Delta, s, dev_status, stream)
                    : launch_one<128, false>(tmQ, tmK, tmV, tmdO, LSE, Delta, s, dev_status, stream);
}

}  // namespace nova
