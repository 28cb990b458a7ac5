// Deterministic dQ for the two-kernel backward of the paper (Section 4.2, "The Backward Pass": one kernel
// reduces dQ over keys, the other reduces dK and dV over queries; the probability matrix is rebuilt from
// the saved log-sum-exp in both).  One CTA owns a 128-row query tile of one head and walks the key tiles
// in order, so every dQ row is summed by one thread block in a fixed order: no atomics, no workspace,
// bitwise reproducible.  Per key tile:
//   S  = Q K_j^T,  dP = dO V_j^T            (smem x smem -> two TMEM accumulators)
//   dS = exp2(S*c - LSE*log2e) * (dP - Delta)   (one thread per query row; bf16 back into TMEM over S)
//   dQ += dS K_j                             (TMEM x smem, K read MN-major; accumulator in TMEM)
// and at the end dQ * scale is rounded once to bf16 and stored.  Costs two contractions more than the
// fused backward (S and dP are computed here and again in the dK/dV kernel): the price of determinism.
//   warp 0      TMA producer (Q and dO once, K and V tiles through a ring)
//   warp 1      UMMA issuer
//   warps 2..5  one thread per query row
// TMEM columns: S / dS [0,128)  dP [128,256)  dQ [256, 256+D).
#include "kernels.h"
#include "ptx.cuh"

namespace nova {
namespace {

constexpr int kDqThreads = 192;
constexpr int kDqTmemCols = 512;

template <int D>
struct DqCfg {
    static constexpr int kHalves = D / kBoxCols;
    static constexpr int kTileBytes = kHalves * kHalfTileBytes;
    static constexpr int kStages = (D == 64) ? 2 : 1;
    static constexpr int kOffQ = 0;
    static constexpr int kOffdO = kTileBytes;
    static constexpr int kOffK = 2 * kTileBytes;
    static constexpr int kOffV = kOffK + kStages * kTileBytes;
    static constexpr int kOffBar = kOffV + kStages * kTileBytes;
    // One CTA per SM (it takes all 512 TMEM columns): ask for more than half of the shared memory so
    // that a second CTA is never made resident only to wait for TMEM.
    static constexpr int kSmemBytes = (kOffBar + 256 + 1024) > 120 * 1024 ? (kOffBar + 256 + 1024) : 120 * 1024;
    static constexpr int kColS = 0, kColdP = 128, kColdQ = 256;
};

struct DqBars {
    uint64_t q_full;
    uint64_t kv_full[2], kv_empty[2];
    uint64_t acc_full;   // UMMA -> rows: S and dP of the tile are complete
    uint64_t ds_ready;   // rows (one arrival per warp) -> UMMA: dS is in TMEM
    uint64_t dq_done;    // UMMA -> rows: the last dQ product is complete
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__device__ __forceinline__ void dq_producer(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV,
                                            const CUtensorMap* tmdO, uint8_t* smem, DqBars* bars, int qt, int bh,
                                            int n_kv) {
    using Cfg = DqCfg<D>;
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
    if (!ok) {  // giving up: let the copies in flight land before the CTA's shared memory goes away
        int none = 0;
        (void)mbar_wait(&bars->q_full, 0, &none);
        for (int st = 0; st < Cfg::kStages; ++st)
            if (armed[st] >= 0) (void)mbar_wait(&bars->kv_full[st], armed[st], &none);
    }
}

template <int D>
__device__ __forceinline__ void dq_mma(uint8_t* smem, DqBars* bars, uint32_t tmem_base, int n_kv) {
    using Cfg = DqCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    constexpr uint32_t kIdescT = umma_idesc_bf16(128, 128, 0, 0);  // S, dP
    constexpr uint32_t kIdescdQ = umma_idesc_bf16(128, D, 0, 1);   // dQ: A from TMEM, B (K) MN-major
    const uint32_t hi = umma_desc_hi_sw128(1024);
    const uint32_t q_k = umma_desc_lo(smem_u32(smem + Cfg::kOffQ), 16);
    const uint32_t do_k = umma_desc_lo(smem_u32(smem + Cfg::kOffdO), 16);
    const uint32_t t_s = tmem_base + Cfg::kColS, t_dp = tmem_base + Cfg::kColdP, t_dq = tmem_base + Cfg::kColdQ;
    // The whole warp runs this role in uniform control flow; one elected lane issues.
    const bool el = elect_one();
    bool ok = mbar_wait(&bars->q_full, 0, abort_flag);
    for (int j = 0; j < n_kv && ok; ++j) {
        const int st = j % Cfg::kStages;
        ok = mbar_wait(&bars->kv_full[st], (j / Cfg::kStages) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t k_k = umma_desc_lo(smem_u32(smem + Cfg::kOffK + st * Cfg::kTileBytes), 16);
        const uint32_t v_k = umma_desc_lo(smem_u32(smem + Cfg::kOffV + st * Cfg::kTileBytes), 16);
        const uint32_t k_m = umma_desc_lo(smem_u32(smem + Cfg::kOffK + st * Cfg::kTileBytes), kHalfTileBytes);
        // S and dP columns are free: the dQ product of the previous tile, which read dS out of them, was
        // queued before this point (the pipe executes in order), after the rows had finished with dP.
        if (el) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = ((k / 4) * kHalfTileBytes + (k % 4) * 32) >> 4;
                umma_ss(t_s, umma_desc_join(q_k + off, hi), umma_desc_join(k_k + off, hi), kIdescT, k > 0 ? 1u : 0u);
            }
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = ((k / 4) * kHalfTileBytes + (k % 4) * 32) >> 4;
                umma_ss(t_dp, umma_desc_join(do_k + off, hi), umma_desc_join(v_k + off, hi), kIdescT, k > 0 ? 1u : 0u);
            }
            tc_commit(&bars->acc_full);
        }
        __syncwarp();
        ok = mbar_wait(&bars->ds_ready, j & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        // dQ += dS K_j: dS from TMEM (16 keys = 8 packed columns per instruction), K MN-major (rows = keys,
        // 64 head-dim elements per 128-byte row, the second 64-wide half 16 KB further).
        if (el) {
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k)
                umma_ts(t_dq, t_s + k * 8, umma_desc_join(k_m + k * 128, hi), kIdescdQ, (j > 0 || k > 0) ? 1u : 0u);
            tc_commit(&bars->kv_empty[st]);  // K_j and V_j are no longer read
            if (j + 1 == n_kv) tc_commit(&bars->dq_done);
        }
        __syncwarp();
    }
    if (!ok) {
        int none = 0;
        if (el) tc_commit(&bars->drain);
        __syncwarp();
        (void)mbar_wait(&bars->drain, 0, &none);
    }
}

template <int D, bool kCausal>
__device__ __forceinline__ void dq_rows(DqBars* bars, uint32_t tmem_base, const float* __restrict__ LSE,
                                        const float* __restrict__ Delta, __nv_bfloat16* __restrict__ dQ, int T, int qt,
                                        int bh, int n_kv, float scale, int warp, int lane) {
    using Cfg = DqCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (warp & 3);
    const int row_local = lane_base + lane;
    const int row = qt * kBlockQ + row_local;
    const uint32_t t_s = tmem_addr(tmem_base, lane_base, Cfg::kColS);
    const uint32_t t_dp = tmem_addr(tmem_base, lane_base, Cfg::kColdP);
    const uint32_t t_dq = tmem_addr(tmem_base, lane_base, Cfg::kColdQ);
    const float c = scale * kLog2e;
    const size_t idx = static_cast<size_t>(bh) * T + row;
    // Rows past the end of the sequence: LSE = +inf gives P = 0 everywhere.
    const float lse2 = (row < T) ? LSE[idx] * kLog2e : INFINITY;
    const float delta = (row < T) ? Delta[idx] : 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
        ok = mbar_wait(&bars->acc_full, j & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const bool diag = kCausal && (j == qt);
        const int keys_left = T - j * kBlockK;
        const int lim = diag ? min(row_local, keys_left - 1) : min(keys_left, kBlockK) - 1;
        // 32 keys at a time: their bf16 dS pairs (16 columns) land on S columns that have already been read.
#pragma unroll 1
        for (int cb = 0; cb < 128; cb += 32) {
            uint32_t sv[32], dv[32], ds[16];
            tmem_ld_x32(t_s + cb, sv);
            tmem_ld_x32(t_dp + cb, dv);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
                float p0 = ex2_approx(fmaf(__uint_as_float(sv[i + 0]), c, -lse2));
                float p1 = ex2_approx(fmaf(__uint_as_float(sv[i + 1]), c, -lse2));
                if (cb + i + 0 > lim) p0 = 0.f;
                if (cb + i + 1 > lim) p1 = 0.f;
                ds[i / 2] = pack_bf16x2(p0 * (__uint_as_float(dv[i + 0]) - delta), p1 * (__uint_as_float(dv[i + 1]) - delta));
            }
            tmem_st_x16(t_s + cb / 2, ds);
        }
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->ds_ready);
    }
    if (!ok) return;
    // dQ row = scale * accumulator, rounded once
    ok = mbar_wait(&bars->dq_done, 0, abort_flag);
    if (!ok) return;
    tc_fence_after();
    uint4* out = reinterpret_cast<uint4*>(dQ + idx * D);
#pragma unroll
    for (int cb = 0; cb < D; cb += 32) {
        uint32_t a[32];
        tmem_ld_x32(t_dq + cb, a);
        tmem_wait_ld();
        if (row < T) {
#pragma unroll
            for (int x = 0; x < 32; x += 8) {
                uint4 v;
                v.x = pack_bf16x2(__uint_as_float(a[x + 0]) * scale, __uint_as_float(a[x + 1]) * scale);
                v.y = pack_bf16x2(__uint_as_float(a[x + 2]) * scale, __uint_as_float(a[x + 3]) * scale);
                v.z = pack_bf16x2(__uint_as_float(a[x + 4]) * scale, __uint_as_float(a[x + 5]) * scale);
                v.w = pack_bf16x2(__uint_as_float(a[x + 6]) * scale, __uint_as_float(a[x + 7]) * scale);
                out[(cb + x) / 8] = v;
            }
        }
    }
}

template <int D, bool kCausal>
__global__ void __launch_bounds__(kDqThreads, 1)
attn_dq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
               const float* __restrict__ LSE, const float* __restrict__ Delta, __nv_bfloat16* __restrict__ dQ, int T,
               int BH, int n_q_tiles, float scale, int* __restrict__ dev_status) {
    using Cfg = DqCfg<D>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    DqBars* bars = reinterpret_cast<DqBars*>(smem + Cfg::kOffBar);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // heaviest query tiles (most key tiles under the causal clamp) first
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
        mbar_init(&bars->ds_ready, 4);
        mbar_init(&bars->dq_done, 1);
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmdO);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, kDqTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    griddep_launch_dependents();
    griddep_wait();  // everything above overlaps the previous kernel of the stream

    if (warp == 0) {
        if (lane == 0) dq_producer<D>(&tmQ, &tmK, &tmV, &tmdO, smem, bars, qt, bh, n_kv);
    } else if (warp == 1) {
        dq_mma<D>(smem, bars, tmem_base, n_kv);
    } else {
        dq_rows<D, kCausal>(bars, tmem_base, LSE, Delta, dQ, T, qt, bh, n_kv, scale, warp, lane);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kDqTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

template <int D, bool kCausal>
cudaError_t launch_one(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       const CUtensorMap& tmdO, const float* LSE, const float* Delta, __nv_bfloat16* dQ,
                       const AttnShape& s, int* dev_status, cudaStream_t stream) {
    const int n_q_tiles = (s.T + kBlockQ - 1) / kBlockQ;
    const int BH = s.B * s.H;
    return launch_overlapped(attn_dq_kernel<D, kCausal>, dim3(static_cast<unsigned>(n_q_tiles) * BH), dim3(kDqThreads),
                             DqCfg<D>::kSmemBytes, stream, tmQ, tmK, tmV, tmdO, LSE, Delta, dQ, s.T, BH, n_q_tiles,
                             s.scale, dev_status);
}

template <int D, bool kCausal>
cudaError_t configure_one() {
    return cudaFuncSetAttribute(attn_dq_kernel<D, kCausal>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                DqCfg<D>::kSmemBytes);
}

}  // namespace

cudaError_t configure_attn_dq() {
    const cudaError_t r[4] = {configure_one<64, true>(), configure_one<64, false>(), configure_one<128, true>(),
                              configure_one<128, false>()};
    for (cudaError_t e : r)
        if (e != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t launch_attn_dq(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                           const CUtensorMap& tmdO, const float* LSE, const float* Delta, __nv_bfloat16* dQ,
                           const AttnShape& s, int* dev_status, cudaStream_t stream) {
    if (s.D == 64) {
        return s.causal ? launch_one<64, true>(tmQ, tmK, tmV, tmdO, LSE, Delta, dQ, s, dev_status, stream)
                        : launch_one<64, false>(tmQ, tmK, tmV, tmdO, LSE, Delta, dQ, s, dev_status, stream);
    }
    return s.causal ? launch_one<128, true>(tmQ, tmK, tmV, tmdO, LSE, Delta, dQ, s, dev_status, stream)
                    : launch_one<128, false>(tmQ, tmK, tmV, tmdO, LSE, Delta, dQ, s, dev_status, stream);
}

}  // namespace nova
