// Fused causal attention backward for sm_100a (paper Section 4.2, "The Backward Pass": P is
// recomputed from the saved log-sum-exp, never stored; dQ reduces over keys, dK/dV over queries;
// the causal loop bound is raised so query tiles above the diagonal are never visited).
//
// One CTA owns one 128-key tile of one (batch, head), keeps K_j and V_j resident in shared memory
// and walks the query tiles i >= j.  Everything is computed transposed (keys on TMEM lanes) so that
// P^T and dS^T can feed the tensor cores straight from TMEM:
//   S^T  = K_j Q_i^T            (smem x smem -> TMEM)
//   dP^T = V_j dO_i^T           (smem x smem -> TMEM)
//   P^T  = exp2(S^T*c - LSE_i*log2e),  dS^T = P^T * (dP^T - Delta_i)      (compute warps, fp32)
//   dV  += P^T  dO_i            (TMEM x smem, dO read MN-major)
//   dK  += dS^T Q_i             (TMEM x smem, Q  read MN-major)
//   dQ_i = dS K_j               (dS^T staged as bf16 in shared memory and read M-major; K MN-major)
// dQ_i partial sums are added into an fp32 accumulator in global memory with vector red.add.
// Roles: warp 0 TMA producer, warp 1 UMMA issuer, warps 4..7 compute (one thread per key row).
#include "kernels.h"
#include "ptx.cuh"

namespace nova {
namespace {

constexpr int kBwdThreads = 256;
constexpr int kBwdTmemCols = 512;

template <int D>
struct BwdCfg {
    static constexpr int kHalves = D / kBoxCols;
    static constexpr int kTileBytes = kHalves * kHalfTileBytes;
    static constexpr int kStages = (D == 64) ? 2 : 1;
    static constexpr int kOffK = 0;
    static constexpr int kOffV = kTileBytes;
    static constexpr int kOffQ = 2 * kTileBytes;
    static constexpr int kOffdO = kOffQ + kStages * kTileBytes;
    static constexpr int kOffdS = kOffdO + kStages * kTileBytes;
    static constexpr int kOffRow = kOffdS + 2 * kHalfTileBytes;  // LSE*log2e and Delta of the query tile, 2 buffers
    static constexpr int kOffBar = kOffRow + 2 * 2 * 128 * 4;
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;
    // TMEM columns
    static constexpr int kColS = 0;      // S^T fp32 [0,128), then P^T bf16 in [0,64)
    static constexpr int kColdP = 128;   // dP^T fp32 [128,256), then dS^T bf16 in [128,192)
    static constexpr int kColdV = 256;
    static constexpr int kColdK = 256 + D;
    // dQ tile: its own columns at D=64; at D=128 the two 64-wide halves reuse the upper halves of
    // the S^T and dP^T regions, which are free once P^T / dS^T have been written.
    static constexpr int kColdQ0 = (D == 64) ? 384 : 64;
    static constexpr int kColdQ1 = 192;
    static constexpr bool kdQAliased = (D == 128);
};

struct BwdBars {
    uint64_t kv_full;
    uint64_t qdo_full[2], qdo_empty[2];
    uint64_t st_full, pds_ready, dq_full, dq_read, row_ready, drain;
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__device__ __forceinline__ void bwd_producer(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV,
                                             const CUtensorMap* tmdO, uint8_t* smem, BwdBars* bars, int kt, int bh,
                                             int i0, int n_it) {
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    int armed[2] = {-1, -1};
    mbar_expect_tx(&bars->kv_full, 2 * Cfg::kTileBytes);
#pragma unroll
    for (int h = 0; h < Cfg::kHalves; ++h) {
        tma_load_3d(smem + Cfg::kOffK + h * kHalfTileBytes, tmK, &bars->kv_full, h * kBoxCols, kt * kBlockK, bh);
        tma_load_3d(smem + Cfg::kOffV + h * kHalfTileBytes, tmV, &bars->kv_full, h * kBoxCols, kt * kBlockK, bh);
    }
    bool ok = true;
    for (int it = 0; it < n_it; ++it) {
        const int st = it % Cfg::kStages;
        const uint32_t ph = (it / Cfg::kStages) & 1;
        ok = mbar_wait(&bars->qdo_empty[st], ph ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(&bars->qdo_full[st], 2 * Cfg::kTileBytes);
        armed[st] = ph;
        const int qrow = (i0 + it) * kBlockQ;
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h) {
            tma_load_3d(smem + Cfg::kOffQ + st * Cfg::kTileBytes + h * kHalfTileBytes, tmQ, &bars->qdo_full[st],
                        h * kBoxCols, qrow, bh);
            tma_load_3d(smem + Cfg::kOffdO + st * Cfg::kTileBytes + h * kHalfTileBytes, tmdO, &bars->qdo_full[st],
                        h * kBoxCols, qrow, bh);
        }
    }
    if (!ok) {
        int none = 0;
        (void)mbar_wait(&bars->kv_full, 0, &none);
        for (int st = 0; st < Cfg::kStages; ++st)
            if (armed[st] >= 0) (void)mbar_wait(&bars->qdo_full[st], armed[st], &none);
    }
}

template <int D>
__device__ __forceinline__ void bwd_mma(uint8_t* smem, BwdBars* bars, uint32_t tmem_base, int n_it) {
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    constexpr uint32_t kIdescT = umma_idesc_bf16(128, 128, 0, 0);   // S^T, dP^T
    constexpr uint32_t kIdescKV = umma_idesc_bf16(128, D, 0, 1);    // dV, dK (A from TMEM, B MN-major)
    constexpr uint32_t kIdescdQ = umma_idesc_bf16(128, 64, 1, 1);   // dQ half (A M-major smem, B MN-major)
    const uint32_t sK = smem_u32(smem + Cfg::kOffK);
    const uint32_t sV = smem_u32(smem + Cfg::kOffV);
    const uint32_t sdS = smem_u32(smem + Cfg::kOffdS);
    const uint32_t t_s = tmem_base + Cfg::kColS, t_dp = tmem_base + Cfg::kColdP;
    const uint32_t t_dv = tmem_base + Cfg::kColdV, t_dk = tmem_base + Cfg::kColdK;

    bool ok = mbar_wait(&bars->kv_full, 0, abort_flag);
    for (int it = 0; it < n_it && ok; ++it) {
        const int st = it % Cfg::kStages;
        const uint32_t ph = (it / Cfg::kStages) & 1;
        if (Cfg::kdQAliased && it > 0) {
            ok = mbar_wait(&bars->dq_read, (it - 1) & 1, abort_flag);
            if (!ok) break;
        }
        ok = mbar_wait(&bars->qdo_full[st], ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sQ = smem_u32(smem + Cfg::kOffQ + st * Cfg::kTileBytes);
        const uint32_t sdO = smem_u32(smem + Cfg::kOffdO + st * Cfg::kTileBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * kHalfTileBytes + (k % 4) * 32;
            umma_ss(t_s, umma_smem_desc_sw128(sK + off, 16, 1024), umma_smem_desc_sw128(sQ + off, 16, 1024), kIdescT,
                    k > 0 ? 1u : 0u);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * kHalfTileBytes + (k % 4) * 32;
            umma_ss(t_dp, umma_smem_desc_sw128(sV + off, 16, 1024), umma_smem_desc_sw128(sdO + off, 16, 1024), kIdescT,
                    k > 0 ? 1u : 0u);
        }
        tc_commit(&bars->st_full);
        ok = mbar_wait(&bars->pds_ready, it & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        // dV += P^T dO_i and dK += dS^T Q_i: 16 queries (8 packed TMEM columns, 16 smem rows) per instruction.
#pragma unroll
        for (int k = 0; k < kBlockQ / 16; ++k)
            umma_ts(t_dv, t_s + k * 8, umma_smem_desc_sw128(sdO + k * 2048, kHalfTileBytes, 1024), kIdescKV,
                    (it > 0 || k > 0) ? 1u : 0u);
#pragma unroll
        for (int k = 0; k < kBlockQ / 16; ++k)
            umma_ts(t_dk, t_dp + k * 8, umma_smem_desc_sw128(sQ + k * 2048, kHalfTileBytes, 1024), kIdescKV,
                    (it > 0 || k > 0) ? 1u : 0u);
        tc_commit(&bars->qdo_empty[st]);
        // dQ_i = dS K_j, 64 head-dim columns per accumulator; 16 keys per instruction.
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h) {
            const uint32_t t_dq = tmem_base + (h == 0 ? Cfg::kColdQ0 : Cfg::kColdQ1);
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k)
                umma_ss(t_dq, umma_smem_desc_sw128(sdS + k * 2048, kHalfTileBytes, 1024),
                        umma_smem_desc_sw128(sK + h * kHalfTileBytes + k * 2048, kHalfTileBytes, 1024), kIdescdQ,
                        k > 0 ? 1u : 0u);
        }
        tc_commit(&bars->dq_full);
    }
    if (!ok) {
        int none = 0;
        tc_commit(&bars->drain);
        (void)mbar_wait(&bars->drain, 0, &none);
    }
}

template <int D, bool kCausal>
__device__ __forceinline__ void bwd_compute(uint8_t* smem, BwdBars* bars, uint32_t tmem_base,
                                            const float* __restrict__ LSE, const float* __restrict__ Delta,
                                            float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dK,
                                            __nv_bfloat16* __restrict__ dV, int T, int kt, int bh, int i0, int n_it,
                                            float scale, int warp, int lane) {
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (warp & 3);
    const int r = lane_base + lane;          // local key row (S^T, dP^T, dV, dK) / local query row (dQ)
    const int key = kt * kBlockK + r;
    const bool key_valid = key < T;
    const float c = scale * kLog2e;
    const uint32_t t_s = tmem_addr(tmem_base, lane_base, Cfg::kColS);
    const uint32_t t_dp = tmem_addr(tmem_base, lane_base, Cfg::kColdP);
    float* row_buf = reinterpret_cast<float*>(smem + Cfg::kOffRow);
    uint8_t* sdS = smem + Cfg::kOffdS;
    const size_t row_base = static_cast<size_t>(bh) * T;
    bool ok = true;

    for (int it = 0; it < n_it; ++it) {
        const int i = i0 + it;
        float* s_lse = row_buf + (it & 1) * 256;
        float* s_dl = s_lse + 128;
        {
            const int q = i * kBlockQ + r;
            // Rows past the end of the sequence get LSE = +inf so that their P is exactly 0.
            s_lse[r] = (q < T) ? LSE[row_base + q] * kLog2e : INFINITY;
            s_dl[r] = (q < T) ? Delta[row_base + q] : 0.f;
        }
        mbar_arrive(&bars->row_ready);  // bounded stand-in for a named barrier among the compute warps
        ok = mbar_wait(&bars->row_ready, it & 1, abort_flag);
        if (!ok) break;
        ok = mbar_wait(&bars->st_full, it & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const bool diag = kCausal && (i == kt);
#pragma unroll 1
        for (int cb = 0; cb < 4; ++cb) {
            uint32_t sv[32], dv[32];
            tmem_ld_x32(t_s + cb * 32, sv);
            tmem_ld_x32(t_dp + cb * 32, dv);
            tmem_wait_ld();
            uint32_t pp[16], dd[16];
#pragma unroll
            for (int q = 0; q < 32; q += 2) {
                const int q0 = cb * 32 + q;
                float p0 = ex2_approx(fmaf(__uint_as_float(sv[q]), c, -s_lse[q0]));
                float p1 = ex2_approx(fmaf(__uint_as_float(sv[q + 1]), c, -s_lse[q0 + 1]));
                // keep (query q, key r) iff the key exists and, on the diagonal tile, key <= query
                if (!key_valid || (diag && r > q0)) p0 = 0.f;
                if (!key_valid || (diag && r > q0 + 1)) p1 = 0.f;
                const float d0 = p0 * (__uint_as_float(dv[q]) - s_dl[q0]);
                const float d1 = p1 * (__uint_as_float(dv[q + 1]) - s_dl[q0 + 1]);
                pp[q / 2] = pack_bf16x2(p0, p1);
                dd[q / 2] = pack_bf16x2(d0, d1);
            }
            tmem_st_x16(t_s + cb * 16, pp);
            tmem_st_x16(t_dp + cb * 16, dd);
            // dS^T row r, queries [32cb, 32cb+32): four 16-byte chunks of the 128-byte swizzled row.
            uint8_t* row_ptr = sdS + (cb >> 1) * kHalfTileBytes + r * 128;
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                const int chunk = (cb & 1) * 4 + ch;
                *reinterpret_cast<uint4*>(row_ptr + ((chunk ^ (r & 7)) << 4)) =
                    make_uint4(dd[ch * 4 + 0], dd[ch * 4 + 1], dd[ch * 4 + 2], dd[ch * 4 + 3]);
            }
        }
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before();
        mbar_arrive(&bars->pds_ready);

        ok = mbar_wait(&bars->dq_full, it & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        {
            const int q = i * kBlockQ + r;
            float* dst = dq_acc + (row_base + q) * D;
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h) {
                const uint32_t t_dq = tmem_addr(tmem_base, lane_base, h == 0 ? Cfg::kColdQ0 : Cfg::kColdQ1);
#pragma unroll
                for (int cb = 0; cb < 64; cb += 32) {
                    uint32_t a[32];
                    tmem_ld_x32(t_dq + cb, a);
                    tmem_wait_ld();
                    if (q < T) {
#pragma unroll
                        for (int x = 0; x < 32; x += 4)
                            red_add_v4_f32(dst + h * 64 + cb + x, __uint_as_float(a[x]), __uint_as_float(a[x + 1]),
                                           __uint_as_float(a[x + 2]), __uint_as_float(a[x + 3]));
                    }
                }
            }
        }
        if (Cfg::kdQAliased) {
            tc_fence_before();
            mbar_arrive(&bars->dq_read);
        }
    }
    if (!ok) return;
    // All UMMAs are complete (the last dq_full commit covers them): write dV and dK for this key tile.
    const uint32_t t_dv = tmem_addr(tmem_base, lane_base, Cfg::kColdV);
    const uint32_t t_dk = tmem_addr(tmem_base, lane_base, Cfg::kColdK);
    uint4* dv_row = reinterpret_cast<uint4*>(dV + (row_base + key) * D);
    uint4* dk_row = reinterpret_cast<uint4*>(dK + (row_base + key) * D);
#pragma unroll
    for (int cb = 0; cb < D; cb += 32) {
        uint32_t a[32], b[32];
        tmem_ld_x32(t_dv + cb, a);
        tmem_ld_x32(t_dk + cb, b);
        tmem_wait_ld();
        if (key_valid) {
#pragma unroll
            for (int x = 0; x < 32; x += 8) {
                uint4 v, w;
                v.x = pack_bf16x2(__uint_as_float(a[x + 0]), __uint_as_float(a[x + 1]));
                v.y = pack_bf16x2(__uint_as_float(a[x + 2]), __uint_as_float(a[x + 3]));
                v.z = pack_bf16x2(__uint_as_float(a[x + 4]), __uint_as_float(a[x + 5]));
                v.w = pack_bf16x2(__uint_as_float(a[x + 6]), __uint_as_float(a[x + 7]));
                w.x = pack_bf16x2(__uint_as_float(b[x + 0]) * scale, __uint_as_float(b[x + 1]) * scale);
                w.y = pack_bf16x2(__uint_as_float(b[x + 2]) * scale, __uint_as_float(b[x + 3]) * scale);
                w.z = pack_bf16x2(__uint_as_float(b[x + 4]) * scale, __uint_as_float(b[x + 5]) * scale);
                w.w = pack_bf16x2(__uint_as_float(b[x + 6]) * scale, __uint_as_float(b[x + 7]) * scale);
                dv_row[(cb + x) / 8] = v;
                dk_row[(cb + x) / 8] = w;
            }
        }
    }
}

template <int D, bool kCausal>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                const float* __restrict__ LSE, const float* __restrict__ Delta, float* __restrict__ dq_acc,
                __nv_bfloat16* __restrict__ dK, __nv_bfloat16* __restrict__ dV, int T, int BH, int n_tiles,
                float scale, int* __restrict__ dev_status) {
    using Cfg = BwdCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    BwdBars* bars = reinterpret_cast<BwdBars*>(smem + Cfg::kOffBar);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Key tile 0 sees every query tile under the causal clamp, so low key tiles go first.
    const int kt = static_cast<int>(blockIdx.x) / BH;
    const int bh = static_cast<int>(blockIdx.x) % BH;
    const int i0 = kCausal ? kt : 0;  // raised lower bound of the query loop
    const int n_it = n_tiles - i0;

    if (threadIdx.x == 0) {
        mbar_init(&bars->kv_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->qdo_full[s], 1);
            mbar_init(&bars->qdo_empty[s], 1);
        }
        mbar_init(&bars->st_full, 1);
        mbar_init(&bars->pds_ready, 128);
        mbar_init(&bars->dq_full, 1);
        mbar_init(&bars->dq_read, 128);
        mbar_init(&bars->row_ready, 128);
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmdO);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, kBwdTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        if (lane == 0) bwd_producer<D>(&tmQ, &tmK, &tmV, &tmdO, smem, bars, kt, bh, i0, n_it);
    } else if (warp == 1) {
        if (lane == 0) bwd_mma<D>(smem, bars, tmem_base, n_it);
    } else if (warp >= 4) {
        bwd_compute<D, kCausal>(smem, bars, tmem_base, LSE, Delta, dq_acc, dK, dV, T, kt, bh, i0, n_it, scale, warp,
                                lane);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kBwdTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

template <int D, bool kCausal>
cudaError_t launch_one(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       const CUtensorMap& tmdO, const float* LSE, const float* Delta, float* dq_acc,
                       __nv_bfloat16* dK, __nv_bfloat16* dV, const AttnShape& s, int* dev_status,
                       cudaStream_t stream) {
    const int n_tiles = (s.T + kBlockK - 1) / kBlockK;
    const int BH = s.B * s.H;
    const dim3 grid(static_cast<unsigned>(n_tiles) * BH);
    attn_bwd_kernel<D, kCausal><<<grid, kBwdThreads, BwdCfg<D>::kSmemBytes, stream>>>(
        tmQ, tmK, tmV, tmdO, LSE, Delta, dq_acc, dK, dV, s.T, BH, n_tiles, s.scale, dev_status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t configure_attn_bwd() {
    cudaError_t e;
    e = cudaFuncSetAttribute(attn_bwd_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_bwd_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_bwd_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_bwd_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdCfg<128>::kSmemBytes);
    return e;
}

cudaError_t launch_attn_bwd(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            const CUtensorMap& tmdO, const float* LSE, const float* Delta, float* dq_acc,
                            __nv_bfloat16* dK, __nv_bfloat16* dV, const AttnShape& s, int* dev_status,
                            cudaStream_t stream) {
    if (s.D == 64) {
        return s.causal ? launch_one<64, true>(tmQ, tmK, tmV, tmdO, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream)
                        : launch_one<64, false>(tmQ, tmK, tmV, tmdO, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream);
    }
    return s.causal ? launch_one<128, true>(tmQ, tmK, tmV, tmdO, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream)
                    : launch_one<128, false>(tmQ, tmK, tmV, tmdO, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream);
}

}  // namespace nova
