// Fused causal attention forward for sm_100a (paper Section 4.2: score contraction, index mask,
// base-2 online softmax, value contraction, causal loop clamp, 1/sum epilogue, LSE saved).
//
// One CTA owns one 128-row query tile of one (batch, head) and walks the key tiles up to the
// diagonal.  Roles:
//   warp 0      TMA producer: Q once, then K and V tiles through mbarrier-guarded rings
//   warp 1      UMMA issuer:  S = Q K^T  (operands in shared memory, accumulator in TMEM)
//                             O += P V   (P read from TMEM as bf16, V from shared memory)
//   warps 2..5  softmax: one thread per query row reads its S row from TMEM, keeps the running
//               max / sum in registers, writes bf16 P back over S, rescales O in TMEM only when the
//               row maximum has grown by more than 2^8 (exact: the final 1/sum and the LSE use the
//               same reference maximum), and runs the epilogue.
// TMEM: columns [0,128) hold S (fp32) then P (bf16 pairs in [0,64)); [128,128+D) hold O (fp32).
// Two CTAs are resident per SM, so one CTA's softmax overlaps the other's tensor-core work.
#include "kernels.h"
#include "ptx.cuh"

namespace nova {
namespace {

constexpr int kFwdThreads = 192;
constexpr int kFwdTmemCols = 256;
constexpr int kColS = 0;
constexpr int kColO = 128;
constexpr float kRescaleThreshold = 8.0f;  // log2 units

template <int D>
struct FwdCfg {
    static constexpr int kHalves = D / kBoxCols;
    static constexpr int kTileBytes = kHalves * kHalfTileBytes;
    static constexpr int kStages = (D == 64) ? 2 : 1;
    static constexpr int kOffQ = 0;
    static constexpr int kOffK = kTileBytes;
    static constexpr int kOffV = kTileBytes * (1 + kStages);
    static constexpr int kOffBar = kTileBytes * (1 + 2 * kStages);
    static constexpr int kSmemBytes = kOffBar + 256 + 1024;  // + barriers + alignment slack
};

struct FwdBars {
    uint64_t q_full;
    uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];
    uint64_t s_full, p_ready, pv_done, drain;
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__device__ __forceinline__ void fwd_producer(const CUtensorMap* tmQ, const CUtensorMap* tmK,
                                             const CUtensorMap* tmV, uint8_t* smem, FwdBars* bars, int qt, int bh,
                                             int n_kv) {
    using Cfg = FwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    int armed_k[2] = {-1, -1}, armed_v[2] = {-1, -1};
    mbar_expect_tx(&bars->q_full, Cfg::kTileBytes);
#pragma unroll
    for (int h = 0; h < Cfg::kHalves; ++h)
        tma_load_3d(smem + Cfg::kOffQ + h * kHalfTileBytes, tmQ, &bars->q_full, h * kBoxCols, qt * kBlockQ, bh);
    bool ok = true;
    for (int j = 0; j < n_kv && ok; ++j) {
        const int st = j % Cfg::kStages;
        const uint32_t ph = (j / Cfg::kStages) & 1;
        ok = mbar_wait(&bars->k_empty[st], ph ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(&bars->k_full[st], Cfg::kTileBytes);
        armed_k[st] = ph;
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_3d(smem + Cfg::kOffK + st * Cfg::kTileBytes + h * kHalfTileBytes, tmK, &bars->k_full[st],
                        h * kBoxCols, j * kBlockK, bh);
        ok = mbar_wait(&bars->v_empty[st], ph ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(&bars->v_full[st], Cfg::kTileBytes);
        armed_v[st] = ph;
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_3d(smem + Cfg::kOffV + st * Cfg::kTileBytes + h * kHalfTileBytes, tmV, &bars->v_full[st],
                        h * kBoxCols, j * kBlockK, bh);
    }
    if (!ok) {
        // Giving up: let the copies already in flight land before the CTA (and its shared memory) goes away.
        int none = 0;
        (void)mbar_wait(&bars->q_full, 0, &none);
        for (int st = 0; st < Cfg::kStages; ++st) {
            if (armed_k[st] >= 0) (void)mbar_wait(&bars->k_full[st], armed_k[st], &none);
            if (armed_v[st] >= 0) (void)mbar_wait(&bars->v_full[st], armed_v[st], &none);
        }
    }
}

template <int D>
__device__ __forceinline__ void fwd_mma(uint8_t* smem, FwdBars* bars, uint32_t tmem_base, int n_kv) {
    using Cfg = FwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    constexpr uint32_t kIdescQK = umma_idesc_bf16(128, 128, 0, 0);
    constexpr uint32_t kIdescPV = umma_idesc_bf16(128, D, 0, 1);
    const uint32_t sQ = smem_u32(smem + Cfg::kOffQ);
    const uint32_t t_s = tmem_base + kColS;
    const uint32_t t_o = tmem_base + kColO;
    bool ok = mbar_wait(&bars->q_full, 0, abort_flag);
    for (int j = 0; j < n_kv && ok; ++j) {
        const int st = j % Cfg::kStages;
        const uint32_t ph = (j / Cfg::kStages) & 1;
        ok = mbar_wait(&bars->k_full[st], ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sK = smem_u32(smem + Cfg::kOffK + st * Cfg::kTileBytes);
        // S = Q K^T: both operands K-major; 16 head-dim elements (32 bytes) per instruction.
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * kHalfTileBytes + (k % 4) * 32;
            umma_ss(t_s, umma_smem_desc_sw128(sQ + off, 16, 1024), umma_smem_desc_sw128(sK + off, 16, 1024),
                    kIdescQK, k > 0 ? 1u : 0u);
        }
        tc_commit(&bars->k_empty[st]);
        tc_commit(&bars->s_full);
        ok = mbar_wait(&bars->p_ready, j & 1, abort_flag);
        if (!ok) break;
        ok = mbar_wait(&bars->v_full[st], ph, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t sV = smem_u32(smem + Cfg::kOffV + st * Cfg::kTileBytes);
        // O += P V: P from TMEM (16 keys = 8 packed columns per instruction), V is MN-major
        // (rows = keys, 64 head-dim elements per 128-byte row, second 64-wide half at +16 KB).
#pragma unroll
        for (int k = 0; k < kBlockK / 16; ++k) {
            umma_ts(t_o, t_s + k * 8, umma_smem_desc_sw128(sV + k * 2048, kHalfTileBytes, 1024), kIdescPV,
                    (j > 0 || k > 0) ? 1u : 0u);
        }
        tc_commit(&bars->v_empty[st]);
        tc_commit(&bars->pv_done);
    }
    if (!ok) {
        // Drain whatever was issued before leaving so TMEM can be released safely.
        int none = 0;
        tc_commit(&bars->drain);
        (void)mbar_wait(&bars->drain, 0, &none);
    }
}

template <int D, bool kCausal>
__device__ __forceinline__ void fwd_softmax(FwdBars* bars, uint32_t tmem_base, __nv_bfloat16* O, float* LSE, int T,
                                            int qt, int bh, int n_kv, float scale, int warp, int lane) {
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (warp & 3);
    const int row_local = lane_base + lane;
    const int row = qt * kBlockQ + row_local;
    const uint32_t t_s = tmem_addr(tmem_base, lane_base, kColS);
    const uint32_t t_o = tmem_addr(tmem_base, lane_base, kColO);
    const float c = scale * kLog2e;
    float m_ref = -INFINITY;  // reference maximum of the raw (unscaled) scores
    float l = 0.f;
    bool ok = true;

    for (int j = 0; j < n_kv; ++j) {
        ok = mbar_wait(&bars->s_full, j & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        uint32_t sr[128];
        tmem_ld_x32(t_s + 0, sr + 0);
        tmem_ld_x32(t_s + 32, sr + 32);
        tmem_ld_x32(t_s + 64, sr + 64);
        tmem_ld_x32(t_s + 96, sr + 96);
        tmem_wait_ld();

        // Mask from indices only: the diagonal tile keeps key <= query; a ragged last tile keeps key < T.
        const bool diag = kCausal && (j == qt);
        const int keys_left = T - j * kBlockK;
        if (diag || keys_left < kBlockK) {
            const int lim = diag ? min(row_local, keys_left - 1) : keys_left - 1;
#pragma unroll
            for (int i = 0; i < 128; ++i)
                if (i > lim) sr[i] = 0xff800000u;  // -inf
        }
        float mx0 = __uint_as_float(sr[0]), mx1 = __uint_as_float(sr[1]), mx2 = __uint_as_float(sr[2]),
              mx3 = __uint_as_float(sr[3]);
#pragma unroll
        for (int i = 4; i < 128; i += 4) {
            mx0 = fmaxf(mx0, __uint_as_float(sr[i]));
            mx1 = fmaxf(mx1, __uint_as_float(sr[i + 1]));
            mx2 = fmaxf(mx2, __uint_as_float(sr[i + 2]));
            mx3 = fmaxf(mx3, __uint_as_float(sr[i + 3]));
        }
        const float m_tile = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));

        if (j == 0) {
            m_ref = m_tile;
        } else {
            const float m_new = fmaxf(m_ref, m_tile);
            const bool grow = (m_new - m_ref) * c > kRescaleThreshold;
            if (__any_sync(0xffffffffu, grow)) {
                const float f = ex2_approx((m_ref - m_new) * c);  // 1 for rows whose maximum did not move
                m_ref = m_new;
                l *= f;
                ok = mbar_wait(&bars->pv_done, (j - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int cb = 0; cb < D; cb += 32) {
                    uint32_t o[32];
                    tmem_ld_x32(t_o + cb, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                    tmem_st_x32(t_o + cb, o);
                }
            }
        }
        const float mc = m_ref * c;
        float l0 = 0.f, l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
        for (int cb = 0; cb < 128; cb += 64) {
            uint32_t pk[32];
#pragma unroll
            for (int i = 0; i < 64; i += 4) {
                const float p0 = ex2_approx(fmaf(__uint_as_float(sr[cb + i + 0]), c, -mc));
                const float p1 = ex2_approx(fmaf(__uint_as_float(sr[cb + i + 1]), c, -mc));
                const float p2 = ex2_approx(fmaf(__uint_as_float(sr[cb + i + 2]), c, -mc));
                const float p3 = ex2_approx(fmaf(__uint_as_float(sr[cb + i + 3]), c, -mc));
                l0 += p0; l1 += p1; l2 += p2; l3 += p3;
                pk[i / 2] = pack_bf16x2(p0, p1);
                pk[i / 2 + 1] = pack_bf16x2(p2, p3);
            }
            tmem_st_x32(t_s + cb / 2, pk);
        }
        l += (l0 + l1) + (l2 + l3);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->p_ready);
    }

    if (ok) ok = mbar_wait(&bars->pv_done, (n_kv - 1) & 1, abort_flag);
    if (!ok) return;
    tc_fence_after();
    const float inv_l = 1.0f / l;
    const bool valid = row < T;
    uint4* orow = reinterpret_cast<uint4*>(O + (static_cast<size_t>(bh) * T + row) * D);
#pragma unroll
    for (int cb = 0; cb < D; cb += 32) {
        uint32_t o[32];
        tmem_ld_x32(t_o + cb, o);
        tmem_wait_ld();
        if (valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
                uint4 v;
                v.x = pack_bf16x2(__uint_as_float(o[i + 0]) * inv_l, __uint_as_float(o[i + 1]) * inv_l);
                v.y = pack_bf16x2(__uint_as_float(o[i + 2]) * inv_l, __uint_as_float(o[i + 3]) * inv_l);
                v.z = pack_bf16x2(__uint_as_float(o[i + 4]) * inv_l, __uint_as_float(o[i + 5]) * inv_l);
                v.w = pack_bf16x2(__uint_as_float(o[i + 6]) * inv_l, __uint_as_float(o[i + 7]) * inv_l);
                orow[(cb + i) / 8] = v;
            }
        }
    }
    if (valid) LSE[static_cast<size_t>(bh) * T + row] = m_ref * scale + logf(l);
}

template <int D, bool kCausal>
__global__ void __launch_bounds__(kFwdThreads, 2)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, __nv_bfloat16* __restrict__ O, float* __restrict__ LSE,
                int T, int BH, int n_q_tiles, float scale, int* __restrict__ dev_status) {
    using Cfg = FwdCfg<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    FwdBars* bars = reinterpret_cast<FwdBars*>(smem + Cfg::kOffBar);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // Heaviest query tiles (most key tiles under the causal clamp) are scheduled first.
    const int qt = n_q_tiles - 1 - static_cast<int>(blockIdx.x) / BH;
    const int bh = static_cast<int>(blockIdx.x) % BH;
    const int n_kv_all = (T + kBlockK - 1) / kBlockK;
    const int n_kv = kCausal ? min(qt + 1, n_kv_all) : n_kv_all;  // causal clamp of the key loop

    if (threadIdx.x == 0) {
        mbar_init(&bars->q_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->k_full[s], 1);
            mbar_init(&bars->k_empty[s], 1);
            mbar_init(&bars->v_full[s], 1);
            mbar_init(&bars->v_empty[s], 1);
        }
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->p_ready, 128);
        mbar_init(&bars->pv_done, 1);
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, kFwdTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        if (lane == 0) fwd_producer<D>(&tmQ, &tmK, &tmV, smem, bars, qt, bh, n_kv);
    } else if (warp == 1) {
        if (lane == 0) fwd_mma<D>(smem, bars, tmem_base, n_kv);
    } else {
        fwd_softmax<D, kCausal>(bars, tmem_base, O, LSE, T, qt, bh, n_kv, scale, warp, lane);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kFwdTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

template <int D, bool kCausal>
cudaError_t launch_one(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV, __nv_bfloat16* O,
                       float* LSE, const AttnShape& s, int* dev_status, cudaStream_t stream) {
    const int n_q_tiles = (s.T + kBlockQ - 1) / kBlockQ;
    const int BH = s.B * s.H;
    const dim3 grid(static_cast<unsigned>(n_q_tiles) * BH);
    attn_fwd_kernel<D, kCausal><<<grid, kFwdThreads, FwdCfg<D>::kSmemBytes, stream>>>(
        tmQ, tmK, tmV, O, LSE, s.T, BH, n_q_tiles, s.scale, dev_status);
    return cudaGetLastError();
}

}  // namespace

cudaError_t configure_attn_fwd() {
    cudaError_t e;
    e = cudaFuncSetAttribute(attn_fwd_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_fwd_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<64>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_fwd_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<128>::kSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(attn_fwd_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdCfg<128>::kSmemBytes);
    return e;
}

cudaError_t launch_attn_fwd(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            __nv_bfloat16* O, float* LSE, const AttnShape& s, int* dev_status,
                            cudaStream_t stream) {
    if (s.D == 64) {
        return s.causal ? launch_one<64, true>(tmQ, tmK, tmV, O, LSE, s, dev_status, stream)
                        : launch_one<64, false>(tmQ, tmK, tmV, O, LSE, s, dev_status, stream);
    }
    return s.causal ? launch_one<128, true>(tmQ, tmK, tmV, O, LSE, s, dev_status, stream)
                    : launch_one<128, false>(tmQ, tmK, tmV, O, LSE, s, dev_status, stream);
}

}  // namespace nova
