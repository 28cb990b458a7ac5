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
//
// Warp roles (512 threads):
//   warp 0       TMA producer (K_j, V_j once; Q_i double-buffered; dO_i single-buffered)
//   warp 1       UMMA issuer, software-pipelined: while the compute warps work on dS of tile i the
//                tensor core runs dV(i) and S^T(i+1); while they work on P of tile i+1 it runs dK(i),
//                dQ(i) and dP^T(i+1)
//   warps 2-3    row loader: LSE*log2e and Delta of the query tile into shared memory
//   warps 4-11   compute: thread = (key row, 64-query half); P phase then dS phase per tile
//   warps 12-15  dQ: one thread per query row moves the partial dQ tile from TMEM into the fp32
//                accumulator (TMA reduce-add through a swizzled staging buffer at D=64,
//                red.global.add.v4.f32 at D=128); a separate kernel scales and rounds it once
//
// TMEM columns (D=64): S^T [0,128)  dP^T/dS^T [128,256)  dV [256,320)  dK [320,384)  dQ [384,448)
//                      P^T [448,512): P^T has its own columns, so S^T of the next query tile is
//                      issued before dV of the current one and the compute warps never wait for it
//              (D=128): S^T/P^T [0,128)  dP^T/dS^T, then dQ [128,256)  dV [256,384)  dK [384,512)
// Where bf16 P^T / dS^T share columns with the fp32 tile they came from, query half h writes only
// over its own already-read columns [64h, 64h+32), so the two compute warpgroups never collide.
#include "kernels.h"
#include "ptx.cuh"

#ifdef NOVA_EXP_TRACE
__device__ long long g_blk[4096 * 4];
extern "C" int nova_exp_read_blk(long long* out) { return (int)cudaMemcpyFromSymbol(out, g_blk, sizeof(long long) * 4096 * 4); }
__device__ long long g_trace[8 * 256];
#define TRACE(slot, idx) do { if (blockIdx.x == 0) g_trace[(slot) * 256 + (idx)] = clock64(); } while (0)
extern "C" int nova_exp_read_trace(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, g_trace, sizeof(long long) * 8 * 256);
}
#else
#define TRACE(slot, idx) do { } while (0)
#endif

namespace nova {
namespace {

constexpr int kBwdThreads = 512;
constexpr int kBwdTmemCols = 512;
constexpr int kComputeThreads = 256;

template <int D>
struct BwdCfg {
    static constexpr int kHalves = D / kBoxCols;
    static constexpr int kTileBytes = kHalves * kHalfTileBytes;
    static constexpr int kOffK = 0;
    static constexpr int kOffV = kTileBytes;
    static constexpr int kOffQ = 2 * kTileBytes;               // 2 stages
    static constexpr int kOffdO = 4 * kTileBytes;              // 1 stage
    static constexpr int kOffdS = 5 * kTileBytes;              // [2 query halves][128 keys][64 queries] bf16
    static constexpr int kOffRow = kOffdS + 2 * kHalfTileBytes;  // 2 x (LSE*log2e[128], Delta[128]) fp32
    // dQ staging for the bulk reduction (D=64 only): 2 buffers x 128 rows x (256 + 16) bytes; the
    // 16-byte pad keeps the per-row 16-byte stores of a warp on distinct banks.
    // dQ staging for the TMA reduction (D=64 only): 2 buffers x 2 boxes of [128 rows x 32 fp32],
    // 128-byte swizzled like every other tile.
    static constexpr bool kBulkdQ = (D == 64);
    static constexpr int kStageBytes = 2 * kHalfTileBytes;
    static constexpr int kOffStage = kOffRow + 2 * 2 * 128 * 4;
    static constexpr int kOffBar = kOffStage + (kBulkdQ ? 2 * kStageBytes : 0);
    static constexpr int kSmemBytes = kOffBar + 512 + 1024;
    static constexpr int kColS = 0;
    static constexpr int kColdP = 128;
    static constexpr int kColdV = 256;
    static constexpr int kColdK = 256 + D;
    static constexpr bool kdQAliased = (D == 128);  // dQ reuses the dP^T region
    static constexpr int kColdQ = (D == 64) ? 384 : 128;
    static constexpr bool kSeparateP = (D == 64);   // P^T in its own columns instead of over S^T
    static constexpr int kColP = kSeparateP ? 448 : 0;
    static constexpr int kPHalfStride = kSeparateP ? 32 : 64;  // column distance between the two query halves of P^T
};

struct BwdBars {
    uint64_t kv_full;
    uint64_t q_full[2], q_empty[2];
    uint64_t do_full, do_empty;
    uint64_t s_full, dp_full;       // UMMA -> compute
    uint64_t p_ready, ds_ready;     // compute (256 arrivals) -> UMMA
    uint64_t dq_full, dq_free;
    uint64_t row_full[2], row_empty[2];
    uint64_t stage_full, stage_free;  // dQ warps <-> their leader thread
    uint64_t mma_done, drain;
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__device__ __forceinline__ void bwd_producer(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV,
                                             const CUtensorMap* tmdO, uint8_t* smem, BwdBars* bars, int kt, int bh,
                                             int i0, int n_it) {
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    int armed_q[2] = {-1, -1}, armed_do = -1;
    mbar_expect_tx(&bars->kv_full, 2 * Cfg::kTileBytes);
#pragma unroll
    for (int h = 0; h < Cfg::kHalves; ++h) {
        tma_load_3d(smem + Cfg::kOffK + h * kHalfTileBytes, tmK, &bars->kv_full, h * kBoxCols, kt * kBlockK, bh);
        tma_load_3d(smem + Cfg::kOffV + h * kHalfTileBytes, tmV, &bars->kv_full, h * kBoxCols, kt * kBlockK, bh);
    }
    bool ok = true;
    for (int it = 0; it < n_it; ++it) {
        const int st = it & 1;
        const int qrow = (i0 + it) * kBlockQ;
        ok = mbar_wait(&bars->q_empty[st], ((it >> 1) & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(&bars->q_full[st], Cfg::kTileBytes);
        armed_q[st] = (it >> 1) & 1;
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_3d(smem + Cfg::kOffQ + st * Cfg::kTileBytes + h * kHalfTileBytes, tmQ, &bars->q_full[st],
                        h * kBoxCols, qrow, bh);
        ok = mbar_wait(&bars->do_empty, (it & 1) ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(&bars->do_full, Cfg::kTileBytes);
        armed_do = it & 1;
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h)
            tma_load_3d(smem + Cfg::kOffdO + h * kHalfTileBytes, tmdO, &bars->do_full, h * kBoxCols, qrow, bh);
    }
    if (!ok) {
        // Giving up: let the copies already in flight land before the CTA's shared memory goes away.
        int none = 0;
        (void)mbar_wait(&bars->kv_full, 0, &none);
        for (int st = 0; st < 2; ++st)
            if (armed_q[st] >= 0) (void)mbar_wait(&bars->q_full[st], armed_q[st], &none);
        if (armed_do >= 0) (void)mbar_wait(&bars->do_full, armed_do, &none);
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
    const uint32_t sdO = smem_u32(smem + Cfg::kOffdO);
    const uint32_t sdS = smem_u32(smem + Cfg::kOffdS);
    const uint32_t t_s = tmem_base + Cfg::kColS, t_dp = tmem_base + Cfg::kColdP;
    const uint32_t t_dv = tmem_base + Cfg::kColdV, t_dk = tmem_base + Cfg::kColdK;

    auto issue_st = [&](int it) {  // S^T(it) = K_j Q_it^T
        const uint32_t sQ = smem_u32(smem + Cfg::kOffQ + (it & 1) * Cfg::kTileBytes);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * kHalfTileBytes + (k % 4) * 32;
            umma_ss(t_s, umma_smem_desc_sw128(sK + off, 16, 1024), umma_smem_desc_sw128(sQ + off, 16, 1024), kIdescT,
                    k > 0 ? 1u : 0u);
        }
        tc_commit(&bars->s_full);
    };
    auto issue_dpt = [&]() {  // dP^T = V_j dO^T
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
            const uint32_t off = (k / 4) * kHalfTileBytes + (k % 4) * 32;
            umma_ss(t_dp, umma_smem_desc_sw128(sV + off, 16, 1024), umma_smem_desc_sw128(sdO + off, 16, 1024), kIdescT,
                    k > 0 ? 1u : 0u);
        }
        tc_commit(&bars->dp_full);
    };

    bool ok = mbar_wait(&bars->kv_full, 0, abort_flag);
    if (ok) ok = mbar_wait(&bars->q_full[0], 0, abort_flag);
    if (ok) ok = mbar_wait(&bars->do_full, 0, abort_flag);
    if (ok) {
        tc_fence_after();
        issue_st(0);
        issue_dpt();
    }
    const uint32_t t_p = tmem_base + Cfg::kColP;
    for (int it = 0; it < n_it && ok; ++it) {
        const int st = it & 1;
        const uint32_t sQ = smem_u32(smem + Cfg::kOffQ + st * Cfg::kTileBytes);
        ok = mbar_wait(&bars->p_ready, it & 1, abort_flag);
        if (!ok) break;
        TRACE(0, it * 8 + 0);
        tc_fence_after();
        if (Cfg::kSeparateP && it + 1 < n_it) {  // S^T columns are free as soon as the compute warps have read them
            ok = mbar_wait(&bars->q_full[st ^ 1], ((it + 1) >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            issue_st(it + 1);
        }
        // dV += P^T dO_i: 16 queries (8 packed TMEM columns, 16 smem rows) per instruction.
#pragma unroll
        for (int k = 0; k < kBlockQ / 16; ++k)
            umma_ts(t_dv, t_p + (k / 4) * Cfg::kPHalfStride + (k % 4) * 8,
                    umma_smem_desc_sw128(sdO + k * 2048, kHalfTileBytes, 1024), kIdescKV, (it > 0 || k > 0) ? 1u : 0u);
        tc_commit(&bars->do_empty);
        if (!Cfg::kSeparateP && it + 1 < n_it) {  // P^T lives in the S^T columns: dV must be queued first
            ok = mbar_wait(&bars->q_full[st ^ 1], ((it + 1) >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            issue_st(it + 1);
        }
        TRACE(0, it * 8 + 1);
        ok = mbar_wait(&bars->ds_ready, it & 1, abort_flag);
        if (!ok) break;
        TRACE(0, it * 8 + 2);
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < kBlockQ / 16; ++k)
            umma_ts(t_dk, t_dp + (k / 4) * 64 + (k % 4) * 8, umma_smem_desc_sw128(sQ + k * 2048, kHalfTileBytes, 1024),
                    kIdescKV, (it > 0 || k > 0) ? 1u : 0u);
        tc_commit(&bars->q_empty[st]);
        // dQ_i = dS K_j, 64 head-dim columns per accumulator half; 16 keys per instruction.
        if (!Cfg::kdQAliased) {  // the dQ warps must have read the previous tile out of the dQ columns
            ok = mbar_wait(&bars->dq_free, (it & 1) ^ 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
        }
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h) {
            const uint32_t t_dq = tmem_base + Cfg::kColdQ + h * 64;
#pragma unroll
            for (int k = 0; k < kBlockK / 16; ++k)
                umma_ss(t_dq, umma_smem_desc_sw128(sdS + k * 2048, kHalfTileBytes, 1024),
                        umma_smem_desc_sw128(sK + h * kHalfTileBytes + k * 2048, kHalfTileBytes, 1024), kIdescdQ,
                        k > 0 ? 1u : 0u);
        }
        tc_commit(&bars->dq_full);
        TRACE(0, it * 8 + 4);
        if (it + 1 < n_it) {
            if (Cfg::kdQAliased) {  // dQ(it) sits in the dP^T region until the dQ warps have read it
                ok = mbar_wait(&bars->dq_free, it & 1, abort_flag);
                if (!ok) break;
            }
            ok = mbar_wait(&bars->do_full, (it + 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            issue_dpt();
        }
        TRACE(0, it * 8 + 5);
    }
    if (ok) {
        tc_commit(&bars->mma_done);
    } else {
        int none = 0;
        tc_commit(&bars->drain);
        (void)mbar_wait(&bars->drain, 0, &none);
    }
}

// Row loader: LSE*log2e and Delta of query tile i into the double-buffered row arrays.
__device__ __forceinline__ void bwd_rows(BwdBars* bars, float* row_buf, const float* __restrict__ LSE,
                                         const float* __restrict__ Delta, int T, size_t row_base, int i0, int n_it,
                                         int tid64) {
    volatile int* abort_flag = &bars->abort_flag;
    for (int it = 0; it < n_it; ++it) {
        const int b = it & 1;
        if (!mbar_wait(&bars->row_empty[b], ((it >> 1) & 1) ^ 1, abort_flag)) return;
        float* s_lse = row_buf + b * 256;
        float* s_dl = s_lse + 128;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
            const int rl = tid64 + 64 * x;
            const int q = (i0 + it) * kBlockQ + rl;
            // Rows past the end of the sequence get LSE = +inf so that their P is exactly 0.
            s_lse[rl] = (q < T) ? LSE[row_base + q] * kLog2e : INFINITY;
            s_dl[rl] = (q < T) ? Delta[row_base + q] : 0.f;
        }
        __syncwarp();
        if ((tid64 & 31) == 0) mbar_arrive(&bars->row_full[b]);
    }
}

// P phase for this thread's 64 queries: p = exp2(s*c - lse*log2e), packed to bf16 pairs.
// kMasked: the tile is the diagonal one and/or holds keys past the end of the sequence.
template <bool kMasked>
__device__ __forceinline__ void bwd_p_phase(const uint32_t (&sv)[64], const float4* s_lse4, float c, uint32_t (&pk)[32],
                                            bool key_valid, bool diag, int r, int q_base) {
#pragma unroll
    for (int g = 0; g < 16; ++g) {
        const float4 l4 = s_lse4[g];
        float p0 = ex2_approx(fmaf(__uint_as_float(sv[4 * g + 0]), c, -l4.x));
        float p1 = ex2_approx(fmaf(__uint_as_float(sv[4 * g + 1]), c, -l4.y));
        float p2 = ex2_approx(fmaf(__uint_as_float(sv[4 * g + 2]), c, -l4.z));
        float p3 = ex2_approx(fmaf(__uint_as_float(sv[4 * g + 3]), c, -l4.w));
        if (kMasked) {
            // keep (query q, key r) iff the key exists and, on the diagonal tile, key <= query
            const int q0 = q_base + 4 * g;
            if (!key_valid || (diag && r > q0 + 0)) p0 = 0.f;
            if (!key_valid || (diag && r > q0 + 1)) p1 = 0.f;
            if (!key_valid || (diag && r > q0 + 2)) p2 = 0.f;
            if (!key_valid || (diag && r > q0 + 3)) p3 = 0.f;
        }
        pk[2 * g + 0] = pack_bf16x2(p0, p1);
        pk[2 * g + 1] = pack_bf16x2(p2, p3);
    }
}

template <int D, bool kCausal>
__device__ __forceinline__ void bwd_compute(uint8_t* smem, BwdBars* bars, uint32_t tmem_base,
                                            __nv_bfloat16* __restrict__ dK, __nv_bfloat16* __restrict__ dV, int T,
                                            int kt, int bh, int i0, int n_it, float scale, int cwarp, int lane) {
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (cwarp & 3);
    const int half = cwarp >> 2;             // which 64 queries of the tile this thread covers
    const int r = lane_base + lane;          // local key row
    const int key = kt * kBlockK + r;
    const bool key_valid = key < T;
    const bool tile_keys_valid = (kt * kBlockK + kBlockK) <= T;
    const float c = scale * kLog2e;
    const uint32_t t_s = tmem_addr(tmem_base, lane_base, Cfg::kColS + 64 * half);
    const uint32_t t_dp = tmem_addr(tmem_base, lane_base, Cfg::kColdP + 64 * half);
    const uint32_t t_p = tmem_addr(tmem_base, lane_base, Cfg::kColP + Cfg::kPHalfStride * half);
    const float* row_buf = reinterpret_cast<const float*>(smem + Cfg::kOffRow);
    uint8_t* sdS_row = smem + Cfg::kOffdS + half * kHalfTileBytes + r * 128;
    bool ok = true;

    for (int it = 0; it < n_it; ++it) {
        const int i = i0 + it;
        const int b = it & 1;
        const float4* s_lse4 = reinterpret_cast<const float4*>(row_buf + b * 256 + 64 * half);
        const float4* s_dl4 = reinterpret_cast<const float4*>(row_buf + b * 256 + 128 + 64 * half);
        ok = mbar_wait(&bars->row_full[b], (it >> 1) & 1, abort_flag);
        if (!ok) break;
        if (lane == 0 && (cwarp & 3) == 0) TRACE(1 + half, it * 8 + 0);
        ok = mbar_wait(&bars->s_full, it & 1, abort_flag);
        if (!ok) break;
        if (lane == 0 && (cwarp & 3) == 0) TRACE(1 + half, it * 8 + 1);
        tc_fence_after();

        // ---- P phase
        uint32_t pk[32];
        {
            uint32_t sv[64];
            tmem_ld_x32(t_s, sv);
            tmem_ld_x32(t_s + 32, sv + 32);
            tmem_wait_ld();
            const bool diag = kCausal && (i == kt);
            if (diag || !tile_keys_valid)
                bwd_p_phase<true>(sv, s_lse4, c, pk, key_valid, diag, r, 64 * half);
            else
                bwd_p_phase<false>(sv, s_lse4, c, pk, true, false, r, 64 * half);
        }
        if (Cfg::kSeparateP && it > 0) {  // dV of the previous tile must be done reading the P^T columns
            ok = mbar_wait(&bars->do_empty, (it - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
        }
        tmem_st_x32(t_p, pk);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0 && (cwarp & 3) == 0) TRACE(1 + half, it * 8 + 2);
        if (lane == 0) mbar_arrive(&bars->p_ready);

        // ---- dS phase: ds = p * (dp - delta); bf16 to TMEM (for dK) and to swizzled smem (for dQ)
        ok = mbar_wait(&bars->dp_full, it & 1, abort_flag);
        if (!ok) break;
        if (it > 0) {  // the dQ UMMA of the previous tile must be done reading the dS staging buffer
            ok = mbar_wait(&bars->dq_full, (it - 1) & 1, abort_flag);
            if (!ok) break;
        }
        if (lane == 0 && (cwarp & 3) == 0) TRACE(1 + half, it * 8 + 4);
        tc_fence_after();
        uint32_t dd[32];
        {
            uint32_t dv[64];
            tmem_ld_x32(t_dp, dv);
            tmem_ld_x32(t_dp + 32, dv + 32);
            tmem_wait_ld();
#pragma unroll
            for (int g = 0; g < 16; ++g) {
                const float4 d4 = s_dl4[g];
                const uint32_t pa = pk[2 * g], pb2 = pk[2 * g + 1];
                const float p0 = __uint_as_float(pa << 16), p1 = __uint_as_float(pa & 0xffff0000u);
                const float p2 = __uint_as_float(pb2 << 16), p3 = __uint_as_float(pb2 & 0xffff0000u);
                const float d0 = p0 * (__uint_as_float(dv[4 * g + 0]) - d4.x);
                const float d1 = p1 * (__uint_as_float(dv[4 * g + 1]) - d4.y);
                const float d2 = p2 * (__uint_as_float(dv[4 * g + 2]) - d4.z);
                const float d3 = p3 * (__uint_as_float(dv[4 * g + 3]) - d4.w);
                dd[2 * g + 0] = pack_bf16x2(d0, d1);
                dd[2 * g + 1] = pack_bf16x2(d2, d3);
            }
        }
        tmem_st_x32(t_dp, dd);
        // dS^T row r, this half's 64 queries: eight 16-byte chunks of one 128-byte swizzled row.
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
            *reinterpret_cast<uint4*>(sdS_row + ((ch ^ (r & 7)) << 4)) =
                make_uint4(dd[ch * 4 + 0], dd[ch * 4 + 1], dd[ch * 4 + 2], dd[ch * 4 + 3]);
        tmem_wait_st();
        fence_proxy_async_smem();
        tc_fence_before();
        __syncwarp();
        if (lane == 0 && (cwarp & 3) == 0) TRACE(1 + half, it * 8 + 6);
        if (lane == 0) {
            mbar_arrive(&bars->ds_ready);
            mbar_arrive(&bars->row_empty[b]);
        }
        if (lane == 0 && (cwarp & 3) == 0) TRACE(1 + half, it * 8 + 7);
    }
    if (ok) ok = mbar_wait(&bars->mma_done, 0, abort_flag);
    if (!ok) return;
    tc_fence_after();
    // dV and dK of this key row: this thread converts D/2 columns of each.
    constexpr int kColsPerThread = D / 2;
    const uint32_t t_dv = tmem_addr(tmem_base, lane_base, Cfg::kColdV + half * kColsPerThread);
    const uint32_t t_dk = tmem_addr(tmem_base, lane_base, Cfg::kColdK + half * kColsPerThread);
    const size_t out_off = (static_cast<size_t>(bh) * T + key) * D + half * kColsPerThread;
    uint4* dv_row = reinterpret_cast<uint4*>(dV + out_off);
    uint4* dk_row = reinterpret_cast<uint4*>(dK + out_off);
#pragma unroll
    for (int cb = 0; cb < kColsPerThread; cb += 32) {
        uint32_t a[32], bq[32];
        tmem_ld_x32(t_dv + cb, a);
        tmem_ld_x32(t_dk + cb, bq);
        tmem_wait_ld();
        if (key_valid) {
#pragma unroll
            for (int x = 0; x < 32; x += 8) {
                uint4 v, w;
                v.x = pack_bf16x2(__uint_as_float(a[x + 0]), __uint_as_float(a[x + 1]));
                v.y = pack_bf16x2(__uint_as_float(a[x + 2]), __uint_as_float(a[x + 3]));
                v.z = pack_bf16x2(__uint_as_float(a[x + 4]), __uint_as_float(a[x + 5]));
                v.w = pack_bf16x2(__uint_as_float(a[x + 6]), __uint_as_float(a[x + 7]));
                w.x = pack_bf16x2(__uint_as_float(bq[x + 0]) * scale, __uint_as_float(bq[x + 1]) * scale);
                w.y = pack_bf16x2(__uint_as_float(bq[x + 2]) * scale, __uint_as_float(bq[x + 3]) * scale);
                w.z = pack_bf16x2(__uint_as_float(bq[x + 4]) * scale, __uint_as_float(bq[x + 5]) * scale);
                w.w = pack_bf16x2(__uint_as_float(bq[x + 6]) * scale, __uint_as_float(bq[x + 7]) * scale);
                dv_row[(cb + x) / 8] = v;
                dk_row[(cb + x) / 8] = w;
            }
        }
    }
}

// dQ warps at D=64.  One thread per query row moves the partial dQ tile from TMEM into a swizzled
// shared-memory staging buffer (double-buffered); a leader thread sends it to the fp32 accumulator
// with two TMA reduce-add operations.  Nothing waits for a reduction to complete except the reuse
// of its staging buffer and the end of the kernel.
__device__ __forceinline__ void bwd_dq_tma(uint8_t* smem, BwdBars* bars, uint32_t tmem_base,
                                           const CUtensorMap* tmAcc, int bh, int i0, int n_it, int qwarp, int lane) {
    constexpr int D = 64;
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (qwarp & 3);
    const int r = lane_base + lane;  // local query row
    const bool leader = (qwarp == 0 && lane == 0);
    const uint32_t t_dq = tmem_addr(tmem_base, lane_base, Cfg::kColdQ);
    bool ok = true;
    for (int it = 0; it < n_it; ++it) {
        const int i = i0 + it;
        if (lane == 0 && qwarp == 0) TRACE(3, it * 8 + 0);
        ok = mbar_wait(&bars->dq_full, it & 1, abort_flag);
        if (!ok) break;
        if (lane == 0 && qwarp == 0) TRACE(3, it * 8 + 1);
        tc_fence_after();
        uint32_t a[64];
        tmem_ld_x32(t_dq, a);
        tmem_ld_x32(t_dq + 32, a + 32);
        tmem_wait_ld();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->dq_free);
        if (it >= 2) {  // the reduction that last used this staging buffer has finished reading it
            ok = mbar_wait(&bars->stage_free, it & 1, abort_flag);
            if (!ok) break;
        }
        uint8_t* stage = smem + Cfg::kOffStage + (it & 1) * Cfg::kStageBytes;
#pragma unroll
        for (int box = 0; box < 2; ++box) {
            uint8_t* row_ptr = stage + box * kHalfTileBytes + r * 128;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch)
                *reinterpret_cast<uint4*>(row_ptr + ((ch ^ (r & 7)) << 4)) =
                    make_uint4(a[box * 32 + ch * 4], a[box * 32 + ch * 4 + 1], a[box * 32 + ch * 4 + 2],
                               a[box * 32 + ch * 4 + 3]);
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->stage_full);
        bool leader_ok = true;
        if (leader) {
            leader_ok = mbar_wait(&bars->stage_full, it & 1, abort_flag);
            if (leader_ok) {
                tma_reduce_add_3d(tmAcc, stage, 0, i * kBlockQ, bh);
                tma_reduce_add_3d(tmAcc, stage + kHalfTileBytes, 32, i * kBlockQ, bh);
                bulk_commit_group();
                if (it > 0) {
                    bulk_wait_group_read<1>();  // the previous tile's staging buffer has been read
                    mbar_arrive(&bars->stage_free);
                }
            }
        }
        // Brings the leader back together with the rest of its warp before the next warp-wide TMEM
        // load, and makes a failed wait of the leader a failure of the whole warp.
        ok = __all_sync(0xffffffffu, leader_ok);
        if (!ok) break;
        if (lane == 0 && qwarp == 0) TRACE(3, it * 8 + 2);
    }
    // Also when giving up: nothing of this thread may stay in flight, and the accumulator must be
    // complete before the kernel ends.
    if (leader) bulk_wait_group<0>();
}

// dQ warps at D=128: one thread per query row adds its partial row with red.global.add.v4.f32.
__device__ __forceinline__ void bwd_dq_red(BwdBars* bars, uint32_t tmem_base, float* __restrict__ dq_acc, int T, int bh,
                                           int i0, int n_it, int qwarp, int lane) {
    constexpr int D = 128;
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (qwarp & 3);
    const int r = lane_base + lane;
    const size_t row_base = static_cast<size_t>(bh) * T;
    for (int it = 0; it < n_it; ++it) {
        const int i = i0 + it;
        if (!mbar_wait(&bars->dq_full, it & 1, abort_flag)) return;
        tc_fence_after();
        const int q = i * kBlockQ + r;
        float* dst = dq_acc + (row_base + q) * D;
#pragma unroll
        for (int cb = 0; cb < D; cb += 32) {
            uint32_t a[32];
            tmem_ld_x32(tmem_addr(tmem_base, lane_base, Cfg::kColdQ + cb), a);
            tmem_wait_ld();
            if (q < T) {
#pragma unroll
                for (int x = 0; x < 32; x += 4)
                    red_add_v4_f32(dst + cb + x, __uint_as_float(a[x]), __uint_as_float(a[x + 1]),
                                   __uint_as_float(a[x + 2]), __uint_as_float(a[x + 3]));
            }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->dq_free);
    }
}

template <int D, bool kCausal>
__global__ void __launch_bounds__(kBwdThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                const __grid_constant__ CUtensorMap tmAcc, const float* __restrict__ LSE,
                const float* __restrict__ Delta, float* __restrict__ dq_acc, __nv_bfloat16* __restrict__ dK,
                __nv_bfloat16* __restrict__ dV, int T, int BH, int n_tiles, float scale,
                int* __restrict__ dev_status) {
    using Cfg = BwdCfg<D>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    BwdBars* bars = reinterpret_cast<BwdBars*>(smem + Cfg::kOffBar);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#ifdef NOVA_EXP_TRACE
    long long blk_t0 = 0;
    if (threadIdx.x == 0) { asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(blk_t0)); }
#endif
    // Key tile 0 sees every query tile under the causal clamp, so low key tiles go first.
    const int kt = static_cast<int>(blockIdx.x) / BH;
    const int bh = static_cast<int>(blockIdx.x) % BH;
    const int i0 = kCausal ? kt : 0;  // raised lower bound of the query loop
    const int n_it = n_tiles - i0;

    if (threadIdx.x == 0) {
        mbar_init(&bars->kv_full, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->q_full[s], 1);
            mbar_init(&bars->q_empty[s], 1);
            mbar_init(&bars->row_full[s], 2);
            mbar_init(&bars->row_empty[s], kComputeThreads / 32);
        }
        mbar_init(&bars->do_full, 1);
        mbar_init(&bars->do_empty, 1);
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->dp_full, 1);
        mbar_init(&bars->p_ready, kComputeThreads / 32);
        mbar_init(&bars->ds_ready, kComputeThreads / 32);
        mbar_init(&bars->dq_full, 1);
        mbar_init(&bars->dq_free, 4);
        mbar_init(&bars->stage_full, 4);
        mbar_init(&bars->stage_free, 1);
        mbar_init(&bars->mma_done, 1);
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        tma_prefetch_desc(&tmAcc);
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
    const size_t row_base = static_cast<size_t>(bh) * T;
#ifdef NOVA_EXP_TRACE

#endif

    if (warp == 0) {
        if (lane == 0) bwd_producer<D>(&tmQ, &tmK, &tmV, &tmdO, smem, bars, kt, bh, i0, n_it);
    } else if (warp == 1) {
        if (lane == 0) bwd_mma<D>(smem, bars, tmem_base, n_it);
    } else if (warp < 4) {
        bwd_rows(bars, reinterpret_cast<float*>(smem + Cfg::kOffRow), LSE, Delta, T, row_base, i0, n_it,
                 (warp - 2) * 32 + lane);
    } else if (warp < 12) {
        bwd_compute<D, kCausal>(smem, bars, tmem_base, dK, dV, T, kt, bh, i0, n_it, scale, warp - 4, lane);
    } else {
        if constexpr (Cfg::kBulkdQ)
            bwd_dq_tma(smem, bars, tmem_base, &tmAcc, bh, i0, n_it, warp - 12, lane);
        else
            bwd_dq_red(bars, tmem_base, dq_acc, T, bh, i0, n_it, warp - 12, lane);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kBwdTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
#ifdef NOVA_EXP_TRACE
    if (threadIdx.x == 0 && blockIdx.x < 4096) {
        long long t1; unsigned smid;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t1));
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        g_blk[blockIdx.x * 4 + 0] = blk_t0; g_blk[blockIdx.x * 4 + 1] = t1; g_blk[blockIdx.x * 4 + 2] = smid; g_blk[blockIdx.x * 4 + 3] = n_it;
    }
#endif
}

template <int D, bool kCausal>
cudaError_t launch_one(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       const CUtensorMap& tmdO, const CUtensorMap& tmAcc, const float* LSE, const float* Delta,
                       float* dq_acc, __nv_bfloat16* dK, __nv_bfloat16* dV, const AttnShape& s, int* dev_status,
                       cudaStream_t stream) {
    const int n_tiles = (s.T + kBlockK - 1) / kBlockK;
    const int BH = s.B * s.H;
    const dim3 grid(static_cast<unsigned>(n_tiles) * BH);
    attn_bwd_kernel<D, kCausal><<<grid, kBwdThreads, BwdCfg<D>::kSmemBytes, stream>>>(
        tmQ, tmK, tmV, tmdO, tmAcc, LSE, Delta, dq_acc, dK, dV, s.T, BH, n_tiles, s.scale, dev_status);
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
                            const CUtensorMap& tmdO, const CUtensorMap& tmAcc, const float* LSE, const float* Delta,
                            float* dq_acc, __nv_bfloat16* dK, __nv_bfloat16* dV, const AttnShape& s, int* dev_status,
                            cudaStream_t stream) {
    if (s.D == 64) {
        return s.causal ? launch_one<64, true>(tmQ, tmK, tmV, tmdO, tmAcc, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream)
                        : launch_one<64, false>(tmQ, tmK, tmV, tmdO, tmAcc, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream);
    }
    return s.causal ? launch_one<128, true>(tmQ, tmK, tmV, tmdO, tmAcc, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream)
                    : launch_one<128, false>(tmQ, tmK, tmV, tmdO, tmAcc, LSE, Delta, dq_acc, dK, dV, s, dev_status, stream);
}

}  // namespace nova
