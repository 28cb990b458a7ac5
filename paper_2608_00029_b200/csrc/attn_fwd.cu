// Fused causal attention forward for sm_100a (paper Section 4.2: score contraction, index mask,
// base-2 online softmax, value contraction, causal loop clamp, 1/sum epilogue, LSE saved).
//
// A work item is a block of 256 query rows of one (batch, head): two 128-row query tiles, A and B,
// that share every K/V tile they both need.  The kernel is persistent and its work is handed out
// dynamically: the grid has one CTA per item, heaviest first (the last query block of a causal problem
// sees every key tile); one CTA per SM starts, and each, while it works on an item, asks the hardware to
// cancel the launch of the next CTA that has not started and takes over its item (cluster launch control),
// so no SM idles while items are left.  The producer warp makes the request and passes the item number to
// the other roles through a two-entry ring in shared memory.  Roles (384 threads):
//   warp 0       TMA producer: Q tiles per item, K and V tiles through mbarrier-guarded rings
//   warp 1       UMMA issuer:  S_t = Q_t K^T  (operands in shared memory, accumulator in TMEM)
//                              O_t += P_t V   (P read from TMEM as bf16, V from shared memory)
//                interleaved over the two tiles: while the softmax warps of tile A work on key tile
//                j+1 the tensor core runs P V and the next Q K^T of tile B, and vice versa
//   warps 4-7    softmax of tile A, warps 8-11 softmax of tile B: one thread per query row reads its
//                S row from TMEM, keeps the running max / sum in registers, writes bf16 P back over
//                S, rescales O in TMEM only when the row maximum has grown by more than 2^8 (exact:
//                the final 1/sum and the LSE use the same reference maximum), and at the end of the
//                item normalises O, stages it in the (now idle) Q tile buffer and sends it out with
//                TMA stores.
// TMEM columns: S_A [0,128)  S_B [128,256)  O_A [256,256+D)  O_B [256+D,256+2D).  P_t (bf16 pairs,
// 64 columns) has columns of its own at D = 64, [384,448) and [448,512): the softmax warps release
// S_t as soon as they have loaded it, so the next Q_t K^T runs while they compute.  At D = 128 all
// 512 columns are taken and P_t lies over the first 64 columns of S_t.
//
// Warp-wide .sync.aligned instructions (TMEM loads/stores) need the whole warp together: wherever
// one lane does extra work (the store leader), the warp is rejoined with a vote before the next one.
#include "kernels.h"
#include "ptx.cuh"

namespace nova {
namespace {

constexpr int kFwdThreads = 384;
constexpr int kFwdTmemCols = 512;
constexpr float kRescaleThreshold = 8.0f;  // log2 units
constexpr int kBlockRows = 2 * kBlockQ;    // query rows per work item

template <int D>
struct FwdCfg {
    static constexpr int kHalves = D / kBoxCols;
    static constexpr int kTileBytes = kHalves * kHalfTileBytes;
    static constexpr int kQStages = (D == 64) ? 2 : 1;
    static constexpr int kKVStages = 2;
    static constexpr int kOffQ = 0;                                    // [kQStages][2 tiles]
    static constexpr int kOffK = kQStages * 2 * kTileBytes;            // [kKVStages]
    static constexpr int kOffV = kOffK + kKVStages * kTileBytes;       // [kKVStages]
    static constexpr int kOffBar = kOffV + kKVStages * kTileBytes;
    static constexpr int kSmemBytes = kOffBar + 512 + 1024;
    static constexpr int kColS = 0;      // + 128 * tile
    static constexpr int kColO = 256;    // + D * tile
    // With D = 64 there is room for P in columns of its own, so that S_t can be overwritten by the
    // next Q K^T as soon as the softmax warps have read it; with D = 128 P lies over S.
    static constexpr bool kSepP = (D == 64);
    static constexpr int kColP = kSepP ? 384 : 0;  // + 64 * tile (kSepP) / + 128 * tile
    static constexpr int kStrideP = kSepP ? 64 : 128;
};

struct FwdBars {
    uint64_t q_full[2], q_empty[2];
    uint64_t k_full[2], k_empty[2], v_full[2], v_empty[2];
    uint64_t s_full[2], s_free[2], p_ready[2], pv_done[2], o_free[2], o_staged[2];  // per query tile
    uint64_t drain;
    WorkRing ring;  // item numbers: producer -> UMMA issuer and softmax warps
    uint32_t tmem_base;
    int abort_flag;
};
constexpr int kWorkConsumers = 1 + 8;  // UMMA issuer warp + 8 softmax warps

// Work items: 256-row query blocks, numbered heaviest first.
struct FwdWork {
    int n_items, BH, n_blocks, n_kv_all, T, H;
    uint32_t orders;  // coordinate orders of the Q, K, V, O tensor maps, four bits each
    bool causal;
    // Item `idx`: block index, head, and the number of key tiles each query tile visits
    // (0 if the tile lies entirely past the end of the sequence).
    __device__ __forceinline__ void get(int idx, int* blk, int* bh, int* n_a, int* n_b) const {
        *blk = n_blocks - 1 - idx / BH;
        *bh = idx % BH;
        const int qt_a = 2 * (*blk), qt_b = qt_a + 1;
        // causal clamp of the key loop: tile qt visits key tiles 0..qt
        *n_a = causal ? min(qt_a + 1, n_kv_all) : n_kv_all;
        *n_b = (qt_b * kBlockQ < T) ? (causal ? min(qt_b + 1, n_kv_all) : n_kv_all) : 0;
    }
};

template <int D, bool kStrided>
__device__ __forceinline__ void fwd_producer(const CUtensorMap* tmQ, const CUtensorMap* tmK,
                                             const CUtensorMap* tmV, uint8_t* smem, FwdBars* bars,
                                             const FwdWork& wk, long long limit, int inject) {
    using Cfg = FwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    int armed_q[2] = {-1, -1}, armed_k[2] = {-1, -1}, armed_v[2] = {-1, -1};
    bool ok = true;
    int w = 0, g = 0;  // items and key tiles loaded so far
    int item = blockIdx.x;
    bool clc_pending = false;
    for (;;) {
        // hand the item (or the end mark) to the other roles
        ok = bars->ring.publish(w, item, abort_flag, limit);
        if (!ok || item < 0) break;
        int blk, bh, n_a, n_b;
        wk.get(item, &blk, &bh, &n_a, &n_b);
        const int head = kStrided ? bh % wk.H : 0, batch = kStrided ? bh / wk.H : 0;
        const int qs = w % Cfg::kQStages;
        const uint32_t qph = (w / Cfg::kQStages) & 1;
        ok = mbar_wait(&bars->q_empty[qs], qph ^ 1, abort_flag, limit);
        if (!ok) break;
        mbar_expect_tx(&bars->q_full[qs], 2 * Cfg::kTileBytes);  // rows past T arrive as zeros
        armed_q[qs] = qph;
#pragma unroll
        for (int t = 0; t < 2; ++t)
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h)
                tma_load_tile<kStrided>(smem + Cfg::kOffQ + (qs * 2 + t) * Cfg::kTileBytes + h * kHalfTileBytes, tmQ,
                              &bars->q_full[qs], wk.orders & 15, h * kBoxCols, blk * kBlockRows + t * kBlockQ, head, batch, bh);
        const int n = max(n_a, n_b);
        for (int j = 0; j < n; ++j, ++g) {
            const int st = g & 1;
            const uint32_t ph = (g >> 1) & 1;
            ok = mbar_wait(&bars->k_empty[st], ph ^ 1, abort_flag, limit);
            if (!ok) break;
            // `inject` (a test aid, 0 in normal use): the very first K tile is never requested, so the wait for
            // it runs out and the kernel leaves through its time-out path
            if (!(inject == 1 && g == 0)) {
                mbar_expect_tx(&bars->k_full[st], Cfg::kTileBytes);
                armed_k[st] = ph;
#pragma unroll
                for (int h = 0; h < Cfg::kHalves; ++h)
                    tma_load_tile<kStrided>(smem + Cfg::kOffK + st * Cfg::kTileBytes + h * kHalfTileBytes, tmK,
                                            &bars->k_full[st], (wk.orders >> 4) & 15, h * kBoxCols, j * kBlockK, head,
                                            batch, bh);
            }
            ok = mbar_wait(&bars->v_empty[st], ph ^ 1, abort_flag, limit);
            if (!ok) break;
            mbar_expect_tx(&bars->v_full[st], Cfg::kTileBytes);
            armed_v[st] = ph;
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h)
                tma_load_tile<kStrided>(smem + Cfg::kOffV + st * Cfg::kTileBytes + h * kHalfTileBytes, tmV, &bars->v_full[st],
                              (wk.orders >> 8) & 15, h * kBoxCols, j * kBlockK, head, batch, bh);
        }
        if (!ok) break;
        // All loads of this item are on their way (the other roles are about two key tiles behind): only now
        // ask for the next item, so that an item is claimed as late as possible and the CTAs that finish early
        // find the remaining ones.
        bars->ring.request();
        clc_pending = true;
        ok = bars->ring.answer(w, &item, abort_flag, limit);
        if (!ok) break;
        clc_pending = false;
        ++w;
    }
    if (!ok) {
        // Giving up: let the copies already in flight land before the CTA's shared memory goes away.
        int none = 0;
        if (clc_pending) (void)mbar_wait(&bars->ring.answer_bar, w & 1, &none);  // the answer must land before the CTA ends
        for (int s = 0; s < 2; ++s) {
            if (armed_q[s] >= 0) (void)mbar_wait(&bars->q_full[s], armed_q[s], &none);
            if (armed_k[s] >= 0) (void)mbar_wait(&bars->k_full[s], armed_k[s], &none);
            if (armed_v[s] >= 0) (void)mbar_wait(&bars->v_full[s], armed_v[s], &none);
        }
    }
}

template <int D>
__device__ __forceinline__ void fwd_mma(uint8_t* smem, FwdBars* bars, uint32_t tmem_base, const FwdWork& wk,
                                        long long limit) {
    using Cfg = FwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    constexpr uint32_t kIdescQK = umma_idesc_bf16(128, 128, 0, 0);
    constexpr uint32_t kIdescPV = umma_idesc_bf16(128, D, 0, 1);
    const uint32_t hi = umma_desc_hi_sw128(1024);
    // Descriptor lower words per buffer; in the loops only a constant (byte offset >> 4) is added.
    uint32_t k_k[2], v_m[2];
#pragma unroll
    for (int st = 0; st < 2; ++st) {
        k_k[st] = umma_desc_lo(smem_u32(smem + Cfg::kOffK + st * Cfg::kTileBytes), 16);
        v_m[st] = umma_desc_lo(smem_u32(smem + Cfg::kOffV + st * Cfg::kTileBytes), kHalfTileBytes);
    }
    uint32_t q_k[2] = {0, 0};  // per item: the two query tiles
    // The whole warp runs this role in uniform control flow; one elected lane issues.
    const bool el = elect_one();
    const int lane = threadIdx.x & 31;
    bool ok = true;
    int w = 0, g = 0;
    int c[2] = {0, 0};   // key tiles processed so far per query tile (phases of its barriers)
    int cq[2] = {0, 0};  // Q K^T issued so far per query tile (phases of s_free)
    int wt[2] = {0, 0};  // items in which the query tile took part so far (phases of o_free)

    // S_t = Q_t K^T for the key tile in stage gk & 1: both operands K-major, 16 head-dim elements
    // (32 bytes) per instruction.
    auto issue_qk = [&](int t, int gk, uint32_t q_desc) {
        const uint32_t t_s = tmem_base + Cfg::kColS + 128 * t;
        const uint32_t b = k_k[gk & 1];
        if (Cfg::kSepP && cq[t] > 0) {  // the softmax warps must have read the previous S_t
            ok = mbar_wait(&bars->s_free[t], (cq[t] - 1) & 1, abort_flag, limit);
            if (!ok) return;
            tc_fence_after();
        }
        ++cq[t];
        if (el) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = ((k / 4) * kHalfTileBytes + (k % 4) * 32) >> 4;
                umma_ss(t_s, umma_desc_join(q_desc + off, hi), umma_desc_join(b + off, hi), kIdescQK,
                        k > 0 ? 1u : 0u);
            }
            tc_commit(&bars->s_full[t]);
        }
        __syncwarp();
    };

    constexpr int kNotPeeked = -3;
    int peeked = kNotPeeked;  // the next item's number, if it was looked at from inside the current item
    bool first_queued = false;  // ... and its first Q K^T products were queued from there
    for (;;) {
        const int item = (peeked != kNotPeeked) ? peeked : bars->ring.take(w, lane, abort_flag, limit);
        peeked = kNotPeeked;
        if (item < 0) {
            ok = (item == -1);
            break;
        }
        int blk, bh, n_a, n_b;
        wk.get(item, &blk, &bh, &n_a, &n_b);
        const int n_t[2] = {n_a, n_b};
        const int n = max(n_a, n_b);
        const int qs = w % Cfg::kQStages;
#pragma unroll
        for (int t = 0; t < 2; ++t)
            q_k[t] = umma_desc_lo(smem_u32(smem + Cfg::kOffQ + (qs * 2 + t) * Cfg::kTileBytes), 16);
        if (!first_queued) {
            ok = mbar_wait(&bars->q_full[qs], (w / Cfg::kQStages) & 1, abort_flag, limit);
            if (ok) ok = mbar_wait(&bars->k_full[g & 1], (g >> 1) & 1, abort_flag, limit);
            if (!ok) break;
            tc_fence_after();
            // P over S: the S columns of both tiles are free, their last P was consumed by a P V queued
            // earlier.  P apart: issue_qk waits until the previous S_t has been read.
            if (n_a > 0) issue_qk(0, g, q_k[0]);
            if (n_b > 0 && ok) issue_qk(1, g, q_k[1]);
            if (!ok) break;
            if (el) tc_commit(&bars->k_empty[g & 1]);  // K tile 0 is no longer read once these have run
            __syncwarp();
        }
        first_queued = false;
        for (int j = 0; j < n && ok; ++j, ++g) {
            const int st = g & 1;
            bool next_k_ready = false;
            if (Cfg::kSepP && j + 1 < n) {
                // Both Q K^T of the next key tile go first: S_t was released right after the softmax
                // warps loaded it, long before their P is ready.
                ok = mbar_wait(&bars->k_full[st ^ 1], ((g + 1) >> 1) & 1, abort_flag, limit);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int t = 0; t < 2; ++t)
                    if (j + 1 < n_t[t] && ok) issue_qk(t, g + 1, q_k[t]);
                if (!ok) break;
            } else if (Cfg::kSepP && Cfg::kQStages > 1) {
                // Last key tile of the item: if the producer has already announced the next item and its Q
                // tiles and first K tile have landed, its first Q K^T products are queued now, exactly like
                // those of a next key tile, so that neither softmax warpgroup waits at the item boundary.
                const int wn = w + 1;
                if (bars->ring.published(wn)) {
                    peeked = bars->ring.take(wn, lane, abort_flag, limit);
                    if (peeked >= 0) {
                        const int qs2 = wn % Cfg::kQStages;
                        bool there = mbar_test(&bars->q_full[qs2], (wn / Cfg::kQStages) & 1) &&
                                mbar_test(&bars->k_full[st ^ 1], ((g + 1) >> 1) & 1);
                        if (__all_sync(0xffffffffu, there)) {
                            int blk2, bh2, n_a2, n_b2;
                            wk.get(peeked, &blk2, &bh2, &n_a2, &n_b2);
                            tc_fence_after();
                            if (n_a2 > 0)
                                issue_qk(0, g + 1, umma_desc_lo(smem_u32(smem + Cfg::kOffQ + (qs2 * 2 + 0) * Cfg::kTileBytes), 16));
                            if (n_b2 > 0 && ok)
                                issue_qk(1, g + 1, umma_desc_lo(smem_u32(smem + Cfg::kOffQ + (qs2 * 2 + 1) * Cfg::kTileBytes), 16));
                            if (!ok) break;
                            if (el) tc_commit(&bars->k_empty[st ^ 1]);
                            __syncwarp();
                            first_queued = true;
                        }
                    }
                }
            }
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                if (j >= n_t[t]) continue;
                const uint32_t t_s = tmem_base + Cfg::kColP + Cfg::kStrideP * t;
                const uint32_t t_o = tmem_base + Cfg::kColO + D * t;
                ok = mbar_wait(&bars->p_ready[t], c[t] & 1, abort_flag, limit);
                if (!ok) break;
                if (j == 0) {
                    ok = mbar_wait(&bars->v_full[st], (g >> 1) & 1, abort_flag, limit);
                    // the previous item's O_t must have been read out of TMEM before it is overwritten
                    if (ok && wt[t] > 0) ok = mbar_wait(&bars->o_free[t], (wt[t] - 1) & 1, abort_flag, limit);
                } else if (t == 0 || j >= n_t[0]) {
                    ok = mbar_wait(&bars->v_full[st], (g >> 1) & 1, abort_flag, limit);
                }
                if (!ok) break;
                tc_fence_after();
                // O_t += P_t V: P from TMEM (16 keys = 8 packed columns per instruction), V is MN-major
                // (rows = keys, 64 head-dim elements per 128-byte row, second 64-wide half at +16 KB).
                if (el) {
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k)
                        umma_ts(t_o, t_s + k * 8, umma_desc_join(v_m[st] + k * 128, hi), kIdescPV,
                                (j > 0 || k > 0) ? 1u : 0u);
                    tc_commit(&bars->pv_done[t]);
                }
                __syncwarp();
                ++c[t];
                if (!Cfg::kSepP && j + 1 < n_t[t]) {  // the S_t columns are free again once this P V has run
                    if (!next_k_ready) {
                        ok = mbar_wait(&bars->k_full[st ^ 1], ((g + 1) >> 1) & 1, abort_flag, limit);
                        if (!ok) break;
                        tc_fence_after();
                        next_k_ready = true;
                    }
                    issue_qk(t, g + 1, q_k[t]);
                }
            }
            if (!ok) break;
            if (el) {
                tc_commit(&bars->v_empty[st]);                    // V tile j is no longer read
                if (j + 1 < n) tc_commit(&bars->k_empty[st ^ 1]);  // nor K tile j+1 (both Q K^T are queued)
            }
            __syncwarp();
        }
        if (!ok) break;
        if (n_a > 0) ++wt[0];
        if (n_b > 0) ++wt[1];
        ++w;
    }
    if (!ok) {
        // Drain whatever was issued before leaving so TMEM can be released safely.
        int none = 0;
        if (el) tc_commit(&bars->drain);
        __syncwarp();
        (void)mbar_wait(&bars->drain, 0, &none);
    }
}

template <int D, bool kCausal, bool kStrided>
__device__ __forceinline__ void fwd_softmax(uint8_t* smem, FwdBars* bars, uint32_t tmem_base, const CUtensorMap* tmO,
                                            float* __restrict__ LSE, float scale, const FwdWork& wk, int t, int swarp,
                                            int lane, long long limit) {
    using Cfg = FwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (swarp & 3);
    const int row_local = lane_base + lane;
    const bool leader = (swarp == 0 && lane == 0);
    const uint32_t t_s = tmem_addr(tmem_base, lane_base, Cfg::kColS + 128 * t);
    const uint32_t t_o = tmem_addr(tmem_base, lane_base, Cfg::kColO + D * t);
    const uint32_t t_p = tmem_addr(tmem_base, lane_base, Cfg::kColP + Cfg::kStrideP * t);
    const float c = scale * kLog2e;
    const int T = wk.T;
    bool ok = true;
    int w = 0, wt = 0, cnt = 0;  // items, items this tile took part in, key tiles processed by this tile
    int pending_qs = -1;         // Q stage whose O store was issued at the end of the previous item

    for (;;) {
        const int item = bars->ring.take(w, lane, abort_flag, limit);
        if (item < 0) {
            ok = (item == -1);
            break;
        }
        int blk, bh, n_a, n_b;
        wk.get(item, &blk, &bh, &n_a, &n_b);
        const int n_kv = (t == 0) ? n_a : n_b;
        const int qt = 2 * blk + t;
        const int row = qt * kBlockQ + row_local;
        const int qs = w % Cfg::kQStages;
        uint8_t* stage = smem + Cfg::kOffQ + (qs * 2 + t) * Cfg::kTileBytes;  // this tile's Q buffer
        if (n_kv == 0) {
            // Tile entirely past the end of the sequence: only release the Q stage, and only once it
            // has been filled, so that this warpgroup never runs ahead of the ring.
            bool leader_ok = true;
            if (leader) {
                if (pending_qs >= 0) {
                    bulk_wait_group_read<0>();
                    mbar_arrive(&bars->q_empty[pending_qs]);
                }
                leader_ok = mbar_wait(&bars->q_full[qs], (w / Cfg::kQStages) & 1, abort_flag, limit);
                if (leader_ok) mbar_arrive(&bars->q_empty[qs]);
            }
            pending_qs = -1;
            ok = __all_sync(0xffffffffu, leader_ok);
            if (!ok) break;
            ++w;
            continue;
        }
        float m_ref = -INFINITY;  // reference maximum of the raw (unscaled) scores
        float l = 0.f;

        for (int j = 0; j < n_kv; ++j, ++cnt) {
            ok = mbar_wait(&bars->s_full[t], cnt & 1, abort_flag, limit);
            if (!ok) break;
            tc_fence_after();
            uint32_t sr[128];
            tmem_ld_x32(t_s + 0, sr + 0);
            tmem_ld_x32(t_s + 32, sr + 32);
            tmem_ld_x32(t_s + 64, sr + 64);
            tmem_ld_x32(t_s + 96, sr + 96);
            tmem_wait_ld();
            if (Cfg::kSepP) {  // S_t may be overwritten by the next Q K^T
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->s_free[t]);
            }

            // Mask from indices only: the diagonal tile keeps key <= query; a ragged last tile keeps key < T.
            const bool diag = kCausal && (j == qt);
            const int keys_left = T - j * kBlockK;
            if (diag || keys_left < kBlockK) {
                const int lim = diag ? min(row_local, keys_left - 1) : keys_left - 1;
#pragma unroll
                for (int i = 0; i < 128; ++i)
                    if (i > lim) sr[i] = 0xff800000u;  // -inf
            }
            float mx0 = fmaxf(__uint_as_float(sr[0]), __uint_as_float(sr[1]));
            float mx1 = fmaxf(__uint_as_float(sr[2]), __uint_as_float(sr[3]));
            float mx2 = fmaxf(__uint_as_float(sr[4]), __uint_as_float(sr[5]));
            float mx3 = fmaxf(__uint_as_float(sr[6]), __uint_as_float(sr[7]));
#pragma unroll
            for (int i = 8; i < 128; i += 8) {
                mx0 = fmax3(mx0, __uint_as_float(sr[i + 0]), __uint_as_float(sr[i + 1]));
                mx1 = fmax3(mx1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
                mx2 = fmax3(mx2, __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
                mx3 = fmax3(mx3, __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
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
                    ok = mbar_wait(&bars->pv_done[t], (cnt - 1) & 1, abort_flag, limit);
                    if (!ok) break;
                    tc_fence_after();
                    #pragma unroll 1
                    for (int cb = 0; cb < D; cb += 16) {
                        uint32_t o[16];
                        tmem_ld_x16(t_o + cb, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 16; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * f);
                        tmem_st_x16(t_o + cb, o);
                    }
                }
            }
            // p = 2^(s * c - m * c): the multiply-subtract and the row sum run on packed fp32 pairs.
            const uint64_t c2 = f32x2_pack(c, c);
            const uint64_t nmc2 = f32x2_pack(-m_ref * c, -m_ref * c);
            uint64_t acc0 = 0, acc1 = 0;  // two pairs of partial sums
            if (Cfg::kSepP && j > 0) {  // the previous P_t must have been consumed (long since, as a rule)
                ok = mbar_wait(&bars->pv_done[t], (cnt - 1) & 1, abort_flag, limit);
                if (!ok) break;
                tc_fence_after();
            }
#pragma unroll
            for (int cb = 0; cb < 128; cb += 64) {
                uint32_t pk[32];
#pragma unroll
                for (int i = 0; i < 64; i += 4) {
                    const uint64_t x01 = f32x2_fma(
                        f32x2_pack(__uint_as_float(sr[cb + i + 0]), __uint_as_float(sr[cb + i + 1])), c2, nmc2);
                    const uint64_t x23 = f32x2_fma(
                        f32x2_pack(__uint_as_float(sr[cb + i + 2]), __uint_as_float(sr[cb + i + 3])), c2, nmc2);
                    float x0, x1, x2, x3;
                    f32x2_unpack(x01, x0, x1);
                    f32x2_unpack(x23, x2, x3);
                    const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
                    acc0 = f32x2_add(acc0, f32x2_pack(p0, p1));
                    acc1 = f32x2_add(acc1, f32x2_pack(p2, p3));
                    pk[i / 2] = pack_bf16x2_int(p0, p1);
                    pk[i / 2 + 1] = pack_bf16x2_int(p2, p3);
                }
                tmem_st_x32(t_p + cb / 2, pk);
            }
            {
                float a0, a1, a2, a3;
                f32x2_unpack(acc0, a0, a1);
                f32x2_unpack(acc1, a2, a3);
                l += (a0 + a1) + (a2 + a3);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->p_ready[t]);
            if (pending_qs >= 0) {
                if (leader) {
                    bulk_wait_group_read<0>();
                    mbar_arrive(&bars->q_empty[pending_qs]);
                }
                pending_qs = -1;
                __syncwarp();
            }
        }
        if (!ok) break;

        // ---- end of the item: O_t / l as bf16 into this tile's Q buffer (no longer read: every
        // Q K^T of the tile completed before its last P V), then TMA stores; LSE straight to global.
        ok = mbar_wait(&bars->pv_done[t], (cnt - 1) & 1, abort_flag, limit);
        if (!ok) break;
        tc_fence_after();
        const float inv_l = 1.0f / l;
#pragma unroll
        for (int cb = 0; cb < D; cb += 32) {
            uint32_t o[32];
            tmem_ld_x32(t_o + cb, o);
            tmem_wait_ld();
            uint8_t* row_ptr = stage + (cb / 64) * kHalfTileBytes + row_local * 128;
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int ch = (cb % 64) / 8 + x;  // 16-byte chunk of the 128-byte swizzled row
                uint4 v;
                v.x = pack_bf16x2(__uint_as_float(o[8 * x + 0]) * inv_l, __uint_as_float(o[8 * x + 1]) * inv_l);
                v.y = pack_bf16x2(__uint_as_float(o[8 * x + 2]) * inv_l, __uint_as_float(o[8 * x + 3]) * inv_l);
                v.z = pack_bf16x2(__uint_as_float(o[8 * x + 4]) * inv_l, __uint_as_float(o[8 * x + 5]) * inv_l);
                v.w = pack_bf16x2(__uint_as_float(o[8 * x + 6]) * inv_l, __uint_as_float(o[8 * x + 7]) * inv_l);
                *reinterpret_cast<uint4*>(row_ptr + ((ch ^ (row_local & 7)) << 4)) = v;
            }
        }
        tc_fence_before();
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
            mbar_arrive(&bars->o_free[t]);    // O_t has been read out of TMEM
            mbar_arrive(&bars->o_staged[t]);  // and this warp's rows are staged
        }
        if (row < T) LSE[static_cast<size_t>(bh) * T + row] = m_ref * scale + logf(l);
        bool leader_ok = true;
        if (leader) {
            leader_ok = mbar_wait(&bars->o_staged[t], wt & 1, abort_flag, limit);
            if (leader_ok) {
#pragma unroll
                for (int h = 0; h < Cfg::kHalves; ++h)
                    tma_store_tile<kStrided>(tmO, stage + h * kHalfTileBytes, (wk.orders >> 12) & 15, h * kBoxCols,
                                             qt * kBlockQ, kStrided ? bh % wk.H : 0, kStrided ? bh / wk.H : 0, bh);
                bulk_commit_group();
                if (Cfg::kQStages == 1) {  // the next item's Q tile needs this very buffer
                    bulk_wait_group_read<0>();
                    mbar_arrive(&bars->q_empty[qs]);
                }
            }
        }
        // With two Q stages the buffer is only needed for the item after next: it is handed back after the next
        // item's first key tile, when the store has long read it, instead of holding this warp up now (worth 7 %
        // at B=8, H=12, T=1024; a separate store thread that waits in the softmax warps' stead was slower).
        if (Cfg::kQStages > 1) pending_qs = qs;
        // Brings the leader back together with the rest of its warp before the next warp-wide TMEM
        // load, and makes a failed wait of the leader a failure of the whole warp.
        ok = __all_sync(0xffffffffu, leader_ok);
        if (!ok) break;
        ++w;
        ++wt;
    }
    if (leader) bulk_wait_group<0>();  // O must be complete before the kernel ends
}

template <int D, bool kCausal, bool kStrided>
__global__ void __launch_bounds__(kFwdThreads, 1)
attn_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                float* __restrict__ LSE, int T, int BH, int H, uint32_t orders, int n_blocks, float scale,
                long long limit, int inject, int* __restrict__ dev_status) {
    using Cfg = FwdCfg<D>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    FwdBars* bars = reinterpret_cast<FwdBars*>(smem + Cfg::kOffBar);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const FwdWork wk{n_blocks * BH, BH, n_blocks, (T + kBlockK - 1) / kBlockK, T, H, orders, kCausal};

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->q_full[s], 1);
            mbar_init(&bars->q_empty[s], 2);  // the store leaders of the two query tiles
            mbar_init(&bars->k_full[s], 1);
            mbar_init(&bars->k_empty[s], 1);
            mbar_init(&bars->v_full[s], 1);
            mbar_init(&bars->v_empty[s], 1);
            mbar_init(&bars->s_full[s], 1);
            mbar_init(&bars->s_free[s], 4);
            mbar_init(&bars->p_ready[s], 4);
            mbar_init(&bars->pv_done[s], 1);
            mbar_init(&bars->o_free[s], 4);
            mbar_init(&bars->o_staged[s], 4);
        }
        mbar_init(&bars->drain, 1);
        bars->ring.init(kWorkConsumers);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmO);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, kFwdTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    griddep_launch_dependents();
    if (warp == 0 && lane == 0) {  // the first item's Q tiles and first K, V tiles on their way into L2 meanwhile
        int blk, bh, n_a, n_b;
        {
            wk.get(blockIdx.x, &blk, &bh, &n_a, &n_b);
            const int head = kStrided ? bh % wk.H : 0, batch = kStrided ? bh / wk.H : 0;
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h) {
                tma_prefetch_tile<kStrided>(&tmK, (wk.orders >> 4) & 15, h * kBoxCols, 0, head, batch, bh);
                tma_prefetch_tile<kStrided>(&tmQ, wk.orders & 15, h * kBoxCols, blk * kBlockRows, head, batch, bh);
                tma_prefetch_tile<kStrided>(&tmV, (wk.orders >> 8) & 15, h * kBoxCols, 0, head, batch, bh);
                tma_prefetch_tile<kStrided>(&tmQ, wk.orders & 15, h * kBoxCols, blk * kBlockRows + kBlockQ, head, batch, bh);
            }
        }
    }
    griddep_wait();  // everything above overlaps the previous kernel of the stream

    if (warp == 0) {
        if (lane == 0) fwd_producer<D, kStrided>(&tmQ, &tmK, &tmV, smem, bars, wk, limit, inject);
    } else if (warp == 1) {
        fwd_mma<D>(smem, bars, tmem_base, wk, limit);
    } else if (warp >= 4) {
        const int t = (warp - 4) >> 2;
        fwd_softmax<D, kCausal, kStrided>(smem, bars, tmem_base, &tmO, LSE, scale, wk, t, (warp - 4) & 3, lane, limit);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kFwdTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

template <int D, bool kCausal>
cudaError_t launch_one(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       const CUtensorMap& tmO, bool strided, uint32_t orders, float* LSE, const AttnShape& s,
                       int num_sms, long long wait_limit, int inject, int* dev_status, cudaStream_t stream) {
    const int n_blocks = (s.T + kBlockRows - 1) / kBlockRows;
    const int BH = s.B * s.H;
    const long long n_items = static_cast<long long>(n_blocks) * BH;
    (void)num_sms;
    const dim3 grid(static_cast<unsigned>(n_items));  // one CTA per item; those that do not start at once are taken over
    if (strided)
        return launch_overlapped(attn_fwd_kernel<D, kCausal, true>, grid, dim3(kFwdThreads), FwdCfg<D>::kSmemBytes,
                                 stream, tmQ, tmK, tmV, tmO, LSE, s.T, BH, s.H, orders, n_blocks, s.scale, wait_limit, inject, dev_status);
    return launch_overlapped(attn_fwd_kernel<D, kCausal, false>, grid, dim3(kFwdThreads), FwdCfg<D>::kSmemBytes, stream,
                             tmQ, tmK, tmV, tmO, LSE, s.T, BH, s.H, orders, n_blocks, s.scale, wait_limit, inject, dev_status);
}

template <int D, bool kCausal, bool kStrided>
cudaError_t configure_one() {
    return cudaFuncSetAttribute(attn_fwd_kernel<D, kCausal, kStrided>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                FwdCfg<D>::kSmemBytes);
}

}  // namespace

cudaError_t configure_attn_fwd() {
    const cudaError_t r[8] = {configure_one<64, true, false>(),  configure_one<64, false, false>(),
                              configure_one<128, true, false>(), configure_one<128, false, false>(),
                              configure_one<64, true, true>(),   configure_one<64, false, true>(),
                              configure_one<128, true, true>(),  configure_one<128, false, true>()};
    for (cudaError_t e : r)
        if (e != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t launch_attn_fwd(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            const CUtensorMap& tmO, bool strided, uint32_t orders, float* LSE, const AttnShape& s,
                            int num_sms, long long wait_limit, int inject, int* dev_status, cudaStream_t stream) {
    if (s.D == 64) {
        return s.causal ? launch_one<64, true>(tmQ, tmK, tmV, tmO, strided, orders, LSE, s, num_sms, wait_limit, inject, dev_status, stream)
                        : launch_one<64, false>(tmQ, tmK, tmV, tmO, strided, orders, LSE, s, num_sms, wait_limit, inject, dev_status, stream);
    }
    return s.causal ? launch_one<128, true>(tmQ, tmK, tmV, tmO, strided, orders, LSE, s, num_sms, wait_limit, inject, dev_status, stream)
                    : launch_one<128, false>(tmQ, tmK, tmV, tmO, strided, orders, LSE, s, num_sms, wait_limit, inject, dev_status, stream);
}

}  // namespace nova
