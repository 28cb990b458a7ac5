// Fused causal attention backward for sm_100a (paper Section 4.2, "The Backward Pass": P is
// recomputed from the saved log-sum-exp, never stored; dQ reduces over keys, dK/dV over queries;
// the causal loop bound is raised so query tiles above the diagonal are never visited).
//
// A work item is one 128-key tile of one (batch, head): K_j and V_j stay in shared memory while the
// query tiles i >= j stream past.  Everything is computed transposed (keys on TMEM lanes) so that
// P^T and dS^T can feed the tensor cores straight from TMEM:
//   S^T  = K_j Q_i^T            (smem x smem -> TMEM)
//   dP^T = V_j dO_i^T           (smem x smem -> TMEM)
//   P^T  = exp2(S^T*c - LSE_i*log2e),  dS^T = P^T * (dP^T - Delta_i)      (compute warps, fp32)
//   dV  += P^T  dO_i            (TMEM x smem, dO read MN-major)
//   dK  += dS^T Q_i             (TMEM x smem, Q  read MN-major)
//   dQ_i = dS K_j               (dS^T staged as bf16 in shared memory and read M-major; K MN-major)
//
// The kernel is persistent: one CTA per SM walks a fixed list of work items, heaviest first and dealt
// out in zig-zag order so that every CTA gets the same number of tile pairs to within one.  All
// pipelines run across item boundaries: the loads, the S^T/dP^T products and the first P phase of the
// next item overlap the dK/dV write-out of the current one.
//
// Warp roles (512 threads):
//   warp 0       TMA producer (K_j, V_j per item and dO_i double-buffered at D=64; Q_i always)
//   warp 1       UMMA issuer, software-pipelined: S^T of the next query tile is issued as soon as the
//                compute warps have read the current one; dK, dQ and the next dP^T run while they
//                work on the next P
//   warps 2-3    row loader: -LSE*log2e and -Delta of the query tile into shared memory
//   warps 4-11   compute: thread = (key row, 64-query half); P phase then dS phase per tile
//                (at D=128 they also send dV and dK at the end of an item, through the dS^T staging buffer)
//   warps 12-15  dQ: one thread per row moves the partial dQ tile from TMEM into the fp32 accumulator
//                with TMA reduce-add operations through a swizzled staging buffer (a separate kernel
//                scales and rounds it once); at D=64 they also send dV and dK
//                of a finished item out through the same buffer with TMA stores
//
// TMEM columns (D=64): S^T [0,128)  dP^T/dS^T [128,256)  dV [256,320)  dK [320,384)  dQ [384,448)
//                      P^T [448,512): P^T has its own columns, so S^T of the next query tile is
//                      issued before dV of the current one and the compute warps never wait for it
//              (D=128): S^T/P^T [0,128)  dP^T/dS^T, then dQ [128,256)  dV [256,384)  dK [384,512)
// Where bf16 P^T / dS^T share columns with the fp32 tile they came from, query half h writes only
// over its own already-read columns [64h, 64h+32), so the two compute warpgroups never collide.
//
// Warp-wide .sync.aligned instructions (TMEM loads/stores) need the whole warp together: wherever
// one lane does extra work (the dQ leader), the warp is rejoined with a vote before the next one.
#include <type_traits>

#include "kernels.h"
#include "ptx.cuh"
#include "work_plan.h"

namespace nova {
namespace {

constexpr int kBwdTmemCols = 512;

template <int D>
struct BwdCfg {
    static constexpr int kHalves = D / kBoxCols;
    static constexpr int kTileBytes = kHalves * kHalfTileBytes;
    static constexpr int kKVStages = (D == 64) ? 2 : 1;
    static constexpr int kdOStages = (D == 64) ? 2 : 1;
    static constexpr int kOffK = 0;                                   // kKVStages x K tile
    static constexpr int kOffV = kKVStages * kTileBytes;              // kKVStages x V tile
    // Three Q stages where shared memory has room: a Q tile is requested two tiles ahead, so that S^T of
    // the next tile never waits for it.
    static constexpr int kQStages = (D == 64) ? 3 : 2;
    static constexpr int kOffQ = 2 * kKVStages * kTileBytes;          // kQStages stages
    static constexpr int kOffdO = kOffQ + kQStages * kTileBytes;      // kdOStages stages
    static constexpr int kOffdS = kOffdO + kdOStages * kTileBytes;    // [2 query halves][128 keys][64 queries] bf16
    static constexpr int kOffRow = kOffdS + 2 * kHalfTileBytes;       // 2 x (-LSE*log2e[128], -Delta[128]) fp32
    // Staging buffer of the dQ warps: two boxes of [128 rows x 128 bytes], 128-byte swizzled like every
    // other tile (fp32 [128 x 32] each for dQ; at D=64 also bf16 [128 x 64] each for dV and dK, which the
    // dQ warps then send out too: kBulkdQ).
    static constexpr bool kBulkdQ = (D == 64);
    static constexpr int kStageBytes = 2 * kHalfTileBytes;
    static constexpr int kOffStage = kOffRow + 2 * 2 * 128 * 4;
    static constexpr int kOffBar = kOffStage + kStageBytes;
    // At D=128 the tiles fill the 227 KB a CTA can have to within 512 bytes, so there is no room for
    // the padding that would let the kernel align its window itself: the kernel checks that the window
    // starts on a 1024-byte boundary (it does on sm_100) and gives up cleanly if not.
    static constexpr int kAlignPad = (D == 64) ? 1024 : 0;
    static constexpr int kSmemBytes = kOffBar + 512 + kAlignPad;
    static_assert(kSmemBytes <= 232448, "exceeds the shared memory of one CTA");
    static constexpr int kColS = 0;
    static constexpr int kColdP = 128;
    static constexpr int kColdV = 256;
    static constexpr int kColdK = 256 + D;
    static constexpr bool kdQAliased = (D == 128);  // dQ reuses the dP^T region
    static constexpr int kColdQ = (D == 64) ? 384 : 128;
    // Where dQ lies over dP^T, a bf16 dS^T kept in those columns would force dK (which reads it) to run before
    // dQ (which overwrites it), and dQ, its read-out and the next dP^T are the chain that sets the period of a
    // tile.  There dK reads dS^T from the shared-memory copy that dQ uses as well (K-major for dK, M-major for
    // dQ), dQ is queued first and dK runs while the dQ warps empty the columns.
    static constexpr bool kdKFromSmem = kdQAliased;
    static constexpr bool kSeparateP = (D == 64);   // P^T in its own columns instead of over S^T
    static constexpr int kColP = kSeparateP ? 448 : 0;
    static constexpr int kPHalfStride = kSeparateP ? 32 : 64;  // column distance between the two query halves of P^T
    // Queries per compute thread: 128 / kQPT warpgroups of compute warps.  Two warpgroups of 64 queries each:
    // four of 32 (four compute warps per scheduler, 768 threads, 80 registers) were measured 26 % slower at
    // D=64 (78.3 against 62.1 us on B=8, H=12, T=1024).
    static constexpr int kQPT = 64;
    static constexpr int kComputeWarps = 4 * (128 / kQPT);
    static constexpr int kThreads = 32 * (4 + kComputeWarps + 4);  // producer, UMMA, 2 row loaders, compute, 4 dQ
};

struct BwdBars {
    uint64_t kv_full[2], kv_empty[2];
    uint64_t q_full[3], q_empty[3];
    uint64_t do_full[2], do_empty[2];
    uint64_t s_full, dp_full;         // UMMA -> compute
    uint64_t p_ready, ds_ready;       // compute (one arrival per warp) -> UMMA
    uint64_t dq_full, dq_free;
    uint64_t row_full[2], row_empty[2];
    uint64_t stage_full, stage_free;  // dQ warps <-> their leader thread
    uint64_t dkv_full, dkv_free;      // UMMA -> readers: dV/dK of an item complete; readers -> UMMA: read out
    uint64_t drain;
    uint64_t out_sync;  // the compute warps among themselves, at the end of an item (D=128)
    uint32_t tmem_base;
    int abort_flag;
};

template <int D, bool kStrided>
__device__ __forceinline__ void bwd_producer(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV,
                                             const CUtensorMap* tmdO, uint8_t* smem, BwdBars* bars,
                                             const WorkList& wl) {
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    int armed_kv[2] = {-1, -1}, armed_q[3] = {-1, -1, -1}, armed_do[2] = {-1, -1};
    bool ok = true;
    int w = 0, g = 0;  // items and query tiles processed so far by this CTA
    for (WorkCursor cur; !wl.done(cur) && ok; wl.advance(cur)) {
        int kt, bh, i0, n_it;
        if (!wl.get(cur, &kt, &bh, &i0, &n_it)) continue;
        const int head = kStrided ? bh % wl.H() : 0, batch = kStrided ? bh / wl.H() : 0;
        const int ks = w % Cfg::kKVStages;
        const uint32_t kph = (w / Cfg::kKVStages) & 1;
        ok = mbar_wait(&bars->kv_empty[ks], kph ^ 1, abort_flag);
        if (!ok) break;
        mbar_expect_tx(&bars->kv_full[ks], 2 * Cfg::kTileBytes);
        armed_kv[ks] = kph;
#pragma unroll
        for (int h = 0; h < Cfg::kHalves; ++h) {
            tma_load_tile<kStrided>(smem + Cfg::kOffK + ks * Cfg::kTileBytes + h * kHalfTileBytes, tmK, &bars->kv_full[ks],
                          (wl.orders() >> 4) & 15, h * kBoxCols, kt * kBlockK, head, batch, bh);
            tma_load_tile<kStrided>(smem + Cfg::kOffV + ks * Cfg::kTileBytes + h * kHalfTileBytes, tmV, &bars->kv_full[ks],
                          (wl.orders() >> 8) & 15, h * kBoxCols, kt * kBlockK, head, batch, bh);
        }
        for (int it = 0; it < n_it; ++it, ++g) {
            const int st = g % Cfg::kQStages;
            const int qrow = (i0 + it) * kBlockQ;
            ok = mbar_wait(&bars->q_empty[st], ((g / Cfg::kQStages) & 1) ^ 1, abort_flag);
            if (!ok) break;
            mbar_expect_tx(&bars->q_full[st], Cfg::kTileBytes);
            armed_q[st] = (g / Cfg::kQStages) & 1;
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h)
                tma_load_tile<kStrided>(smem + Cfg::kOffQ + st * Cfg::kTileBytes + h * kHalfTileBytes, tmQ, &bars->q_full[st],
                              wl.orders() & 15, h * kBoxCols, qrow, head, batch, bh);
            const int ds = g % Cfg::kdOStages;
            const uint32_t dph = (g / Cfg::kdOStages) & 1;
            ok = mbar_wait(&bars->do_empty[ds], dph ^ 1, abort_flag);
            if (!ok) break;
            mbar_expect_tx(&bars->do_full[ds], Cfg::kTileBytes);
            armed_do[ds] = dph;
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h)
                tma_load_tile<kStrided>(smem + Cfg::kOffdO + ds * Cfg::kTileBytes + h * kHalfTileBytes, tmdO, &bars->do_full[ds],
                              (wl.orders() >> 12) & 15, h * kBoxCols, qrow, head, batch, bh);
        }
        ++w;
    }
    if (!ok) {
        // Giving up: let the copies already in flight land before the CTA's shared memory goes away.
        int none = 0;
        for (int s = 0; s < 2; ++s) {
            if (armed_kv[s] >= 0) (void)mbar_wait(&bars->kv_full[s], armed_kv[s], &none);
            if (armed_do[s] >= 0) (void)mbar_wait(&bars->do_full[s], armed_do[s], &none);
        }
        for (int s = 0; s < Cfg::kQStages; ++s)
            if (armed_q[s] >= 0) (void)mbar_wait(&bars->q_full[s], armed_q[s], &none);
    }
}

template <int D>
__device__ __forceinline__ void bwd_mma(uint8_t* smem, BwdBars* bars, uint32_t tmem_base, const WorkList& wl) {
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    constexpr uint32_t kIdescT = umma_idesc_bf16(128, 128, 0, 0);   // S^T, dP^T
    constexpr uint32_t kIdescKV = umma_idesc_bf16(128, D, 0, 1);    // dV, dK (A from TMEM, B MN-major)
    constexpr uint32_t kIdescdQ = umma_idesc_bf16(128, 64, 1, 1);   // dQ half (A M-major smem, B MN-major)
    constexpr uint32_t kIdescdQWide = umma_idesc_bf16(128, D, 1, 1);  // all D columns of dQ at once
    const uint32_t t_s = tmem_base + Cfg::kColS, t_dp = tmem_base + Cfg::kColdP;
    const uint32_t t_dv = tmem_base + Cfg::kColdV, t_dk = tmem_base + Cfg::kColdK;
    const uint32_t t_p = tmem_base + Cfg::kColP;
    // Descriptor lower words per buffer, computed once; in the loops only a constant (byte offset >> 4)
    // is added.  "_k": read K-major (rows of the operand are its M/N index), "_m": read MN-major (rows
    // are its K index; LBO = distance between 64-element halves).
    const uint32_t hi = umma_desc_hi_sw128(1024);
    // Q stage st: the address field counts 16-byte units, so a stage is kTileBytes / 16 further on.
    const uint32_t q_k0 = umma_desc_lo(smem_u32(smem + Cfg::kOffQ), 16);
    const uint32_t q_m0 = umma_desc_lo(smem_u32(smem + Cfg::kOffQ), kHalfTileBytes);
    constexpr uint32_t kQStageStep = Cfg::kTileBytes >> 4;
    uint32_t do_k[2], do_m[2];
#pragma unroll
    for (int st = 0; st < 2; ++st) {
        do_k[st] = umma_desc_lo(smem_u32(smem + Cfg::kOffdO + (st % Cfg::kdOStages) * Cfg::kTileBytes), 16);
        do_m[st] = umma_desc_lo(smem_u32(smem + Cfg::kOffdO + (st % Cfg::kdOStages) * Cfg::kTileBytes), kHalfTileBytes);
    }
    const uint32_t ds_m = umma_desc_lo(smem_u32(smem + Cfg::kOffdS), kHalfTileBytes);
    const uint32_t ds_k = umma_desc_lo(smem_u32(smem + Cfg::kOffdS), 16);
    uint32_t k_k = 0, v_k = 0, k_m = 0;  // per item
    // The whole warp runs this role in uniform control flow; one elected lane issues.
    const bool el = elect_one();

    auto issue_st = [&](int gq, uint32_t kd) {  // S^T = K Q^T: K tile `kd`, query tile in Q stage gq % kQStages
        const uint32_t b = q_k0 + (gq % Cfg::kQStages) * kQStageStep;
        if (el) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = ((k / 4) * kHalfTileBytes + (k % 4) * 32) >> 4;
                umma_ss(t_s, umma_desc_join(kd + off, hi), umma_desc_join(b + off, hi), kIdescT, k > 0 ? 1u : 0u);
            }
            tc_commit(&bars->s_full);
        }
        __syncwarp();
    };
    auto issue_dpt = [&](int gq, uint32_t vd) {  // dP^T = V dO^T: V tile `vd`, query tile in dO stage gq % kdOStages
        const uint32_t b = do_k[gq % Cfg::kdOStages];
        if (el) {
#pragma unroll
            for (int k = 0; k < D / 16; ++k) {
                const uint32_t off = ((k / 4) * kHalfTileBytes + (k % 4) * 32) >> 4;
                umma_ss(t_dp, umma_desc_join(vd + off, hi), umma_desc_join(b + off, hi), kIdescT, k > 0 ? 1u : 0u);
            }
            tc_commit(&bars->dp_full);
        }
        __syncwarp();
    };

    bool ok = true;
    bool first_queued = false;  // S^T and dP^T of this item's first tile were queued during the previous item
    int w = 0, g = 0;
    for (WorkCursor cur; !wl.done(cur) && ok; wl.advance(cur)) {
        int kt, bh, i0, n_it;
        if (!wl.get(cur, &kt, &bh, &i0, &n_it)) continue;
        // With K/V double-buffered the next item's tiles arrive while this one runs, and the products
        // of its first query tile are queued from inside this item's last iteration (below), exactly
        // as for any other next tile: the compute warps never see the item boundary.
        int kt_n, bh_n, i0_n, n_it_n;
        WorkCursor nxt = cur;
        wl.advance(nxt);
        const bool has_next = Cfg::kKVStages > 1 && !wl.done(nxt) && wl.get(nxt, &kt_n, &bh_n, &i0_n, &n_it_n);
        const int ks_n = (w + 1) % Cfg::kKVStages;
        const uint32_t k_k_n = umma_desc_lo(smem_u32(smem + Cfg::kOffK + ks_n * Cfg::kTileBytes), 16);
        const uint32_t v_k_n = umma_desc_lo(smem_u32(smem + Cfg::kOffV + ks_n * Cfg::kTileBytes), 16);
        const int ks = w % Cfg::kKVStages;
        k_k = umma_desc_lo(smem_u32(smem + Cfg::kOffK + ks * Cfg::kTileBytes), 16);
        k_m = umma_desc_lo(smem_u32(smem + Cfg::kOffK + ks * Cfg::kTileBytes), kHalfTileBytes);
        v_k = umma_desc_lo(smem_u32(smem + Cfg::kOffV + ks * Cfg::kTileBytes), 16);
        ok = mbar_wait(&bars->kv_full[ks], (w / Cfg::kKVStages) & 1, abort_flag);
        if (ok) ok = mbar_wait(&bars->q_full[g % Cfg::kQStages], (g / Cfg::kQStages) & 1, abort_flag);
        if (ok && Cfg::kdQAliased && g > 0 && !wl.no_dq()) ok = mbar_wait(&bars->dq_free, (g - 1) & 1, abort_flag);
        if (ok) ok = mbar_wait(&bars->do_full[g % Cfg::kdOStages], (g / Cfg::kdOStages) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        // The S^T and dP^T columns are free: the last dV / dK (and, at D=128, the dQ read-out) of the
        // previous item were queued or awaited before this point and the pipe executes in order.
        if (!first_queued) {
            issue_st(g, k_k);
            issue_dpt(g, v_k);
        }
        first_queued = false;
        for (int it = 0; it < n_it && ok; ++it, ++g) {
            const bool more = it + 1 < n_it;
            const bool cross = !more && has_next && Cfg::kSeparateP && !Cfg::kdQAliased;  // next tile opens the next item
            ok = mbar_wait(&bars->p_ready, g & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            if (Cfg::kSeparateP && (more || cross)) {  // S^T columns are free as soon as the compute warps have read them
                if (cross) ok = mbar_wait(&bars->kv_full[ks_n], ((w + 1) / Cfg::kKVStages) & 1, abort_flag);
                if (ok) ok = mbar_wait(&bars->q_full[(g + 1) % Cfg::kQStages], ((g + 1) / Cfg::kQStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_st(g + 1, cross ? k_k_n : k_k);
            }
            if (it == 0 && w > 0) {  // the previous item's dV/dK have been read out of TMEM
                ok = mbar_wait(&bars->dkv_free, (w - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
            }
            // dV += P^T dO_i: 16 queries (8 packed TMEM columns, 16 smem rows = 2048 bytes) per instruction.
            if (el) {
                const uint32_t b = do_m[g % Cfg::kdOStages];
#pragma unroll
                for (int k = 0; k < kBlockQ / 16; ++k)
                    umma_ts(t_dv, t_p + (k / 4) * Cfg::kPHalfStride + (k % 4) * 8, umma_desc_join(b + k * 128, hi),
                            kIdescKV, (it > 0 || k > 0) ? 1u : 0u);
                tc_commit(&bars->do_empty[g % Cfg::kdOStages]);
            }
            __syncwarp();
            if (!Cfg::kSeparateP && more) {  // P^T lives in the S^T columns: dV must be queued first
                ok = mbar_wait(&bars->q_full[(g + 1) % Cfg::kQStages], ((g + 1) / Cfg::kQStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_st(g + 1, k_k);
            }
            ok = mbar_wait(&bars->ds_ready, g & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            if (Cfg::kdKFromSmem) {
                // dQ_i = dS K_j first, all D columns per instruction (the dP^T columns it lands in were read by the
                // compute warps before they arrived on ds_ready), then dK += dS^T Q_i with dS^T from shared memory.
                if (el) {
                    if (!wl.no_dq()) {
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k)
                            umma_ss(tmem_base + Cfg::kColdQ, umma_desc_join(ds_m + k * 128, hi),
                                    umma_desc_join(k_m + k * 128, hi), kIdescdQWide, k > 0 ? 1u : 0u);
                        tc_commit(&bars->dq_full);
                    }
                    const uint32_t b = q_m0 + (g % Cfg::kQStages) * kQStageStep;
#pragma unroll
                    for (int k = 0; k < kBlockQ / 16; ++k) {
                        const uint32_t off = ((k / 4) * kHalfTileBytes + (k % 4) * 32) >> 4;
                        umma_ss(t_dk, umma_desc_join(ds_k + off, hi), umma_desc_join(b + k * 128, hi), kIdescKV,
                                (it > 0 || k > 0) ? 1u : 0u);
                    }
                    tc_commit(&bars->q_empty[g % Cfg::kQStages]);
                }
                __syncwarp();
            } else {
            if (el) {
                const uint32_t b = q_m0 + (g % Cfg::kQStages) * kQStageStep;
#pragma unroll
                for (int k = 0; k < kBlockQ / 16; ++k)
                    // bf16 dS^T of 16 queries: 8 packed columns at the start of the fp32 columns of their thread
                    umma_ts(t_dk, t_dp + (k / (Cfg::kQPT / 16)) * Cfg::kQPT + (k % (Cfg::kQPT / 16)) * 8,
                            umma_desc_join(b + k * 128, hi), kIdescKV,
                            (it > 0 || k > 0) ? 1u : 0u);
                tc_commit(&bars->q_empty[g % Cfg::kQStages]);
            }
            __syncwarp();
            // dQ_i = dS K_j, 64 head-dim columns per accumulator half; 16 keys per instruction.
            if (!Cfg::kdQAliased && !wl.no_dq()) {  // the dQ warps must have read the previous tile out of the dQ columns
                ok = mbar_wait(&bars->dq_free, (g & 1) ^ 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
            }
            if (el && !wl.no_dq()) {
#pragma unroll
                for (int h = 0; h < Cfg::kHalves; ++h) {
                    const uint32_t t_dq = tmem_base + Cfg::kColdQ + h * 64;
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k)
                        umma_ss(t_dq, umma_desc_join(ds_m + k * 128, hi),
                                umma_desc_join(k_m + h * (kHalfTileBytes >> 4) + k * 128, hi), kIdescdQ,
                                k > 0 ? 1u : 0u);
                }
                tc_commit(&bars->dq_full);
            }
            __syncwarp();
            }
            if (more || cross) {
                if (Cfg::kdQAliased && !wl.no_dq()) {  // dQ sits in the dP^T region until the dQ warps have read it
                    ok = mbar_wait(&bars->dq_free, g & 1, abort_flag);
                    if (!ok) break;
                }
                ok = mbar_wait(&bars->do_full[(g + 1) % Cfg::kdOStages], ((g + 1) / Cfg::kdOStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_dpt(g + 1, cross ? v_k_n : v_k);
                if (cross) first_queued = true;
            }
        }
        if (!ok) break;
        if (el) {
            tc_commit(&bars->kv_empty[ks]);  // K_j and V_j are no longer read
            tc_commit(&bars->dkv_full);      // dV and dK of this item are complete
        }
        __syncwarp();
        ++w;
    }
    if (!ok) {
        int none = 0;
        if (el) tc_commit(&bars->drain);
        __syncwarp();
        (void)mbar_wait(&bars->drain, 0, &none);
    }
}

// Row loader: -LSE*log2e and -Delta of each query tile into the double-buffered row arrays (negated,
// so that the compute warps fold them in with a packed fma / add).
__device__ __forceinline__ void bwd_rows(BwdBars* bars, float* row_buf, const float* __restrict__ LSE,
                                         const float* __restrict__ Delta, int T, const WorkList& wl, int tid64) {
    volatile int* abort_flag = &bars->abort_flag;
    int g = 0;
    for (WorkCursor cur; !wl.done(cur); wl.advance(cur)) {
        int kt, bh, i0, n_it;
        if (!wl.get(cur, &kt, &bh, &i0, &n_it)) continue;
        const size_t row_base = static_cast<size_t>(bh) * T;
        for (int it = 0; it < n_it; ++it, ++g) {
            const int b = g & 1;
            if (!mbar_wait(&bars->row_empty[b], ((g >> 1) & 1) ^ 1, abort_flag)) return;
            float* s_lse = row_buf + b * 256;
            float* s_dl = s_lse + 128;
#pragma unroll
            for (int x = 0; x < 2; ++x) {
                const int rl = tid64 + 64 * x;
                const int q = (i0 + it) * kBlockQ + rl;
                // Rows past the end of the sequence get LSE = +inf so that their P is exactly 0.
                s_lse[rl] = (q < T) ? -LSE[row_base + q] * kLog2e : -INFINITY;
                s_dl[rl] = (q < T) ? -Delta[row_base + q] : 0.f;
            }
            __syncwarp();
            if ((tid64 & 31) == 0) mbar_arrive(&bars->row_full[b]);
        }
    }
}

// P phase for this thread's N queries: p = exp2(s*c - lse*log2e), left in place of the scores as fp32
// (the dS phase multiplies by the unrounded p: only what feeds a contraction is rounded to bf16, paper
// Section 4.3).  `s_lse4` holds -lse*log2e; the multiply-add runs on packed fp32 pairs.
// kMasked: the tile is the diagonal one and/or holds keys past the end of the sequence.
template <bool kMasked, int N>
__device__ __forceinline__ void bwd_p_phase(uint32_t (&sv)[N], const float4* s_lse4, float c, bool key_valid, bool diag,
                                            int r, int q_base) {
#pragma unroll
    for (int g = 0; g < N / 4; ++g) {
        const float4 l4 = s_lse4[g];
        const uint64_t c2 = f32x2_pack(c, c);
        float x0, x1, x2, x3;
        f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(sv[4 * g + 0]), __uint_as_float(sv[4 * g + 1])), c2,
                               f32x2_pack(l4.x, l4.y)), x0, x1);
        f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(sv[4 * g + 2]), __uint_as_float(sv[4 * g + 3])), c2,
                               f32x2_pack(l4.z, l4.w)), x2, x3);
        float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
        if (kMasked) {
            // keep (query q, key r) iff the key exists and, on the diagonal tile, key <= query
            const int q0 = q_base + 4 * g;
            if (!key_valid || (diag && r > q0 + 0)) p0 = 0.f;
            if (!key_valid || (diag && r > q0 + 1)) p1 = 0.f;
            if (!key_valid || (diag && r > q0 + 2)) p2 = 0.f;
            if (!key_valid || (diag && r > q0 + 3)) p3 = 0.f;
        }
        sv[4 * g + 0] = __float_as_uint(p0);
        sv[4 * g + 1] = __float_as_uint(p1);
        sv[4 * g + 2] = __float_as_uint(p2);
        sv[4 * g + 3] = __float_as_uint(p3);
    }
}

// Compute warps.  A thread owns one key row and kQPT consecutive queries of the tile (64: two warpgroups;
// 32: four), i.e. columns [kQPT*part, kQPT*(part+1)) of S^T and dP^T.
template <int D, bool kCausal, bool kStrided>
__device__ __forceinline__ void bwd_compute(uint8_t* smem, BwdBars* bars, uint32_t tmem_base, const CUtensorMap* tmdK,
                                            const CUtensorMap* tmdV, int T, float scale, const WorkList& wl, int cwarp,
                                            int lane) {
    using Cfg = BwdCfg<D>;
    constexpr int kQPT = Cfg::kQPT;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (cwarp & 3);
    const int part = cwarp >> 2;             // which kQPT queries of the tile this thread covers
    const int half = (part * kQPT) / 64;     // the 64-query half they lie in (a box of the dS^T staging buffer)
    const int r = lane_base + lane;          // local key row
    const float c = scale * kLog2e;
    const uint32_t t_s = tmem_addr(tmem_base, lane_base, Cfg::kColS + kQPT * part);
    const uint32_t t_dp = tmem_addr(tmem_base, lane_base, Cfg::kColdP + kQPT * part);
    // bf16 P^T: kQPT / 2 packed columns, in columns of their own or over this thread's own S^T columns
    const uint32_t t_p = tmem_addr(tmem_base, lane_base, Cfg::kColP + (Cfg::kSeparateP ? kQPT / 2 : kQPT) * part);
    const float* row_buf = reinterpret_cast<const float*>(smem + Cfg::kOffRow);
    uint8_t* sdS_row = smem + Cfg::kOffdS + half * kHalfTileBytes + r * 128;
    const int ch0 = ((part * kQPT) % 64) / 8;  // first 16-byte chunk of this thread's queries in the 128-byte row
    bool ok = true;
    int w = 0, g = 0;
    int n_sync = 0;  // uses of out_sync so far

    for (WorkCursor cur; !wl.done(cur) && ok; wl.advance(cur)) {
        int kt, bh, i0, n_it;
        if (!wl.get(cur, &kt, &bh, &i0, &n_it)) continue;
        const int key = kt * kBlockK + r;
        const bool key_valid = key < T;
        const bool tile_keys_valid = (kt * kBlockK + kBlockK) <= T;

        for (int it = 0; it < n_it; ++it, ++g) {
            const int i = i0 + it;
            const int b = g & 1;
            const float4* s_lse4 = reinterpret_cast<const float4*>(row_buf + b * 256 + kQPT * part);
            const float4* s_dl4 = reinterpret_cast<const float4*>(row_buf + b * 256 + 128 + kQPT * part);
            // Three non-blocking probes issued together, so that their latencies overlap; each is followed up by
            // a proper wait only if it failed (-2 % against three waits in a row).
            const bool row_there = mbar_test(&bars->row_full[b], (g >> 1) & 1);
            const bool s_there = mbar_test(&bars->s_full, g & 1);
            const bool dp_there = mbar_test(&bars->dp_full, g & 1);
            if (!row_there) ok = mbar_wait(&bars->row_full[b], (g >> 1) & 1, abort_flag);
            if (ok && !s_there) ok = mbar_wait(&bars->s_full, g & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();

            // ---- P phase: the scores become fp32 probabilities in place
            uint32_t pf[kQPT];
#pragma unroll
            for (int x = 0; x < kQPT; x += 32) tmem_ld_x32(t_s + x, pf + x);
            tmem_wait_ld();
            {
                const bool diag = kCausal && (i == kt);
                if (diag || !tile_keys_valid)
                    bwd_p_phase<true, kQPT>(pf, s_lse4, c, key_valid, diag, r, kQPT * part);
                else
                    bwd_p_phase<false, kQPT>(pf, s_lse4, c, true, false, r, kQPT * part);
            }
            // P^T as bf16 into TMEM for dV.  Where P^T has columns of its own (kEarlydP) the store must wait
            // until dV of the previous tile has read them: dP^T of this tile was queued after that dV and the
            // tensor pipe completes in order, so the dp_full wait covers it, and the first dP^T load is issued
            // before the P^T store is awaited so that the two TMEM round trips overlap.
            constexpr bool kEarlydP = Cfg::kSeparateP && !Cfg::kdQAliased;
            static_assert(kEarlydP || !Cfg::kSeparateP, "P^T columns of their own need the dp_full wait below");
            if (kEarlydP) {
                if (!dp_there) ok = mbar_wait(&bars->dp_full, g & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
            }
#pragma unroll
            for (int x = 0; x < kQPT; x += 32) {
                uint32_t pk[16];
#pragma unroll
                for (int y = 0; y < 16; ++y)
                    pk[y] = pack_bf16x2(__uint_as_float(pf[x + 2 * y]), __uint_as_float(pf[x + 2 * y + 1]));
                tmem_st_x16(t_p + x / 2, pk);
            }
            uint32_t dv[16];
            if (kEarlydP) tmem_ld_x16(t_dp, dv);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->p_ready);
            if (!kEarlydP) {
                ok = mbar_wait(&bars->dp_full, g & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                tmem_ld_x16(t_dp, dv);
            }
            // ---- dS phase, 16 queries at a time: ds = p * (dp - delta) in fp32, rounded once to bf16, to TMEM
            // (over this thread's own, already read dP^T columns) for dK and to swizzled smem for dQ.
            // dP^T of this tile was queued after dQ of the previous one and the tensor pipe completes in order,
            // so the dp_full wait also covers "the previous dQ has finished reading the dS staging buffer".
#pragma unroll
            for (int x = 0; x < kQPT; x += 16) {
                tmem_wait_ld();
                uint32_t dd[8];
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    const float4 d4 = s_dl4[x / 4 + y];  // holds -delta
                    float d0, d1, d2, d3;
                    f32x2_unpack(f32x2_mul(f32x2_pack(__uint_as_float(pf[x + 4 * y + 0]), __uint_as_float(pf[x + 4 * y + 1])),
                                           f32x2_add(f32x2_pack(__uint_as_float(dv[4 * y + 0]), __uint_as_float(dv[4 * y + 1])),
                                                     f32x2_pack(d4.x, d4.y))), d0, d1);
                    f32x2_unpack(f32x2_mul(f32x2_pack(__uint_as_float(pf[x + 4 * y + 2]), __uint_as_float(pf[x + 4 * y + 3])),
                                           f32x2_add(f32x2_pack(__uint_as_float(dv[4 * y + 2]), __uint_as_float(dv[4 * y + 3])),
                                                     f32x2_pack(d4.z, d4.w))), d2, d3);
                    dd[2 * y + 0] = pack_bf16x2(d0, d1);
                    dd[2 * y + 1] = pack_bf16x2(d2, d3);
                }
                if (x + 16 < kQPT) tmem_ld_x16(t_dp + x + 16, dv);  // all of dv has been consumed above
                if (!Cfg::kdKFromSmem) tmem_st_x8(t_dp + x / 2, dd);
                if (Cfg::kdKFromSmem || !wl.no_dq()) {  // dS^T row r: two 16-byte chunks of one 128-byte swizzled row
                    const int ch = ch0 + x / 8;
                    *reinterpret_cast<uint4*>(sdS_row + (((ch + 0) ^ (r & 7)) << 4)) = make_uint4(dd[0], dd[1], dd[2], dd[3]);
                    *reinterpret_cast<uint4*>(sdS_row + (((ch + 1) ^ (r & 7)) << 4)) = make_uint4(dd[4], dd[5], dd[6], dd[7]);
                }
            }
            if (!Cfg::kdKFromSmem) tmem_wait_st();
            fence_proxy_async_smem();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(&bars->ds_ready);
                mbar_arrive(&bars->row_empty[b]);
            }
        }
        if (!ok) break;
        if constexpr (!Cfg::kBulkdQ) {
            // ---- end of the item (D=128): dV, then dK (scaled), of this key row, D/2 columns of each per thread,
            // rounded to bf16 into the dS^T staging buffer (idle now: every product of the item has completed)
            // as two boxes of [128 keys x 64 columns], and out with two TMA stores each.  (Stores of 16 bytes
            // per thread straight to global memory, 256 bytes apart, took 5700 clocks per item and held up the
            // loads of the next item behind them.)
            constexpr int kColsPerThread = D / 2;
            const uint32_t t_dv = tmem_addr(tmem_base, lane_base, Cfg::kColdV + half * kColsPerThread);
            const uint32_t t_dk = tmem_addr(tmem_base, lane_base, Cfg::kColdK + half * kColsPerThread);
            ok = mbar_wait(&bars->dkv_full, w & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const int hh = kStrided ? bh % wl.H() : 0, bb = kStrided ? bh / wl.H() : 0;
            uint8_t* out_row = smem + Cfg::kOffdS + half * kHalfTileBytes + r * 128;
            const bool store_leader = (cwarp == 0 && lane == 0);
            // all compute warps together (bounded, like every wait here)
            auto all_warps = [&]() -> bool {
                __syncwarp();
                if (lane == 0) mbar_arrive(&bars->out_sync);
                const bool fine = mbar_wait(&bars->out_sync, n_sync & 1, abort_flag);
                ++n_sync;
                return fine;
            };
#pragma unroll
            for (int which = 0; which < 2 && ok; ++which) {
                uint32_t a[kColsPerThread];
                const uint32_t t_src = which ? t_dk : t_dv;
#pragma unroll
                for (int cb = 0; cb < kColsPerThread; cb += 32) tmem_ld_x32(t_src + cb, a + cb);
                tmem_wait_ld();
                if (which == 1) {  // both accumulators have left tensor memory
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bars->dkv_free);
                    // the buffer holds dV until the copy engine has read it
                    if (store_leader) bulk_wait_group_read<0>();
                    ok = all_warps();
                    if (!ok) break;
                }
                const float f = which ? scale : 1.0f;
#pragma unroll
                for (int ch = 0; ch < kColsPerThread / 8; ++ch)
                    *reinterpret_cast<uint4*>(out_row + ((ch ^ (r & 7)) << 4)) = make_uint4(
                        pack_bf16x2(__uint_as_float(a[8 * ch + 0]) * f, __uint_as_float(a[8 * ch + 1]) * f),
                        pack_bf16x2(__uint_as_float(a[8 * ch + 2]) * f, __uint_as_float(a[8 * ch + 3]) * f),
                        pack_bf16x2(__uint_as_float(a[8 * ch + 4]) * f, __uint_as_float(a[8 * ch + 5]) * f),
                        pack_bf16x2(__uint_as_float(a[8 * ch + 6]) * f, __uint_as_float(a[8 * ch + 7]) * f));
                fence_proxy_async_smem();
                ok = all_warps();
                if (!ok) break;
                if (store_leader) {
                    const CUtensorMap* tm = which ? tmdK : tmdV;
                    const int order = which ? (wl.orders() >> 16) & 15 : (wl.orders() >> 20) & 15;
                    tma_store_tile<kStrided>(tm, smem + Cfg::kOffdS, order, 0, kt * kBlockK, hh, bb, bh);
                    tma_store_tile<kStrided>(tm, smem + Cfg::kOffdS + kHalfTileBytes, order, kBoxCols, kt * kBlockK, hh, bb, bh);
                    bulk_commit_group();
                }
            }
            if (!ok) break;
            // the next item's dS phase writes this buffer: the copy engine must have read dK
            if (store_leader) bulk_wait_group_read<0>();
            ok = all_warps();
            if (!ok) break;
        }
        ++w;
    }
    // Also when giving up: the stores of dV and dK must be complete before the kernel ends.
    if (!Cfg::kBulkdQ && cwarp == 0 && lane == 0) bulk_wait_group<0>();
}

// dQ warps at D=64.  One thread per row.  Per query tile they move the partial dQ tile from TMEM into
// a swizzled shared-memory staging buffer, and a leader thread sends it to the fp32 accumulator with
// two TMA reduce-add operations.  At the end of a work item the same warps pull dV and dK out of
// TMEM, convert them and send them out through the same buffer with two TMA stores, so the compute
// warps move on to the next item at once.  Nothing waits for a reduction or a store to complete
// except the end of the kernel; before the staging buffer is refilled, the leader checks that the copy
// engine has read it.
template <bool kStrided>
__device__ __forceinline__ void bwd_dq_tma(uint8_t* smem, BwdBars* bars, uint32_t tmem_base, const CUtensorMap* tmAcc,
                                           const CUtensorMap* tmdK, const CUtensorMap* tmdV, float scale,
                                           const WorkList& wl, int qwarp, int lane) {
    constexpr int D = 64;
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (qwarp & 3);
    const int r = lane_base + lane;  // local row: query row for dQ, key row for dV/dK
    const bool leader = (qwarp == 0 && lane == 0);
    const uint32_t t_dq = tmem_addr(tmem_base, lane_base, Cfg::kColdQ);
    const uint32_t t_dv = tmem_addr(tmem_base, lane_base, Cfg::kColdV);
    const uint32_t t_dk = tmem_addr(tmem_base, lane_base, Cfg::kColdK);
    uint8_t* stage = smem + Cfg::kOffStage;
    uint8_t* row0 = stage + r * 128;                   // this thread's row in box 0
    uint8_t* row1 = stage + kHalfTileBytes + r * 128;  // and in box 1
    const int sw = r & 7;
    bool ok = true;
    int w = 0, g = 0, u = 0;  // items, query tiles, uses of the staging buffer so far

    // Hands the filled staging buffer to the leader, who issues the copies of `kind`
    // (0: dQ reduce-add, 1: dV/dK store) at row `row` of head `bh`.
    auto flush = [&](int kind, int row, int bh) -> bool {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->stage_full);
        bool leader_ok = true;
        if (leader) {
            leader_ok = mbar_wait(&bars->stage_full, u & 1, abort_flag);
            if (leader_ok) {
                if (kind == 0) {
                    tma_reduce_add_3d(tmAcc, stage, 0, row, bh);
                    tma_reduce_add_3d(tmAcc, stage + kHalfTileBytes, 32, row, bh);
                } else {
                    const int hh = kStrided ? bh % wl.H() : 0, bb = kStrided ? bh / wl.H() : 0;
                    tma_store_tile<kStrided>(tmdV, stage, (wl.orders() >> 20) & 15, 0, row, hh, bb, bh);
                    tma_store_tile<kStrided>(tmdK, stage + kHalfTileBytes, (wl.orders() >> 16) & 15, 0, row, hh, bb, bh);
                }
                bulk_commit_group();
            }
        }
        ++u;
        // Brings the leader back together with the rest of its warp before the next warp-wide TMEM
        // load, and makes a failed wait of the leader a failure of the whole warp.
        return __all_sync(0xffffffffu, leader_ok);
    };

    // Before the staging buffer is refilled: the leader waits until the copy engine has read the
    // previous contents.  This comes after the TMEM read-out of the new tile, so the tensor core is
    // never held up by a copy that is still draining.
    auto stage_reusable = [&]() -> bool {
        if (u == 0) return true;
        if (leader) {
            bulk_wait_group_read<0>();
            mbar_arrive(&bars->stage_free);
        }
        __syncwarp();
        return mbar_wait(&bars->stage_free, (u - 1) & 1, abort_flag);
    };

    for (WorkCursor cur; !wl.done(cur) && ok; wl.advance(cur)) {
        int kt, bh, i0, n_it;
        if (!wl.get(cur, &kt, &bh, &i0, &n_it)) continue;
        for (int it = 0; it < n_it && !wl.no_dq(); ++it, ++g) {
            ok = mbar_wait(&bars->dq_full, g & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            // The staging buffer first (its previous contents were handed to the copy engine a whole tile ago),
            // then the tile leaves TMEM 32 columns = one box at a time, which keeps the register count down.
            ok = stage_reusable();
            if (!ok) break;
#pragma unroll
            for (int hb = 0; hb < 2; ++hb) {
                uint32_t a[32];
                tmem_ld_x32(t_dq + 32 * hb, a);
                tmem_wait_ld();
                uint8_t* rowp = hb ? row1 : row0;
                // fp32 [128 rows x 32 columns] per box: eight 16-byte chunks per row, 128-byte swizzle
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    *reinterpret_cast<uint4*>(rowp + ((ch ^ sw) << 4)) =
                        make_uint4(a[ch * 4], a[ch * 4 + 1], a[ch * 4 + 2], a[ch * 4 + 3]);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->dq_free);
            ok = flush(0, (i0 + it) * kBlockQ, bh);
            if (!ok) break;
        }
        if (!ok) break;
        // ---- end of the item: dV and dK rows of this key tile, bf16 [128 rows x 64 columns] per box
        ok = mbar_wait(&bars->dkv_full, w & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        ok = stage_reusable();
        if (!ok) break;
#pragma unroll
        for (int cb = 0; cb < 64; cb += 32) {  // 32 accumulator columns at a time keeps the register count down
            uint32_t a[32];
            tmem_ld_x32(t_dv + cb, a);
            tmem_wait_ld();
#pragma unroll
            for (int ch = 0; ch < 4; ++ch)  // 8 bf16 = 16 bytes per chunk
                *reinterpret_cast<uint4*>(row0 + (((cb / 8 + ch) ^ sw) << 4)) =
                    make_uint4(pack_bf16x2(__uint_as_float(a[8 * ch + 0]), __uint_as_float(a[8 * ch + 1])),
                               pack_bf16x2(__uint_as_float(a[8 * ch + 2]), __uint_as_float(a[8 * ch + 3])),
                               pack_bf16x2(__uint_as_float(a[8 * ch + 4]), __uint_as_float(a[8 * ch + 5])),
                               pack_bf16x2(__uint_as_float(a[8 * ch + 6]), __uint_as_float(a[8 * ch + 7])));
            tmem_ld_x32(t_dk + cb, a);
            tmem_wait_ld();
#pragma unroll
            for (int ch = 0; ch < 4; ++ch)
                *reinterpret_cast<uint4*>(row1 + (((cb / 8 + ch) ^ sw) << 4)) = make_uint4(
                    pack_bf16x2(__uint_as_float(a[8 * ch + 0]) * scale, __uint_as_float(a[8 * ch + 1]) * scale),
                    pack_bf16x2(__uint_as_float(a[8 * ch + 2]) * scale, __uint_as_float(a[8 * ch + 3]) * scale),
                    pack_bf16x2(__uint_as_float(a[8 * ch + 4]) * scale, __uint_as_float(a[8 * ch + 5]) * scale),
                    pack_bf16x2(__uint_as_float(a[8 * ch + 6]) * scale, __uint_as_float(a[8 * ch + 7]) * scale));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->dkv_free);
        ok = flush(1, kt * kBlockK, bh);
        ++w;
    }
    // Also when giving up: nothing of this thread may stay in flight, and the accumulator, dK and dV
    // must be complete before the kernel ends.
    if (leader) bulk_wait_group<0>();
}

// dQ warps at D=128.  One thread per query row; the partial dQ tile is 128 fp32 columns, i.e. four
// boxes of the accumulator's tensor map, and the staging buffer holds two.  The dQ columns are the dP^T
// columns of the next tile, so how soon they are handed back sets the period of a tile: the first 64
// columns go straight into the two halves of the staging buffer, the other 64 are loaded into the same
// registers, and the columns are released before any copy is issued.  A reduction runs at about 25 bytes
// per clock and SM however it is issued (TMA or red.global, measured), 2600 clocks for the 64 KB of a tile
// against 2600 clocks of tensor work, so the copy engine must never idle: every box is a bulk group of its
// own, boxes 0 and 1 are issued together, box 2 goes into the first half as soon as box 0 has been read
// (box 1 still being read), box 3 into the second half once box 1 has been.
__device__ __forceinline__ void bwd_dq_tma_wide(uint8_t* smem, BwdBars* bars, uint32_t tmem_base,
                                                const CUtensorMap* tmAcc, const WorkList& wl, int qwarp, int lane) {
    constexpr int D = 128;
    using Cfg = BwdCfg<D>;
    volatile int* abort_flag = &bars->abort_flag;
    const uint32_t lane_base = 32u * (qwarp & 3);
    const int r = lane_base + lane;  // local query row
    const bool leader = (qwarp == 0 && lane == 0);
    const uint32_t t_dq = tmem_addr(tmem_base, lane_base, Cfg::kColdQ);
    uint8_t* stage = smem + Cfg::kOffStage;
    uint8_t* row_ptr = stage + r * 128;
    const int sw = r & 7;
    bool ok = true;
    int g = 0, nf = 0, nr = 0;  // query tiles; uses of stage_full and of stage_free so far

    // 32 columns of this thread's row into half hb of the staging buffer (one box).
    auto fill = [&](const uint32_t* a, int hb) {
#pragma unroll
        for (int ch = 0; ch < 8; ++ch)
            *reinterpret_cast<uint4*>(row_ptr + hb * kHalfTileBytes + ((ch ^ sw) << 4)) =
                make_uint4(a[ch * 4], a[ch * 4 + 1], a[ch * 4 + 2], a[ch * 4 + 3]);
    };
    // Hands filled boxes to the leader, who adds them into the accumulator: half `first` at column `col`,
    // and with n = 2 the other half at col + 32; one bulk group per box.
    auto send = [&](int first, int n, int col, int row, int bh) -> bool {
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->stage_full);
        bool leader_ok = true;
        if (leader) {
            leader_ok = mbar_wait(&bars->stage_full, nf & 1, abort_flag);
            if (leader_ok) {
                for (int k = 0; k < n; ++k) {
                    tma_reduce_add_3d(tmAcc, stage + (first + k) * kHalfTileBytes, col + 32 * k, row, bh);
                    bulk_commit_group();
                }
            }
        }
        ++nf;
        return __all_sync(0xffffffffu, leader_ok);
    };
    // Before a half of the staging buffer is refilled the copy engine must have read what was sent from it:
    // all groups (kPending = 0) or all but the latest one (kPending = 1).
    auto reusable = [&](auto pending) -> bool {
        if (leader) {
            bulk_wait_group_read<decltype(pending)::value>();
            mbar_arrive(&bars->stage_free);
        }
        __syncwarp();
        const bool fine = mbar_wait(&bars->stage_free, nr & 1, abort_flag);
        ++nr;
        return __all_sync(0xffffffffu, fine);  // also brings the warp together before its next TMEM instruction
    };

    for (WorkCursor cur; !wl.done(cur) && ok && !wl.no_dq(); wl.advance(cur)) {
        int kt, bh, i0, n_it;
        if (!wl.get(cur, &kt, &bh, &i0, &n_it)) continue;
        for (int it = 0; it < n_it && ok; ++it, ++g) {
            ok = mbar_wait(&bars->dq_full, g & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const int row = (i0 + it) * kBlockQ;
            uint32_t a[64];
            tmem_ld_x32(t_dq, a);
            tmem_ld_x32(t_dq + 32, a + 32);
            if (g > 0) ok = reusable(std::integral_constant<int, 0>{});  // boxes 2, 3 of the previous tile
            tmem_wait_ld();
            if (!ok) break;
            fill(a, 0);
            fill(a + 32, 1);
            tmem_ld_x32(t_dq + 64, a);
            tmem_ld_x32(t_dq + 96, a + 32);
            tmem_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->dq_free);  // the whole tile has left TMEM
            ok = send(0, 2, 0, row, bh);
            if (ok) ok = reusable(std::integral_constant<int, 1>{});  // box 0 read, box 1 may still be in flight
            if (!ok) break;
            fill(a, 0);
            ok = send(0, 1, 64, row, bh);
            if (ok) ok = reusable(std::integral_constant<int, 1>{});  // box 1 read
            if (!ok) break;
            fill(a + 32, 1);
            ok = send(1, 1, 96, row, bh);
        }
    }
    // Also when giving up: nothing of this thread may stay in flight, and the accumulator must be
    // complete before the kernel ends.
    if (leader) bulk_wait_group<0>();
}

template <int D, bool kCausal, bool kStrided>
__global__ void __launch_bounds__(BwdCfg<D>::kThreads, 1)
attn_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmdO,
                const __grid_constant__ CUtensorMap tmAcc, const __grid_constant__ CUtensorMap tmdK,
                const __grid_constant__ CUtensorMap tmdV, const float* __restrict__ LSE,
                const float* __restrict__ Delta, __nv_bfloat16* __restrict__ dK,
                __nv_bfloat16* __restrict__ dV, const TensorStrides sdk, const TensorStrides sdv, int T,
                const __grid_constant__ WorkArgs wa, float scale, int* __restrict__ dev_status) {
    using Cfg = BwdCfg<D>;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    if (Cfg::kAlignPad == 0 && smem != smem_raw) {
        // No room to realign: give up before anything is set up, but only once the predecessor in the stream
        // has completed (the status word is global memory, and this grid must not finish ahead of it).
        griddep_wait();
        if (threadIdx.x == 0) atomicExch(dev_status, kDevTimeout);
        return;
    }
    BwdBars* bars = reinterpret_cast<BwdBars*>(smem + Cfg::kOffBar);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WorkList wl{wa, kCausal};

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bars->kv_full[s], 1);
            mbar_init(&bars->kv_empty[s], 1);
            mbar_init(&bars->q_full[s], 1);
            mbar_init(&bars->q_empty[s], 1);
            if (s == 0) {
                mbar_init(&bars->q_full[2], 1);
                mbar_init(&bars->q_empty[2], 1);
            }
            mbar_init(&bars->do_full[s], 1);
            mbar_init(&bars->do_empty[s], 1);
            mbar_init(&bars->row_full[s], 2);
            mbar_init(&bars->row_empty[s], Cfg::kComputeWarps);
        }
        mbar_init(&bars->s_full, 1);
        mbar_init(&bars->dp_full, 1);
        mbar_init(&bars->p_ready, Cfg::kComputeWarps);
        mbar_init(&bars->ds_ready, Cfg::kComputeWarps);
        mbar_init(&bars->dq_full, 1);
        mbar_init(&bars->dq_free, 4);
        mbar_init(&bars->stage_full, 4);
        mbar_init(&bars->stage_free, 1);
        mbar_init(&bars->dkv_full, 1);
        mbar_init(&bars->dkv_free, Cfg::kBulkdQ ? 4 : Cfg::kComputeWarps);
        mbar_init(&bars->drain, 1);
        mbar_init(&bars->out_sync, Cfg::kComputeWarps);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmQ);
        tma_prefetch_desc(&tmK);
        tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmdO);
        tma_prefetch_desc(&tmAcc);
        tma_prefetch_desc(&tmdK);
        tma_prefetch_desc(&tmdV);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, kBwdTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    griddep_launch_dependents();
    if (warp == 0 && lane == 0) {  // the first item's K, V and first Q, dO tiles on their way into L2 meanwhile
        int kt, bh, i0, n_it;
        if (wl.get(WorkCursor{}, &kt, &bh, &i0, &n_it)) {
            const int head = kStrided ? bh % wl.H() : 0, batch = kStrided ? bh / wl.H() : 0;
#pragma unroll
            for (int h = 0; h < Cfg::kHalves; ++h) {
                tma_prefetch_tile<kStrided>(&tmK, (wl.orders() >> 4) & 15, h * kBoxCols, kt * kBlockK, head, batch, bh);
                tma_prefetch_tile<kStrided>(&tmQ, wl.orders() & 15, h * kBoxCols, i0 * kBlockQ, head, batch, bh);
                tma_prefetch_tile<kStrided>(&tmV, (wl.orders() >> 8) & 15, h * kBoxCols, kt * kBlockK, head, batch, bh);
                tma_prefetch_tile<kStrided>(&tmdO, (wl.orders() >> 12) & 15, h * kBoxCols, i0 * kBlockQ, head, batch, bh);
            }
        }
    }
    griddep_wait();  // everything above overlaps the previous kernel of the stream

    if (warp == 0) {
        if (lane == 0) bwd_producer<D, kStrided>(&tmQ, &tmK, &tmV, &tmdO, smem, bars, wl);
    } else if (warp == 1) {
        bwd_mma<D>(smem, bars, tmem_base, wl);
    } else if (warp < 4) {
        bwd_rows(bars, reinterpret_cast<float*>(smem + Cfg::kOffRow), LSE, Delta, T, wl, (warp - 2) * 32 + lane);
    } else if (warp < 4 + Cfg::kComputeWarps) {
        bwd_compute<D, kCausal, kStrided>(smem, bars, tmem_base, &tmdK, &tmdV, T, scale, wl, warp - 4, lane);
    } else {
        if constexpr (Cfg::kBulkdQ)
            bwd_dq_tma<kStrided>(smem, bars, tmem_base, &tmAcc, &tmdK, &tmdV, scale, wl, warp - 4 - Cfg::kComputeWarps, lane);
        else
            bwd_dq_tma_wide(smem, bars, tmem_base, &tmAcc, wl, warp - 4 - Cfg::kComputeWarps, lane);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kBwdTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

template <int D, bool kCausal>
cudaError_t launch_one(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                       const CUtensorMap& tmdO, const CUtensorMap& tmAcc, const CUtensorMap& tmdK,
                       const CUtensorMap& tmdV, bool strided, uint32_t orders, bool no_dq, const float* LSE,
                       const float* Delta, __nv_bfloat16* dK, __nv_bfloat16* dV, const TensorStrides& sdk,
                       const TensorStrides& sdv, const AttnShape& s, int num_sms, int* dev_status, cudaStream_t stream) {
    static_assert(kBlockK == 128 && kBlockQ == 128, "the work plan counts 128-row tiles");
    const int BH = s.B * s.H;
    int n_tiles = 0, n_ctas = 0;
    const WorkPlan plan = bwd_work_plan(BH, s.T, D, kCausal, num_sms, &n_tiles, &n_ctas);
    const dim3 grid(static_cast<unsigned>(n_ctas));  // one persistent CTA per SM
    const WorkArgs wa{BH, n_tiles, s.H, orders, no_dq ? 1 : 0, plan};
    if (strided)
        return launch_overlapped(attn_bwd_kernel<D, kCausal, true>, grid, dim3(BwdCfg<D>::kThreads), BwdCfg<D>::kSmemBytes,
                                 stream, tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, LSE, Delta, dK, dV, sdk, sdv, s.T, wa,
                                 s.scale, dev_status);
    return launch_overlapped(attn_bwd_kernel<D, kCausal, false>, grid, dim3(BwdCfg<D>::kThreads), BwdCfg<D>::kSmemBytes, stream,
                             tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, LSE, Delta, dK, dV, sdk, sdv, s.T, wa, s.scale,
                             dev_status);
}

template <int D, bool kCausal, bool kStrided>
cudaError_t configure_one() {
    return cudaFuncSetAttribute(attn_bwd_kernel<D, kCausal, kStrided>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                BwdCfg<D>::kSmemBytes);
}

}  // namespace

cudaError_t configure_attn_bwd() {
    const cudaError_t r[8] = {configure_one<64, true, false>(),  configure_one<64, false, false>(),
                              configure_one<128, true, false>(), configure_one<128, false, false>(),
                              configure_one<64, true, true>(),   configure_one<64, false, true>(),
                              configure_one<128, true, true>(),  configure_one<128, false, true>()};
    for (cudaError_t e : r)
        if (e != cudaSuccess) return e;
    return cudaSuccess;
}

cudaError_t launch_attn_bwd(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                            const CUtensorMap& tmdO, const CUtensorMap& tmAcc, const CUtensorMap& tmdK,
                            const CUtensorMap& tmdV, bool strided, uint32_t orders, bool no_dq, const float* LSE,
                            const float* Delta, __nv_bfloat16* dK, __nv_bfloat16* dV, const TensorStrides& sdk,
                            const TensorStrides& sdv, const AttnShape& s, int num_sms, int* dev_status,
                            cudaStream_t stream) {
    if (s.D == 64) {
        return s.causal ? launch_one<64, true>(tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, strided, orders, no_dq, LSE, Delta, dK, dV, sdk, sdv, s, num_sms, dev_status, stream)
                        : launch_one<64, false>(tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, strided, orders, no_dq, LSE, Delta, dK, dV, sdk, sdv, s, num_sms, dev_status, stream);
    }
    return s.causal ? launch_one<128, true>(tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, strided, orders, no_dq, LSE, Delta, dK, dV, sdk, sdv, s, num_sms, dev_status, stream)
                    : launch_one<128, false>(tmQ, tmK, tmV, tmdO, tmAcc, tmdK, tmdV, strided, orders, no_dq, LSE, Delta, dK, dV, sdk, sdv, s, num_sms, dev_status, stream);
}

}  // namespace nova
