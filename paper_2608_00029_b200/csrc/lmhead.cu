// Fused language-model loss head for sm_100a (paper Section 4.1, case study "Fusing a Reduction into a
// Contraction Epilogue"; Section 6.1 "Fused Loss Head"): logits = X W^T by one tcgen05 contraction whose
// epilogue, while the accumulator tile is still in tensor memory, reduces it along the vocabulary axis to one
// partial (max, sum of exponentials) pair per row and per 128 vocabulary entries, writes the logits as bf16
// and picks out each row's target logit; a small second kernel merges the partial pairs with the rescaling
// rule (a sum is multiplied by the exponential of the difference of the maxima before it is added) into the
// row's log-sum-exp and cross-entropy.  The logits are never read back.
//
// Main kernel, persistent, one CTA per SM, 320 threads.  An output tile is 128 rows x 256 vocabulary entries;
// tiles are dealt out with the row tile varying fastest, so the CTAs that run together share a W tile in L2.
//   warp 0     TMA producer: per 64-wide k block one X box [128 x 64] and one W box [256 x 64] into a
//              four-stage ring
//   warp 1     UMMA issuer: 4 instructions (M 128, N 256, K 16) per k block into one of two accumulator
//              buffers in tensor memory (2 x 256 columns), so the epilogue of a tile runs under the
//              contraction of the next
//   warps 2-9  epilogue: two threads per row, 128 columns each, read in chunks of 32: running maximum and
//              sum in base 2 (one rescale per chunk), bf16 logits to global memory, the partial pair to the
//              workspace, the target's logit if it lies in the thread's columns
#include <cmath>

#include "../../include/nova_lmhead.h"
#include "kernels.h"
#include "ptx.cuh"

namespace nova {
namespace {

constexpr int kThreads = 320;
constexpr int kEpiWarps = 8;
constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kPart = 128;  // vocabulary entries per partial (max, sum) pair
constexpr int kStages = 4;
constexpr int kABytes = kBM * kBK * 2, kBBytes = kBN * kBK * 2;
constexpr int kStageBytes = kABytes + kBBytes;
// Staging of the bf16 logits on their way out: per epilogue warp one box of [32 rows x 64 columns], 128-byte
// swizzled like every other tile, sent with a TMA store (coalesced, clipped at the edges of the matrix).
constexpr int kOutBoxBytes = 32 * 128;
constexpr int kOffOut = kStages * kStageBytes;
constexpr int kOffBar = kOffOut + kEpiWarps * kOutBoxBytes;
constexpr int kSmemBytes = kOffBar + 256 + 1024;
static_assert(kSmemBytes <= 232448, "exceeds the shared memory of one CTA");
constexpr int kTmemCols = 512;

struct Bars {
    uint64_t full[kStages], empty[kStages];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
};

struct Tiles {
    int n_tiles, m_tiles, k_blocks;
    __device__ __forceinline__ void get(int t, int* m_tile, int* n_tile) const {
        *n_tile = t / m_tiles;
        *m_tile = t % m_tiles;
    }
};

__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(smem_u32(smem_dst)), "l"(m), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
                 : "memory");
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* m, const void* smem_src, int c0, int c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(m),
                 "r"(smem_u32(smem_src)), "r"(c0), "r"(c1)
                 : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
lmhead_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW,
              const __grid_constant__ CUtensorMap tmL, const int* __restrict__ targets, int store_logits,
              float2* __restrict__ partials,
              float* __restrict__ tgt_logit, int M, int N, int K, int* __restrict__ dev_status) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Bars* bars = reinterpret_cast<Bars*>(smem + kOffBar);
    volatile int* abort_flag = &bars->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Tiles tl{((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN), (M + kBM - 1) / kBM, (K + kBK - 1) / kBK};

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars->acc_full[b], 1);
            mbar_init(&bars->acc_empty[b], kEpiWarps);
        }
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmW);
        if (store_logits) tma_prefetch_desc(&tmL);
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    griddep_launch_dependents();
    griddep_wait();

    if (warp == 0) {
        if (lane == 0) {
            // ---- producer
            int armed[kStages];
            for (int s = 0; s < kStages; ++s) armed[s] = -1;
            bool ok = true;
            int g = 0;  // k blocks loaded so far
            for (int t = blockIdx.x; t < tl.n_tiles && ok; t += gridDim.x) {
                int m_tile, n_tile;
                tl.get(t, &m_tile, &n_tile);
                for (int kb = 0; kb < tl.k_blocks; ++kb, ++g) {
                    const int s = g % kStages;
                    const uint32_t ph = (g / kStages) & 1;
                    ok = mbar_wait(&bars->empty[s], ph ^ 1, abort_flag);
                    if (!ok) break;
                    // rows past M or N and columns past K arrive as zeros and add nothing
                    mbar_expect_tx(&bars->full[s], kStageBytes);
                    armed[s] = ph;
                    tma_load_2d(smem + s * kStageBytes, &tmX, &bars->full[s], kb * kBK, m_tile * kBM);
                    tma_load_2d(smem + s * kStageBytes + kABytes, &tmW, &bars->full[s], kb * kBK, n_tile * kBN);
                }
            }
            if (!ok) {  // giving up: let the copies in flight land before the shared memory goes away
                int none = 0;
                for (int s = 0; s < kStages; ++s)
                    if (armed[s] >= 0) (void)mbar_wait(&bars->full[s], armed[s], &none);
            }
        }
    } else if (warp == 1) {
        // ---- UMMA issuer: the whole warp in uniform control flow, one elected lane issues
        constexpr uint32_t kIdesc = umma_idesc_bf16(kBM, kBN, 0, 0);
        const uint32_t hi = umma_desc_hi_sw128(1024);
        const bool el = elect_one();
        bool ok = true;
        int g = 0, it = 0;
        for (int t = blockIdx.x; t < tl.n_tiles && ok; t += gridDim.x, ++it) {
            const int ab = it & 1;
            // the epilogue warps must have read this buffer's previous tile out of tensor memory
            ok = mbar_wait(&bars->acc_empty[ab], ((it >> 1) & 1) ^ 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_acc = tmem_base + ab * kBN;
            for (int kb = 0; kb < tl.k_blocks; ++kb, ++g) {
                const int s = g % kStages;
                ok = mbar_wait(&bars->full[s], (g / kStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                if (el) {
                    const uint32_t a = umma_desc_lo(smem_u32(smem + s * kStageBytes), 16);
                    const uint32_t b = umma_desc_lo(smem_u32(smem + s * kStageBytes + kABytes), 16);
#pragma unroll
                    for (int k = 0; k < kBK / 16; ++k)  // 16 k elements = 32 bytes further along the swizzled rows
                        umma_ss(t_acc, umma_desc_join(a + 2 * k, hi), umma_desc_join(b + 2 * k, hi), kIdesc,
                                (kb > 0 || k > 0) ? 1u : 0u);
                    tc_commit(&bars->empty[s]);
                    if (kb == tl.k_blocks - 1) tc_commit(&bars->acc_full[ab]);
                }
                __syncwarp();
            }
        }
        if (!ok) {
            int none = 0;
            if (el) tc_commit(&bars->drain);
            __syncwarp();
            (void)mbar_wait(&bars->drain, 0, &none);
        }
    } else {
        // ---- epilogue: a warp may only touch the TMEM lanes 32 * (warp id mod 4) .. +31
        const uint32_t lane_base = 32u * (warp & 3);
        const int half = (warp - 2) >> 2;
        const int row_local = lane_base + lane;
        bool ok = true;
        int it = 0;
        int it_stores = 0;  // logits boxes this warp has sent so far
        for (int t = blockIdx.x; t < tl.n_tiles && ok; t += gridDim.x, ++it) {
            int m_tile, n_tile;
            tl.get(t, &m_tile, &n_tile);
            const int ab = it & 1;
            const int row = m_tile * kBM + row_local;
            const int col0 = n_tile * kBN + half * kPart;  // first vocabulary entry of this thread
            const int tgt = (row < M) ? targets[row] : -1;
            ok = mbar_wait(&bars->acc_full[ab], (it >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_acc = tmem_addr(tmem_base, lane_base, ab * kBN + half * kPart);
            float m2 = -INFINITY;  // running maximum in base-2 units (logit * log2 e)
            float l = 0.f;         // running sum of 2^(z * log2 e - m2)
            uint8_t* out_row = smem + kOffOut + (warp - 2) * kOutBoxBytes + lane * 128;  // this thread's staging row
#pragma unroll 1
            for (int c = 0; c < kPart; c += 32) {
                uint32_t z[32];
                __syncwarp();  // lanes may have parted ways over their rows and targets
                tmem_ld_x32(t_acc + c, z);
                tmem_wait_ld();
                const int valid = min(32, N - (col0 + c));  // vocabulary entries of this chunk that exist
                if (valid <= 0) continue;
                if (tgt >= col0 + c && tgt < col0 + c + 32 && row < M) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (tgt == col0 + c + i) tgt_logit[row] = __uint_as_float(z[i]);
                }
                if (store_logits) {
                    // 32 logits = 64 bytes = four 16-byte chunks of this thread's 128-byte staging row; the box is
                    // sent after every second chunk of 32 (64 columns) and must have been read before it is refilled
                    if ((c & 32) == 0 && it_stores > 0) {
                        if (lane == 0) bulk_wait_group_read<0>();
                        __syncwarp();
                    }
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(z[8 * x + 0]), __uint_as_float(z[8 * x + 1]));
                        v.y = pack_bf16x2(__uint_as_float(z[8 * x + 2]), __uint_as_float(z[8 * x + 3]));
                        v.z = pack_bf16x2(__uint_as_float(z[8 * x + 4]), __uint_as_float(z[8 * x + 5]));
                        v.w = pack_bf16x2(__uint_as_float(z[8 * x + 6]), __uint_as_float(z[8 * x + 7]));
                        const int ch = (c & 32) / 8 + x;
                        *reinterpret_cast<uint4*>(out_row + ((ch ^ (lane & 7)) << 4)) = v;
                    }
                    if ((c & 32) != 0 || col0 + c + 32 >= N) {
                        // the box is as full as it gets: rows past M and columns past N are clipped by the copy
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            tma_store_2d(&tmL, smem + kOffOut + (warp - 2) * kOutBoxBytes, col0 + (c & ~63),
                                         m_tile * kBM + static_cast<int>(lane_base));
                            bulk_commit_group();
                        }
                        ++it_stores;
                    }
                }
                if (valid < 32) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i >= valid) z[i] = 0xff800000u;  // -inf: takes no part in the statistics
                }
                float mx0 = fmaxf(__uint_as_float(z[0]), __uint_as_float(z[1]));
                float mx1 = fmaxf(__uint_as_float(z[2]), __uint_as_float(z[3]));
#pragma unroll
                for (int i = 4; i < 32; i += 4) {
                    mx0 = fmax3(mx0, __uint_as_float(z[i + 0]), __uint_as_float(z[i + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(z[i + 2]), __uint_as_float(z[i + 3]));
                }
                const float m_new = fmaxf(m2, fmaxf(mx0, mx1) * kLog2e);  // finite: the chunk has a valid entry
                l *= ex2_approx(m2 - m_new);                               // 0 the first time (m2 = -inf)
                m2 = m_new;
                const uint64_t c2 = f32x2_pack(kLog2e, kLog2e);
                const uint64_t nm2 = f32x2_pack(-m_new, -m_new);
                uint64_t acc0 = 0, acc1 = 0;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    float x0, x1, x2, x3;
                    f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(z[i + 0]), __uint_as_float(z[i + 1])), c2, nm2), x0, x1);
                    f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(z[i + 2]), __uint_as_float(z[i + 3])), c2, nm2), x2, x3);
                    acc0 = f32x2_add(acc0, f32x2_pack(ex2_approx(x0), ex2_approx(x1)));
                    acc1 = f32x2_add(acc1, f32x2_pack(ex2_approx(x2), ex2_approx(x3)));
                }
                float a0, a1, a2, a3;
                f32x2_unpack(acc0, a0, a1);
                f32x2_unpack(acc1, a2, a3);
                l += (a0 + a1) + (a2 + a3);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->acc_empty[ab]);  // the buffer may receive the tile after next
            // partial pair of this row for vocabulary entries [col0, col0 + 128): maximum in natural units
            if (row < M && col0 < N)
                partials[static_cast<size_t>(col0 / kPart) * M + row] = make_float2(m2 * kLn2, l);
        }
        if (lane == 0) bulk_wait_group<0>();  // the logits must be complete before the kernel ends
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

// ------------------------------------------------------------------------------------------------------------
// The same kernel for a pair of CTAs (a cluster of two SMs, tcgen05 cta_group::2).  The single-CTA kernel above
// is bound by the path from L2 into shared memory: every 64-wide k block brings 16 KB of X and 32 KB of W per
// 4.2 MFLOP.  Here two CTAs share a 256-row by 256-entry tile: each holds its own 128 rows of X and one half
// (128 vocabulary entries) of the W tile, and one instruction of the leader CTA (rank 0) multiplies both halves
// of both (M = 256, N = 256, K = 16); the accumulator rows of a CTA land in its own tensor memory.  32 KB
// instead of 48 KB per k block and SM.
//   warp 0     producer, as above, with a six-stage ring of (X [128 x 64], W half [128 x 64])
//   warp 1     leader only: UMMA issuer.  It needs a stage to have landed in both CTAs: the copies of both
//              CTAs count their bytes on the leader's `full` barrier (cp.async.bulk.tensor with cta_group::2 may
//              name a barrier of the peer).  One commit signals the `empty` (and `acc_full`) barriers of both.
//   warps 2-9  epilogue on the CTA's own 128 rows, as above; the peer's warps release an accumulator buffer by
//              arriving on the leader's barrier
// Every CTA fetches what it needs itself: no copy is shared between the two.
constexpr int kPairStages = 6;
constexpr int kPairWBytes = (kBN / 2) * kBK * 2;
constexpr int kPairStageBytes = kABytes + kPairWBytes;
constexpr int kPairOffOut = kPairStages * kPairStageBytes;
constexpr int kPairOffBar = kPairOffOut + kEpiWarps * kOutBoxBytes;
constexpr int kPairSmemBytes = kPairOffBar + 256 + 1024;
static_assert(kPairSmemBytes <= 232448, "exceeds the shared memory of one CTA");

struct PairBars {
    uint64_t full[kPairStages], empty[kPairStages];
    uint64_t acc_full[2], acc_empty[2];
    uint64_t drain;
    uint32_t tmem_base;
    int abort_flag;
};
static_assert(sizeof(PairBars) <= 256, "barrier block");

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Address, in the cluster's shared window, of the same location in the shared memory of CTA `rank`.
__device__ __forceinline__ uint32_t cluster_map(const void* local, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(local)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Bounded wait with cluster-scope acquire (the arrivals may come from the peer CTA).
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok)
            : "r"(smem_u32(bar)), "r"(parity)
            : "memory");
        if (ok) return true;
        if (*abort_flag != 0) return false;
        if (clock64() - t0 > kWaitLimitCycles) {
            *abort_flag = 1;
            return false;
        }
    }
}
// 2-D tiled load into this CTA's shared memory whose bytes are counted on a barrier given by its address in
// the cluster's shared window (the leader's, for both CTAs of a pair).  The data go to this CTA only.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* m, uint32_t bar_cluster_addr, int c0,
                                                 int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(m), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D (+)= A B over the CTA pair; issued by one thread of the leader CTA.
__device__ __forceinline__ void umma_ss_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// One arrival on the barrier at this shared-memory offset in both CTAs of the pair, once every tcgen05
// operation issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(static_cast<uint16_t>(3))
                 : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
lmhead_pair_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmWh,
                   const __grid_constant__ CUtensorMap tmL, const int* __restrict__ targets, int store_logits,
                   float2* __restrict__ partials, float* __restrict__ tgt_logit, int M, int N, int K,
                   int* __restrict__ dev_status) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    PairBars* bars = reinterpret_cast<PairBars*>(smem + kPairOffBar);
    volatile int* abort_flag = &bars->abort_flag;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
    const int m_pairs = ((M + kBM - 1) / kBM + 1) / 2;
    const int n_tile_pairs = m_pairs * ((N + kBN - 1) / kBN);
    const int k_blocks = (K + kBK - 1) / kBK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&bars->acc_full[b], 1);
            mbar_init(&bars->acc_empty[b], 2 * kEpiWarps);  // the leader's: the epilogue warps of both CTAs
        }
        mbar_init(&bars->drain, 1);
        bars->abort_flag = 0;
        fence_mbar_init();
        tma_prefetch_desc(&tmX);
        tma_prefetch_desc(&tmWh);
        if (store_logits) tma_prefetch_desc(&tmL);
    }
    if (warp == 1) {
        tmem_alloc_pair(&bars->tmem_base, kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // the peer's barriers exist before anything is sent to them
    tc_fence_after();
    const uint32_t tmem_base = bars->tmem_base;
    griddep_launch_dependents();
    griddep_wait();

    if (warp == 0) {
        if (lane == 0) {
            // ---- producer: this CTA's rows of X and its half of the W tile; the leader's barrier counts the
            // bytes of both CTAs (the leader announces them)
            int armed[kPairStages];
            uint32_t full_leader[kPairStages];
            for (int s = 0; s < kPairStages; ++s) {
                armed[s] = -1;
                full_leader[s] = cluster_map(&bars->full[s], 0);
            }
            bool ok = true;
            int g = 0;
            for (int tp = pair; tp < n_tile_pairs && ok; tp += n_pairs) {
                const int n_tile = tp / m_pairs, m_tile = 2 * (tp % m_pairs) + static_cast<int>(rank);
                for (int kb = 0; kb < k_blocks; ++kb, ++g) {
                    const int s = g % kPairStages;
                    const uint32_t ph = (g / kPairStages) & 1;
                    ok = mbar_wait_cluster(&bars->empty[s], ph ^ 1, abort_flag);
                    if (!ok) break;
                    if (leader) {
                        mbar_expect_tx(&bars->full[s], 2 * kPairStageBytes);
                        armed[s] = ph;
                    }
                    tma_load_2d_pair(smem + s * kPairStageBytes, &tmX, full_leader[s], kb * kBK, m_tile * kBM);
                    tma_load_2d_pair(smem + s * kPairStageBytes + kABytes, &tmWh, full_leader[s], kb * kBK,
                                     n_tile * kBN + static_cast<int>(rank) * (kBN / 2));
                }
            }
            if (!ok) {  // giving up: let the copies in flight land before the shared memory goes away
                int none = 0;
                for (int s = 0; s < kPairStages; ++s)
                    if (armed[s] >= 0) (void)mbar_wait_cluster(&bars->full[s], armed[s], &none);
                if (!leader) __nanosleep(20000);  // the peer's copies are counted by the leader: give them time
            }
        }
    } else if (warp == 1) {
        const bool el = elect_one();
        bool ok = true;
        int g = 0, it = 0;
        if (leader) {
            // ---- UMMA issuer for the pair
            constexpr uint32_t kIdesc = umma_idesc_bf16(2 * kBM, kBN, 0, 0);
            const uint32_t hi = umma_desc_hi_sw128(1024);
            for (int tp = pair; tp < n_tile_pairs && ok; tp += n_pairs, ++it) {
                const int ab = it & 1;
                ok = mbar_wait_cluster(&bars->acc_empty[ab], ((it >> 1) & 1) ^ 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_acc = tmem_base + ab * kBN;
                for (int kb = 0; kb < k_blocks; ++kb, ++g) {
                    const int s = g % kPairStages;
                    const uint32_t ph = (g / kPairStages) & 1;
                    ok = mbar_wait_cluster(&bars->full[s], ph, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    if (el) {
                        const uint32_t a = umma_desc_lo(smem_u32(smem + s * kPairStageBytes), 16);
                        const uint32_t b = umma_desc_lo(smem_u32(smem + s * kPairStageBytes + kABytes), 16);
#pragma unroll
                        for (int k = 0; k < kBK / 16; ++k)
                            umma_ss_pair(t_acc, umma_desc_join(a + 2 * k, hi), umma_desc_join(b + 2 * k, hi), kIdesc,
                                         (kb > 0 || k > 0) ? 1u : 0u);
                        tc_commit_pair(&bars->empty[s]);
                        if (kb == k_blocks - 1) tc_commit_pair(&bars->acc_full[ab]);
                    }
                    __syncwarp();
                }
            }
            if (!ok) {  // giving up: what has been issued must have finished before the shared memory goes away
                int none = 0;
                if (el)
                    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                                     smem_u32(&bars->drain))
                                 : "memory");
                __syncwarp();
                (void)mbar_wait(&bars->drain, 0, &none);
            }
        }
    } else {
        // ---- epilogue on this CTA's 128 rows
        const uint32_t lane_base = 32u * (warp & 3);
        const int half = (warp - 2) >> 2;
        const int row_local = lane_base + lane;
        const uint32_t acc_empty_remote[2] = {cluster_map(&bars->acc_empty[0], 0), cluster_map(&bars->acc_empty[1], 0)};
        bool ok = true;
        int it = 0;
        int it_stores = 0;
        for (int tp = pair; tp < n_tile_pairs && ok; tp += n_pairs, ++it) {
            const int n_tile = tp / m_pairs, m_tile = 2 * (tp % m_pairs) + static_cast<int>(rank);
            const int ab = it & 1;
            const int row = m_tile * kBM + row_local;
            const int col0 = n_tile * kBN + half * kPart;
            const int tgt = (row < M) ? targets[row] : -1;
            const bool rows_exist = m_tile * kBM + static_cast<int>(lane_base) < M;  // of this warp's 32 rows, any
            ok = mbar_wait_cluster(&bars->acc_full[ab], (it >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_acc = tmem_addr(tmem_base, lane_base, ab * kBN + half * kPart);
            float m2 = -INFINITY;
            float l = 0.f;
            uint8_t* out_row = smem + kPairOffOut + (warp - 2) * kOutBoxBytes + lane * 128;
#pragma unroll 1
            for (int c = 0; c < kPart; c += 32) {
                uint32_t z[32];
                __syncwarp();
                tmem_ld_x32(t_acc + c, z);
                tmem_wait_ld();
                const int valid = min(32, N - (col0 + c));
                if (valid <= 0) continue;
                if (tgt >= col0 + c && tgt < col0 + c + 32 && row < M) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (tgt == col0 + c + i) tgt_logit[row] = __uint_as_float(z[i]);
                }
                if (store_logits && rows_exist) {
                    if ((c & 32) == 0 && it_stores > 0) {
                        if (lane == 0) bulk_wait_group_read<0>();
                        __syncwarp();
                    }
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        uint4 v;
                        v.x = pack_bf16x2(__uint_as_float(z[8 * x + 0]), __uint_as_float(z[8 * x + 1]));
                        v.y = pack_bf16x2(__uint_as_float(z[8 * x + 2]), __uint_as_float(z[8 * x + 3]));
                        v.z = pack_bf16x2(__uint_as_float(z[8 * x + 4]), __uint_as_float(z[8 * x + 5]));
                        v.w = pack_bf16x2(__uint_as_float(z[8 * x + 6]), __uint_as_float(z[8 * x + 7]));
                        const int ch = (c & 32) / 8 + x;
                        *reinterpret_cast<uint4*>(out_row + ((ch ^ (lane & 7)) << 4)) = v;
                    }
                    if ((c & 32) != 0 || col0 + c + 32 >= N) {
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            tma_store_2d(&tmL, smem + kPairOffOut + (warp - 2) * kOutBoxBytes, col0 + (c & ~63),
                                         m_tile * kBM + static_cast<int>(lane_base));
                            bulk_commit_group();
                        }
                        ++it_stores;
                    }
                }
                if (valid < 32) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i >= valid) z[i] = 0xff800000u;
                }
                float mx0 = fmaxf(__uint_as_float(z[0]), __uint_as_float(z[1]));
                float mx1 = fmaxf(__uint_as_float(z[2]), __uint_as_float(z[3]));
#pragma unroll
                for (int i = 4; i < 32; i += 4) {
                    mx0 = fmax3(mx0, __uint_as_float(z[i + 0]), __uint_as_float(z[i + 1]));
                    mx1 = fmax3(mx1, __uint_as_float(z[i + 2]), __uint_as_float(z[i + 3]));
                }
                const float m_new = fmaxf(m2, fmaxf(mx0, mx1) * kLog2e);
                l *= ex2_approx(m2 - m_new);
                m2 = m_new;
                const uint64_t c2 = f32x2_pack(kLog2e, kLog2e);
                const uint64_t nm2 = f32x2_pack(-m_new, -m_new);
                uint64_t acc0 = 0, acc1 = 0;
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    float x0, x1, x2, x3;
                    f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(z[i + 0]), __uint_as_float(z[i + 1])), c2, nm2), x0, x1);
                    f32x2_unpack(f32x2_fma(f32x2_pack(__uint_as_float(z[i + 2]), __uint_as_float(z[i + 3])), c2, nm2), x2, x3);
                    acc0 = f32x2_add(acc0, f32x2_pack(ex2_approx(x0), ex2_approx(x1)));
                    acc1 = f32x2_add(acc1, f32x2_pack(ex2_approx(x2), ex2_approx(x3)));
                }
                float a0, a1, a2, a3;
                f32x2_unpack(acc0, a0, a1);
                f32x2_unpack(acc1, a2, a3);
                l += (a0 + a1) + (a2 + a3);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {  // the buffer may receive the tile after next: tell the leader
                if (leader) mbar_arrive(&bars->acc_empty[ab]);
                else mbar_arrive_remote(acc_empty_remote[ab]);
            }
            if (row < M && col0 < N)
                partials[static_cast<size_t>(col0 / kPart) * M + row] = make_float2(m2 * kLn2, l);
        }
        if (lane == 0) bulk_wait_group<0>();
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();  // neither CTA's shared or tensor memory goes away while the other may still use it
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
    if (threadIdx.x == 0 && bars->abort_flag != 0) atomicExch(dev_status, kDevTimeout);
}

// Merge of the partial statistics of each row (paper Section 4.1: "a running maximum and a running sum do not
// combine via the same operation that accumulates them"): the pair with the smaller maximum has its sum
// multiplied by exp(smaller - larger) before the sums are added.  A block takes 32 rows; its 8 warps each walk
// every eighth partial of those rows (the partials of consecutive rows are adjacent, so a warp reads 256
// contiguous bytes per step, many steps in flight), and the 8 intermediate pairs of a row are merged by the
// same rule through shared memory.
constexpr int kMergeRows = 32, kMergeSlices = 8;

__device__ __forceinline__ void merge_pair(float& m, float& l, float m2, float l2) {
    if (l2 > 0.f) {
        if (m2 > m) {
            l = l * __expf(m - m2) + l2;  // exp(-inf) = 0 while nothing has been merged yet
            m = m2;
        } else {
            l += l2 * __expf(m2 - m);
        }
    }
}

__global__ void __launch_bounds__(kMergeRows * kMergeSlices)
lmhead_merge_kernel(const float2* __restrict__ partials, const float* __restrict__ tgt_logit,
                    const int* __restrict__ targets, float* __restrict__ lse, float* __restrict__ loss, int M, int N,
                    int n_part) {
    __shared__ float2 inter[kMergeSlices][kMergeRows];
    griddep_launch_dependents();
    griddep_wait();
    const int rl = threadIdx.x % kMergeRows, slice = threadIdx.x / kMergeRows;
    const int row = blockIdx.x * kMergeRows + rl;
    float m = -INFINITY, l = 0.f;
    if (row < M) {
#pragma unroll 8
        for (int p = slice; p < n_part; p += kMergeSlices) {
            const float2 q = partials[static_cast<size_t>(p) * M + row];
            merge_pair(m, l, q.x, q.y);
        }
    }
    inter[slice][rl] = make_float2(m, l);
    __syncthreads();
    if (slice == 0 && row < M) {
        for (int s = 1; s < kMergeSlices; ++s) merge_pair(m, l, inter[s][rl].x, inter[s][rl].y);
        const float v = m + logf(l);
        const int t = targets[row];
        lse[row] = v;
        loss[row] = (t >= 0 && t < N) ? v - tgt_logit[row] : 0.f;
    }
}

}  // namespace

size_t lmhead_workspace_bytes(int M, int N) {
    const size_t n_part = (static_cast<size_t>(N) + kPart - 1) / kPart;
    const size_t bytes = n_part * M * sizeof(float2) + static_cast<size_t>(M) * sizeof(float);
    return (bytes + 255) & ~size_t(255);
}

cudaError_t configure_lmhead() {
    cudaError_t e = cudaFuncSetAttribute(lmhead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(lmhead_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kPairSmemBytes);
}

cudaError_t launch_lmhead(const CUtensorMap& tmX, const CUtensorMap& tmW, const CUtensorMap& tmWh, const CUtensorMap& tmL,
                          bool store_logits, const int* targets, float* lse, float* loss, int M, int N, int K,
                          void* workspace, int num_sms, int* dev_status, cudaStream_t stream) {
    const int n_part = (N + kPart - 1) / kPart;
    float2* partials = static_cast<float2*>(workspace);
    float* tgt_logit = reinterpret_cast<float*>(partials + static_cast<size_t>(n_part) * M);
    const int m_tiles = (M + kBM - 1) / kBM;
    const long long n_tiles = static_cast<long long>(m_tiles) * ((N + kBN - 1) / kBN);
    cudaError_t e;
    if (m_tiles >= 2 && num_sms >= 2) {  // pairs of CTAs on 256-row tiles
        const long long tile_pairs = static_cast<long long>((m_tiles + 1) / 2) * ((N + kBN - 1) / kBN);
        const long long pairs = tile_pairs < num_sms / 2 ? tile_pairs : num_sms / 2;
        e = launch_overlapped(lmhead_pair_kernel, dim3(static_cast<unsigned>(2 * pairs)), dim3(kThreads), kPairSmemBytes,
                              stream, tmX, tmWh, tmL, targets, store_logits ? 1 : 0, partials, tgt_logit, M, N, K,
                              dev_status);
    } else {
        const dim3 grid(static_cast<unsigned>(n_tiles < num_sms ? n_tiles : num_sms));
        e = launch_overlapped(lmhead_kernel, grid, dim3(kThreads), kSmemBytes, stream, tmX, tmW, tmL, targets,
                              store_logits ? 1 : 0, partials, tgt_logit, M, N, K, dev_status);
    }
    if (e != cudaSuccess) return e;
    return launch_overlapped(lmhead_merge_kernel, dim3((M + kMergeRows - 1) / kMergeRows),
                             dim3(kMergeRows * kMergeSlices), 0, stream,
                             static_cast<const float2*>(partials), static_cast<const float*>(tgt_logit), targets, lse, loss,
                             M, N, n_part);
}

int lmhead_boxes(int* box_rows_x, int* box_rows_w) {
    *box_rows_x = kBM;
    *box_rows_w = kBN;
    return kBK;
}

}  // namespace nova
