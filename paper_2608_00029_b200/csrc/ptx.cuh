// Thin inline-PTX wrappers for the sm_100a features the attention kernels use:
// mbarrier, TMA (cp.async.bulk.tensor; every copy targets this CTA only), tcgen05 (TMEM allocation,
// UMMA issue/commit, TMEM load/store) and the shared-memory / instruction descriptors of UMMA.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace nova {

// Device status word values (see nova_attn_poll_device_status).
constexpr int kDevOk = 0;
constexpr int kDevTimeout = 1;

// Upper bound of every spin-wait, in SM clock cycles (about a quarter of a second).  No legitimate
// wait in these kernels lasts longer than a few hundred microseconds.
constexpr long long kWaitLimitCycles = 1ll << 29;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ------------------------------------------------------------------ programmatic dependent launch
// Every kernel of the library is launched so that it may start while its predecessor in the stream
// is still draining: its set-up (barriers, TMEM, descriptor prefetch) then overlaps the predecessor's
// tail.  griddep_wait() blocks until the predecessor has completed and its writes are visible; nothing
// that reads or writes global memory may come before it.  griddep_launch_dependents() lets the
// successor be scheduled as soon as every CTA of this grid has issued it or exited.  Both are no-ops
// in a kernel launched the ordinary way.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// ------------------------------------------------------------------------------------------ mbarrier
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Non-blocking probe: true if the phase has completed, false at once if it has not (try_wait above may keep the
// thread suspended for a while before it answers false; this one never does).  For looking ahead without
// committing to a wait.
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// Same test, but the hardware may keep the thread suspended for up to `hint_ns` while the phase is
// incomplete (it resumes at once when the phase completes).  A suspended thread issues nothing, so
// waiting warps do not take issue slots from the warps that share their scheduler.
__device__ __forceinline__ bool mbar_try_wait_suspend(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}

// Bounded wait.  Returns false if the phase did not complete within `limit` cycles or if another
// thread of the CTA already gave up (*abort_flag != 0); the caller then leaves through the common
// exit path.  `abort_flag` lives in shared memory.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                          long long limit = kWaitLimitCycles) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 8; ++i)
            if (mbar_try_wait_suspend(bar, parity, 20000u)) return true;
        if (*abort_flag != 0) return false;
        if (clock64() - t0 > limit) {
            *abort_flag = 1;
            return false;
        }
    }
}

// ------------------------------------------------------------------ dynamic work distribution
// A persistent CTA that has finished its work item asks the hardware to cancel the launch of a CTA of the same
// grid that has not started yet and takes over that CTA's index (sm_100 cluster launch control).  The grid is
// launched with one CTA per work item; as many as fit start at once, the rest are handed out this way in
// launch order, so that no CTA idles while another still has items queued.  The request is asynchronous: the
// 16-byte answer lands in shared memory and completes 16 bytes on `bar`.  After a request has failed (nothing
// left to cancel) no further request may be made.
__device__ __forceinline__ void clc_try_cancel(void* smem_response16, uint64_t* bar) {
    asm volatile(
        "clusterlaunchcontrol.try_cancel.async.shared::cta.mbarrier::complete_tx::bytes.b128 [%0], [%1];"
        ::"r"(smem_u32(smem_response16)), "r"(smem_u32(bar))
        : "memory");
}
// Decodes an answer: the x index of the cancelled CTA, or -1 if nothing was cancelled.
__device__ __forceinline__ int clc_cancelled_cta(const void* smem_response16) {
    uint32_t ok, x;
    asm volatile(
        "{\n\t.reg .b128 r;\n\t.reg .pred p;\n\t"
        "ld.shared.b128 r, [%2];\n\t"
        "clusterlaunchcontrol.query_cancel.is_canceled.pred.b128 p, r;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "mov.u32 %1, 0;\n\t"
        "@p clusterlaunchcontrol.query_cancel.get_first_ctaid::x.b32.b128 %1, r;\n\t}"
        : "=r"(ok), "=r"(x)
        : "r"(smem_u32(smem_response16))
        : "memory");
    return ok ? static_cast<int>(x) : -1;
}

// The ring through which a CTA's producer thread tells the other roles which work item comes next: two
// entries in shared memory.  The producer publishes the number of the w-th item of this CTA (or -1: no more),
// each consumer warp (or single-thread role) takes it and frees the entry.  The producer gets the numbers
// from the hardware: its own CTA index first, then the indices of CTAs whose launch it cancels.
struct WorkRing {
    uint64_t full[2], empty[2], answer_bar;
    uint4 response;
    int item[2];

    __device__ __forceinline__ void init(int consumers) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], consumers);
        }
        mbar_init(&answer_bar, 1);
    }
    // ---- producer (one thread)
    __device__ __forceinline__ bool publish(int w, int it, volatile int* abort_flag, long long limit) {
        if (!mbar_wait(&empty[w & 1], ((w >> 1) & 1) ^ 1, abort_flag, limit)) return false;
        item[w & 1] = it;
        mbar_arrive(&full[w & 1]);
        return true;
    }
    // Asks for the item after the w-th; at most one request is outstanding, and none follows a failed one.
    __device__ __forceinline__ void request() {
        mbar_expect_tx(&answer_bar, 16);
        clc_try_cancel(&response, &answer_bar);
    }
    __device__ __forceinline__ bool answer(int w, int* next, volatile int* abort_flag, long long limit) {
        if (!mbar_wait(&answer_bar, w & 1, abort_flag, limit)) return false;
        *next = clc_cancelled_cta(&response);
        return true;
    }
    // ---- consumers: the w-th item, -1 when there are no more, -2 if the wait was given up
    __device__ __forceinline__ int take(int w, int lane, volatile int* abort_flag, long long limit) {  // a whole warp
        if (!mbar_wait(&full[w & 1], (w >> 1) & 1, abort_flag, limit)) return -2;
        const int it = *reinterpret_cast<volatile int*>(&item[w & 1]);
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[w & 1]);
        return it;
    }
    __device__ __forceinline__ int take_single(int w, volatile int* abort_flag, long long limit) {  // one thread
        if (!mbar_wait(&full[w & 1], (w >> 1) & 1, abort_flag, limit)) return -2;
        const int it = *reinterpret_cast<volatile int*>(&item[w & 1]);
        mbar_arrive(&empty[w & 1]);
        return it;
    }
    // Has the w-th item been published yet?  Non-blocking; the same answer in every lane of a converged warp.
    __device__ __forceinline__ bool published(int w) {
        return __all_sync(0xffffffffu, mbar_test(&full[w & 1], (w >> 1) & 1));
    }
};

// ------------------------------------------------------------------------------------------ TMA
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
// 3-D tiled load global -> shared (this CTA), completion counted in bytes on `bar`.
// c0 * sizeof(element) must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int c0,
                                            int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(m), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
// 3-D tiled reduce-add shared (this CTA) -> global through a tensor map: global += smem box.
// Completion is tracked by this thread's bulk async-groups.  Coordinates must be non-negative.
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* m, const void* smem_src, int c0, int c1, int c2) {
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(m),
                 "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}
// 3-D tiled store shared (this CTA) -> global through a tensor map; rows outside the tensor are
// clipped.  Completion is tracked by this thread's bulk async-groups.
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* m, const void* smem_src, int c0, int c1, int c2) {
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(m),
                 "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}
// Tile copies of the bf16 tensors Q, K, V, O, dO, dK, dV.  The kernels come in two builds.  Plain
// (kStrided = false): heads and batches merge into one dimension, the maps are 3-D [D, T, B*H] and the
// coordinate is (d, t, bh).  Strided: the maps are 4-D [D, x, y, z] with token, head and batch in order
// of increasing stride (so that slices of a fused [B,T,3,H,D] projection output can be read in place);
// `order` says which of the three sits where: 0: (t,h,b)  1: (h,t,b)  2: (t,b,h)  3: (b,t,h)  4: (h,b,t)
// 5: (b,h,t).
__device__ __forceinline__ void tma_order_coords(int order, int t, int h, int b, int& c1, int& c2, int& c3) {
    switch (order) {
        case 0: c1 = t; c2 = h; c3 = b; break;
        case 1: c1 = h; c2 = t; c3 = b; break;
        case 2: c1 = t; c2 = b; c3 = h; break;
        case 3: c1 = b; c2 = t; c3 = h; break;
        case 4: c1 = h; c2 = b; c3 = t; break;
        default: c1 = b; c2 = h; c3 = t; break;
    }
}
template <bool kStrided>
__device__ __forceinline__ void tma_load_tile(void* smem_dst, const CUtensorMap* m, uint64_t* bar, int order, int d,
                                              int t, int h, int b, int bh) {
    if constexpr (!kStrided) {
        tma_load_3d(smem_dst, m, bar, d, t, bh);
        return;
    }
    int c1, c2, c3;
    tma_order_coords(order, t, h, b, c1, c2, c3);
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(smem_dst)), "l"(m), "r"(smem_u32(bar)), "r"(d), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
// Asks for the box at the given coordinates to be brought into L2; nothing is written anywhere, so it
// may run ahead of griddep_wait().
template <bool kStrided>
__device__ __forceinline__ void tma_prefetch_tile(const CUtensorMap* m, int order, int d, int t, int h, int b, int bh) {
    if constexpr (!kStrided) {
        asm volatile("cp.async.bulk.prefetch.tensor.3d.L2.global.tile [%0, {%1, %2, %3}];" ::"l"(m), "r"(d), "r"(t),
                     "r"(bh)
                     : "memory");
        return;
    }
    int c1, c2, c3;
    tma_order_coords(order, t, h, b, c1, c2, c3);
    asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];" ::"l"(m), "r"(d), "r"(c1),
                 "r"(c2), "r"(c3)
                 : "memory");
}
template <bool kStrided>
__device__ __forceinline__ void tma_store_tile(const CUtensorMap* m, const void* smem_src, int order, int d, int t,
                                               int h, int b, int bh) {
    if constexpr (!kStrided) {
        tma_store_3d(m, smem_src, d, t, bh);
        return;
    }
    int c1, c2, c3;
    tma_order_coords(order, t, h, b, c1, c2, c3);
    asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%2, %3, %4, %5}], [%1];" ::"l"(m),
                 "r"(smem_u32(smem_src)), "r"(d), "r"(c1), "r"(c2), "r"(c3)
                 : "memory");
}
// Make generic-proxy writes to shared memory visible to the async proxy (TMA, UMMA operand reads).
__device__ __forceinline__ void fence_proxy_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ------------------------------------------------------------------------------------------ TMEM
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)),
                 "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// mbarrier arrive once every tcgen05 operation previously issued by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

// True in exactly one lane of a fully converged warp.  Roles whose work is issued by a single thread
// (UMMA, TMA) run with the whole warp in uniform control flow and guard only the issuing instructions
// with this, so that addresses and descriptors stay in uniform registers.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}

// D[tmem] (+)= A[smem] * B[smem]; `accumulate` == 0 overwrites D.
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem].
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Instruction descriptor of tcgen05.mma.kind::f16 with bf16 operands and an fp32 accumulator.
// a_mn / b_mn: 0 = operand is K-major in shared memory, 1 = MN-major.
__host__ __device__ constexpr uint32_t umma_idesc_bf16(int M, int N, int a_mn, int b_mn) {
    return (1u << 4)                       // D format: F32
           | (1u << 7)                     // A format: BF16
           | (1u << 10)                    // B format: BF16
           | (uint32_t(a_mn) << 15)        // A major
           | (uint32_t(b_mn) << 16)        // B major
           | (uint32_t(N >> 3) << 17)      // N / 8
           | (uint32_t(M >> 4) << 24);     // M / 16
}

// Shared-memory matrix descriptor, 128-byte swizzle (rows of 128 bytes, 8-row groups of 1024 bytes).
//   K-major operand : rows are M/N indices; `sbo_bytes` = distance between 8-row groups (1024);
//                     `lbo_bytes` unused by hardware for swizzled K-major layouts.
//   MN-major operand: rows are K indices; 64 MN elements (bf16) per row; `lbo_bytes` = distance
//                     between 64-element MN chunks, `sbo_bytes` = distance between 8-row K groups.
__device__ __forceinline__ uint64_t umma_smem_desc_sw128(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= uint64_t((smem_addr & 0x3FFFFu) >> 4);
    d |= uint64_t((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= uint64_t((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= uint64_t(1) << 46;   // descriptor version for sm_100
    d |= uint64_t(2) << 61;   // SWIZZLE_128B
    return d;
}

// The same descriptor split in two: the constant upper word and the lower word as a function of the
// address, so that a hot loop only adds a byte offset (>> 4) to a precomputed lower word.
__device__ __forceinline__ uint32_t umma_desc_hi_sw128(uint32_t sbo_bytes) {
    return ((sbo_bytes >> 4) & 0x3FFFu) | (1u << 14) | (2u << 29);
}
__device__ __forceinline__ uint32_t umma_desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
    return ((smem_addr & 0x3FFFFu) >> 4) | (((lbo_bytes >> 4) & 0x3FFFu) << 16);
}
__device__ __forceinline__ uint64_t umma_desc_join(uint32_t lo, uint32_t hi) {
    return (static_cast<uint64_t>(hi) << 32) | lo;
}

// TMEM address: lane in bits [31:16], column in bits [15:0].
__device__ __forceinline__ uint32_t tmem_addr(uint32_t base, uint32_t lane, uint32_t col) {
    return base + (lane << 16) + col;
}

// 32 lanes x 32 bits, N consecutive columns: thread `l` of the warp receives row (lane_base + l).
#define NOVA_R4(r, o) "=r"(r[o]), "=r"(r[o + 1]), "=r"(r[o + 2]), "=r"(r[o + 3])
#define NOVA_W4(r, o) "r"(r[o]), "r"(r[o + 1]), "r"(r[o + 2]), "r"(r[o + 3])

__device__ __forceinline__ void tmem_ld_x32(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : NOVA_R4(r, 0), NOVA_R4(r, 4), NOVA_R4(r, 8), NOVA_R4(r, 12), NOVA_R4(r, 16), NOVA_R4(r, 20),
          NOVA_R4(r, 24), NOVA_R4(r, 28)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_x16(uint32_t taddr, uint32_t* r) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : NOVA_R4(r, 0), NOVA_R4(r, 4), NOVA_R4(r, 8), NOVA_R4(r, 12)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_x8(uint32_t taddr, const uint32_t* r) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0, %1, %2, %3, %4, %5, %6, %7};" ::NOVA_W4(r, 0),
                 NOVA_W4(r, 4), "r"(taddr)
                 : "memory");
}
__device__ __forceinline__ void tmem_st_x32(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31};"
        ::NOVA_W4(r, 0), NOVA_W4(r, 4), NOVA_W4(r, 8), NOVA_W4(r, 12), NOVA_W4(r, 16), NOVA_W4(r, 20),
          NOVA_W4(r, 24), NOVA_W4(r, 28), "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st_x16(uint32_t taddr, const uint32_t* r) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15};"
        ::NOVA_W4(r, 0), NOVA_W4(r, 4), NOVA_W4(r, 8), NOVA_W4(r, 12), "r"(taddr)
        : "memory");
}

// ------------------------------------------------------------------------------------------ math
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Packed pairs of fp32 in one 64-bit register: sm_100 executes fma/add on both halves in one
// instruction, which halves the issue slots of the softmax arithmetic.
__device__ __forceinline__ uint64_t f32x2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f32x2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f32x2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t f32x2_add(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f32x2_mul(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// max of three in one instruction
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
// Two fp32 -> packed bf16x2 (round to nearest even); `lo` lands in the low 16 bits.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// The same packing on the integer pipe (two adds and a byte permute) instead of the conversion unit,
// which shares its issue port with exp2: rounds to nearest with ties away from zero, for finite inputs
// (a tie is one fp32 value in 65536, so the difference from round-to-nearest-even does not bias sums).
__device__ __forceinline__ uint32_t pack_bf16x2_int(float lo, float hi) {
    return __byte_perm(__float_as_uint(lo) + 0x8000u, __float_as_uint(hi) + 0x8000u, 0x7632);
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// At most N of this thread's bulk groups still pending (.read: only their shared-memory reads).
template <int N>
__device__ __forceinline__ void bulk_wait_group() {
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void named_barrier_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

}  // namespace nova
