// Work distribution of the backward kernel: which (key tile, head) items a CTA processes, in which order.
// Shared by the kernel (device) and by the launch code and the tests (host).
#pragma once
#include <cstdint>

namespace nova {

// This CTA's list of work items.  The heads are taken in chunks small enough for a chunk's fp32 dQ
// accumulator and its Q, K, V, dO to stay in L2 while the chunk is worked on: every key tile of a head adds
// into the same accumulator rows and reads the same Q and dO tiles, and with all heads in flight at once
// those lines were evicted between two uses (a TMA reduce-add that misses L2 runs at less than half the
// rate of one that hits).  Within a chunk the items are ordered by weight (key tile 0 of a causal problem
// sees every query tile, the last key tile only one) and dealt to the CTAs in zig-zag passes; a chunk is
// padded to whole passes, so that the heavy items of the next chunk start together on all CTAs (the
// padding costs the idle CTAs one item of the lightest class per chunk).
struct WorkPlan {
    int chunk;             // heads per chunk (the last chunk may have fewer)
    int n_chunks;
    int passes_per_chunk;  // of a full chunk
    int passes_last;       // of the last chunk
};
// Position in the list: chunk and pass within the chunk.  Stepping it costs no division.
struct WorkCursor {
    int ck = 0, lp = 0;
};
// What the list is computed from.  It is a kernel parameter, and the roles read its fields from the parameter
// space where they need them instead of carrying copies in registers through their inner loops (every thread of
// this kernel is at its register limit).
struct WorkArgs {
    int BH, n_tiles, H;
    uint32_t orders;  // coordinate orders of the Q, K, V, dO, dK, dV tensor maps, four bits each
    int no_dq;        // dK/dV half of the two-kernel backward: no dQ product, no accumulator traffic
    WorkPlan plan;
};
struct WorkList {
    const WorkArgs& a;
    bool causal;
    __host__ __device__ __forceinline__ int H() const { return a.H; }
    __host__ __device__ __forceinline__ uint32_t orders() const { return a.orders; }
    __host__ __device__ __forceinline__ bool no_dq() const { return a.no_dq != 0; }
    __host__ __device__ __forceinline__ bool done(const WorkCursor& c) const { return c.ck >= a.plan.n_chunks; }
    __host__ __device__ __forceinline__ void advance(WorkCursor& c) const {
        const int n = (c.ck == a.plan.n_chunks - 1) ? a.plan.passes_last : a.plan.passes_per_chunk;
        if (++c.lp >= n) {
            c.lp = 0;
            ++c.ck;
        }
    }
    // Item at the cursor: returns false if this CTA has none in that pass.
    __device__ __forceinline__ bool get(const WorkCursor& cur, int* kt, int* bh, int* i0, int* n_it) const {
        return get_for(cur, static_cast<int>(gridDim.x), static_cast<int>(blockIdx.x), kt, bh, i0, n_it);
    }
    // The same for CTA `cta` of `n_ctas` (also callable on the host, where the tests walk the lists).
    __host__ __device__ __forceinline__ bool get_for(const WorkCursor& cur, int n_ctas, int cta, int* kt, int* bh, int* i0,
                                                     int* n_it) const {
        const int BH = a.BH, n_tiles = a.n_tiles;
        const int h0 = cur.ck * a.plan.chunk;
        const int c = (BH - h0 < a.plan.chunk) ? BH - h0 : a.plan.chunk;
        // zig-zag within the chunk, and the other way round in every second chunk, so that what is left
        // uneven at the end of one chunk is evened out by the next
        const int idx = cur.lp * n_ctas + (((cur.lp ^ cur.ck) & 1) ? (n_ctas - 1 - cta) : cta);
        if (idx >= c * n_tiles) return false;
        *kt = idx / c;
        *bh = h0 + idx - *kt * c;
        *i0 = causal ? *kt : 0;  // raised lower bound of the query loop
        *n_it = n_tiles - *i0;
        return true;
    }
};

// Heads per chunk for a working set of about `budget` bytes, chosen among the nearby sizes for the least
// idle time in the padded last pass of a chunk.
inline WorkPlan make_work_plan(int BH, int n_tiles, long long T, int D, bool causal, int n_ctas, long long budget,
                               int min_passes) {
    const long long per_head = T * D * 12;  // fp32 accumulator + Q, K, V, dO
    long long cb = budget / per_head;
    const long long c_min = (static_cast<long long>(min_passes) * n_ctas + n_tiles - 1) / n_tiles;  // heads for min_passes passes
    if (cb < c_min) cb = c_min;
    if (cb < 1) cb = 1;
    int best = BH;
    if (cb * 3 / 2 < BH) {
        const int n_chunks = static_cast<int>((BH + cb - 1) / cb);
        const int even = (BH + n_chunks - 1) / n_chunks;
        double best_cost = 1e30;
        int lo = even / 2 > 1 ? even / 2 : 1;
        if (lo < c_min) lo = static_cast<int>(c_min < even ? c_min : even);
        const int hi = even + even / 4;
        for (int c = hi; c >= lo; --c) {
            const long long items = static_cast<long long>(c) * n_tiles;
            const long long passes = (items + n_ctas - 1) / n_ctas;
            const double idle = static_cast<double>(passes * n_ctas - items) * (causal ? 1.0 : n_tiles);
            const double work = static_cast<double>(items) * (causal ? (n_tiles + 1) * 0.5 : n_tiles);
            // a small penalty on chunks far from the budget on either side
            const double cost = idle / work + 0.02 * (c > even ? static_cast<double>(c - even) / even : static_cast<double>(even - c) / even);
            if (cost < best_cost) { best_cost = cost; best = c; }
        }
    }
    WorkPlan wp;
    wp.chunk = best;
    wp.n_chunks = (BH + best - 1) / best;
    wp.passes_per_chunk = static_cast<int>((static_cast<long long>(best) * n_tiles + n_ctas - 1) / n_ctas);
    const int last = BH - (wp.n_chunks - 1) * best;
    wp.passes_last = static_cast<int>((static_cast<long long>(last) * n_tiles + n_ctas - 1) / n_ctas);
    return wp;
}

// The plan the backward launch uses for a problem on a device of `num_sms` SMs: one persistent CTA per SM
// (fewer if there are fewer items).  Chunks of about 48 MB (accumulator and inputs of their heads) and of at
// least two passes: measured on B=16, H=32, T=1024, D=128, 704 -> 565 us against all heads in one list; 24 to
// 96 MB and two to four passes differ by a few percent either way.
inline WorkPlan bwd_work_plan(int BH, long long T, int D, bool causal, int num_sms, int* n_tiles_out, int* grid_out) {
    const int n_tiles = static_cast<int>((T + 127) / 128);
    const long long n_items = static_cast<long long>(n_tiles) * BH;
    const int grid = static_cast<int>(n_items < num_sms ? n_items : num_sms);
    *n_tiles_out = n_tiles;
    *grid_out = grid;
    return make_work_plan(BH, n_tiles, T, D, causal, grid, 48ll << 20, 2);
}

}  // namespace nova
