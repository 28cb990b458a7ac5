// Work distribution of the backward kernel: which (key tile, head) items a CTA processes, in which order.
// Shared by the kernel (device) and by the launch code and the tests (host).
#pragma once
#include <cstdint>
#include <mutex>

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

inline WorkPlan work_plan_for_chunk(int BH, int n_tiles, int n_ctas, int chunk) {
    WorkPlan wp;
    wp.chunk = chunk;
    wp.n_chunks = (BH + chunk - 1) / chunk;
    wp.passes_per_chunk = static_cast<int>((static_cast<long long>(chunk) * n_tiles + n_ctas - 1) / n_ctas);
    const int last = BH - (wp.n_chunks - 1) * chunk;
    wp.passes_last = static_cast<int>((static_cast<long long>(last) * n_tiles + n_ctas - 1) / n_ctas);
    return wp;
}

// Largest load of a CTA over the mean load (in tiles) when the items are dealt out by `wp`.
inline double work_plan_imbalance(int BH, int n_tiles, bool causal, int n_ctas, const WorkPlan& wp) {
    const WorkArgs wa{BH, n_tiles, 1, 0u, 0, wp};
    const WorkList wl{wa, causal};
    long long total = 0, worst = 0;
    for (int cta = 0; cta < n_ctas; ++cta) {
        long long load = 0;
        for (WorkCursor cur; !wl.done(cur); wl.advance(cur)) {
            int kt, bh, i0, n_it;
            if (wl.get_for(cur, n_ctas, cta, &kt, &bh, &i0, &n_it)) load += n_it;
        }
        total += load;
        if (load > worst) worst = load;
    }
    return total > 0 ? static_cast<double>(worst) * n_ctas / static_cast<double>(total) : 1.0;
}

// Heads per chunk for a working set of about `budget` bytes and at least `min_passes` passes per chunk:
// among up to 32 sizes around that, the one whose dealing leaves the CTAs' loads most even (the loads are
// counted exactly, by walking every CTA's list).
inline WorkPlan make_work_plan(int BH, int n_tiles, long long T, int D, bool causal, int n_ctas, long long budget,
                               int min_passes) {
    const long long per_head = T * D * 12;  // fp32 accumulator + Q, K, V, dO
    long long cb = budget / per_head;
    const long long c_min = (static_cast<long long>(min_passes) * n_ctas + n_tiles - 1) / n_tiles;  // heads for min_passes passes
    if (cb < c_min) cb = c_min;
    if (cb < 1) cb = 1;
    if (cb * 3 / 2 >= BH) return work_plan_for_chunk(BH, n_tiles, n_ctas, BH);  // everything fits: one list
    const int n_chunks = static_cast<int>((BH + cb - 1) / cb);
    const int even = (BH + n_chunks - 1) / n_chunks;
    int lo = even - even / 3 > 1 ? even - even / 3 : 1;
    if (lo < c_min) lo = static_cast<int>(c_min < even ? c_min : even);
    const int hi = even + even / 4;
    const int step = (hi - lo) / 32 + 1;
    int best = even;
    double best_cost = 1e30;
    for (int c = hi; c >= lo; c -= step) {
        const double imbalance = work_plan_imbalance(BH, n_tiles, causal, n_ctas, work_plan_for_chunk(BH, n_tiles, n_ctas, c));
        // a small penalty on chunks far from the budget on either side
        const double cost = imbalance + 0.02 * (c > even ? c - even : even - c) / even;
        if (cost < best_cost) {
            best_cost = cost;
            best = c;
        }
    }
    return work_plan_for_chunk(BH, n_tiles, n_ctas, best);
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
    // The plan is a pure function of the shape; choosing it walks every item, so the last few are kept.
    struct Entry {
        int BH, D, causal, num_sms;
        long long T;
        WorkPlan plan;
        bool valid;
    };
    constexpr int kEntries = 16;
    static Entry cache[kEntries] = {};
    static int next = 0;
    static std::mutex mutex;
    std::lock_guard<std::mutex> lock(mutex);
    for (const Entry& e : cache)
        if (e.valid && e.BH == BH && e.T == T && e.D == D && e.causal == (causal ? 1 : 0) && e.num_sms == num_sms) return e.plan;
    const WorkPlan plan = make_work_plan(BH, n_tiles, T, D, causal, grid, 48ll << 20, 2);
    cache[next] = Entry{BH, D, causal ? 1 : 0, num_sms, T, plan, true};
    next = (next + 1) % kEntries;
    return plan;
}

}  // namespace nova
