// Event 5 and event 6 of the step: the gradient store.
//
// Rule (Section 1 of the paper, "accumulated to M"; Section 3, event 6): gradients of one image are kept
// until M have arrived; their average is then handed on and the store for that image starts over.  Rows
// are taken to arrive in index order, so a call that brings k rows for an image holding c0 earlier ones
// completes floor((c0 + k) / M) groups, split exactly at every M-th arrival, and leaves (c0 + k) mod M.
//
// Plan on the device, nothing is read back:
//   1. keys = Image IDs (out-of-range -> sentinel that sorts last); stable radix sort with the row index
//      as value, so rows of one image are contiguous and still in arrival order.
//   2. flag pass: position i of the sorted array starts a group if it is the first row of its image or if
//      (c0 + rank within image) is a multiple of M; a group is complete if the image has enough further
//      rows to reach the next multiple.  Per-tile counts of (groups, complete groups).
//   3. one-block scan of the tile counts.
//   4. plan pass: the flags again, now with their global prefix: group g starts at grp_start[g]; complete
//      groups get consecutive ready-queue slots (a counter-threshold stream compaction: ballot-free block
//      scan of the "count reaches M" predicate).
//   5. reduce pass: a warp sums the rows of each of its groups (fp32, arrival order, whole rows staged through
//      shared memory by asynchronous copies, addressed through the sort permutation) and either writes the
//      average to its queue slot or, for the open group, the running sum and count back to the table.  The
//      warp that owns the first group of an image also settles what the image's last, still open group
//      leaves in the table, so no two warps touch one table row.
//   6. commit (by the block of the reduce pass that finishes last): the queue length grows by the number of
//      complete groups (or the call is dropped whole if the queue would overflow).
// HBM bound: the reduce pass reads every gradient row once and reads/writes one accumulator row per
// distinct image; the sort and flag passes move 4-byte keys only.
#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int AF_THREADS = 256;
constexpr int AF_ITEMS = 4;
constexpr int AF_TILE = AF_THREADS * AF_ITEMS;

__device__ __forceinline__ uint32_t warp_inclusive_max(uint32_t v) {
    const unsigned lane = lane_id();
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= (unsigned)o) v = max(v, t);
    }
    return v;
}

// Flags of the AF_ITEMS consecutive sorted positions a thread owns.
struct TileFlags {
    uint32_t key[AF_ITEMS];
    bool head[AF_ITEMS];       // starts a group
    bool first[AF_ITEMS];      // ... and is the first row of its image in this call
    bool complete[AF_ITEMS];   // ... and the group reaches M
    int c0[AF_ITEMS];          // rows the image already holds in the table
    int seq[AF_ITEMS];         // group heads: how many groups of the image this call completes before this one
    int64_t i0;                // first position owned by this thread
};

// smem: 34 words.  Every thread of the block must call this.
// run_end (optional): run_end[first position of an image's run] = one past its last position.
__device__ __forceinline__ void tile_flags(TileFlags& f, const uint32_t* __restrict__ ks, int64_t n, uint32_t vocab,
                                           int M, const int32_t* __restrict__ cnt, uint32_t* smem,
                                           DevState* __restrict__ state, uint32_t* __restrict__ run_end = nullptr) {
    const int64_t tile0 = (int64_t)blockIdx.x * AF_TILE;
    f.i0 = tile0 + (int64_t)threadIdx.x * AF_ITEMS;
    uint32_t prev = vocab;   // key just before this thread's first position
    if (f.i0 < n && f.i0 > 0) prev = ks[f.i0 - 1];
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) f.key[t] = (f.i0 + t < n) ? ks[f.i0 + t] : vocab;

    // start of the image's run that covers the tile's first position (the run may begin in an earlier tile).  Warp 0
    // searches backwards with all its lanes at once: first one round of probes at distances 1, 2, 4, ... brackets the
    // start, then rounds of 32 evenly spaced probes narrow the bracket by a factor of 32 each, so that even a run of
    // millions of rows (a hot image) costs a handful of trips to memory, and the usual short run one.
    if (threadIdx.x < 32) {
        const int lane0 = (int)threadIdx.x;
        const uint32_t key0 = __shfl_sync(0xffffffffu, f.key[0], 0);
        int64_t start = tile0;
        const bool spans = tile0 > 0 && tile0 < n && ks[tile0 - 1] == key0;      // the same words for every lane
        if (spans) {
            int64_t hi = tile0 - 1;                                  // ks[hi] == key0
            const int64_t far = hi - ((int64_t)1 << lane0);
            const bool same = lane0 < 31 && far >= 0 && ks[far] == key0;
            const int k = __popc(__ballot_sync(0xffffffffu, same));  // probes 0 .. k-1 still lie inside the run
            int64_t lo = hi - ((int64_t)1 << k);                     // ks[lo] != key0, or lo < 0
            if (lo < -1) lo = -1;
            if (k > 0) hi -= (int64_t)1 << (k - 1);
            while (hi - lo > 1) {
                const int64_t step = (hi - lo + 31) / 32;
                const int64_t p = hi - (int64_t)(lane0 + 1) * step;
                const bool in = p > lo && ks[p] == key0;
                const int m = __popc(__ballot_sync(0xffffffffu, in));
                hi -= (int64_t)m * step;
                const int64_t below = hi - step;
                if (below > lo) lo = below;                          // the first probe that failed (it lies above the old lo)
            }
            start = hi;
        }
        if (lane0 == 0) smem[33] = (uint32_t)start;
    }
    // run start of every position: inclusive max-scan of "index if run head"
    uint32_t local_max = 0;
    uint32_t run_start[AF_ITEMS];
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) {
        const uint32_t before = t == 0 ? prev : f.key[t - 1];
        const bool run_head = (f.i0 + t < n) && (f.i0 + t == 0 || f.key[t] != before);
        if (run_head) { local_max = (uint32_t)(f.i0 + t) + 1u; }   // +1 so that 0 means "none"
        run_start[t] = local_max;
    }
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    uint32_t inc = warp_inclusive_max(local_max);
    if (lane == 31) smem[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < (AF_THREADS / 32) ? smem[lane] : 0u;
        w = warp_inclusive_max(w);
        smem[lane] = w;
    }
    __syncthreads();
    uint32_t before_thread = __shfl_up_sync(0xffffffffu, inc, 1);
    if (lane == 0) before_thread = 0;
    if (warp > 0) before_thread = max(before_thread, smem[warp - 1]);
    const uint32_t carry = smem[33];
    __syncthreads();

#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) {
        const int64_t i = f.i0 + t;
        f.head[t] = f.first[t] = f.complete[t] = false;
        f.c0[t] = 0; f.seq[t] = 0;
        if (i >= n || f.key[t] >= vocab) continue;
        uint32_t rs = max(run_start[t], before_thread);
        const int64_t start = rs ? (int64_t)rs - 1 : (int64_t)carry;
        const int64_t j = i - start;                 // rank of this row among the call's rows of its image
        const int c0 = cnt[f.key[t]];
        f.c0[t] = c0;
        const int rem = (int)((c0 + j) % M);
        if (j == 0 || rem == 0) {
            f.head[t] = true;
            f.first[t] = (j == 0);
            f.seq[t] = (int)((c0 + j) / M);          // c0 < M: the first group of the image gets 0
            const int64_t last = i + (M - rem) - 1;  // the row that brings the count to M
            f.complete[t] = last < n && ks[last] == f.key[t];
        }
        const uint32_t after = i + 1 < n ? ks[i + 1] : vocab;
        if (after >= vocab) state->n_valid = i + 1;                     // exactly one thread sees this
        if (run_end && after != f.key[t]) run_end[start] = (uint32_t)(i + 1);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0 && (n == 0 || ks[0] >= vocab)) state->n_valid = 0;   // no valid row at all
}

struct RowSource {
    const uint32_t* perm; const float* grads; int64_t ld; const int32_t* src_row; const float* scale;
};

__global__ void __launch_bounds__(AF_THREADS)
acc_flag_kernel(const uint32_t* __restrict__ ks, int64_t n, uint32_t vocab, int M, const int32_t* __restrict__ cnt,
                uint2* __restrict__ tile_cnt, DevState* __restrict__ state) {
    wait_for_predecessor();
    __shared__ uint32_t smem[34];
    TileFlags f;
    tile_flags(f, ks, n, vocab, M, cnt, smem, state);
    uint32_t g = 0, c = 0;
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) { g += f.head[t]; c += f.complete[t]; }
    uint32_t tg, tc;
    block_exclusive_scan(g, smem, &tg);
    block_exclusive_scan(c, smem, &tc);
    if (threadIdx.x == 0) tile_cnt[blockIdx.x] = make_uint2(tg, tc);
}

__global__ void __launch_bounds__(AF_THREADS)
acc_plan_kernel(const uint32_t* __restrict__ ks, int64_t n, uint32_t vocab, int M, const int32_t* __restrict__ cnt,
                const uint2* __restrict__ tile_cnt, uint4* __restrict__ grp_rec, RowSource rs,
                int2* __restrict__ pmeta, uint32_t* __restrict__ blk_first, uint32_t* __restrict__ run_end,
                DevState* __restrict__ state) {
    wait_for_predecessor();
    __shared__ uint32_t smem[34];
    TileFlags f;
    tile_flags(f, ks, n, vocab, M, cnt, smem, state, run_end);
    uint32_t g = 0, c = 0;
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) { g += f.head[t]; c += f.complete[t]; }
    const uint2 tile_base = tile_cnt[blockIdx.x];
    uint32_t gi = tile_base.x + block_exclusive_scan(g, smem, nullptr);
    uint32_t ci = tile_base.y + block_exclusive_scan(c, smem, nullptr);
    const int64_t q_base = state->q_count;
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) {
        // the reduce pass hands out spans of ACC_SPAN sorted positions: index of the first group that starts in each
        if (((f.i0 + t) % ACC_SPAN) == 0 && f.i0 + t < n && f.key[t] < vocab) blk_first[(f.i0 + t) / ACC_SPAN] = gi;
        if (!f.head[t]) continue;
        // one 16-byte record per group: start position (top bit: first group of its image in this call), image ID,
        // ready-queue slot (-1: the group stays open), and for the image's first group the rows the image already held,
        // for a later one its number among the groups of the image that this call completes
        grp_rec[gi] = make_uint4((uint32_t)(f.i0 + t) | (f.first[t] ? 0x80000000u : 0u), f.key[t],
                                 (uint32_t)(f.complete[t] ? (int32_t)(q_base + ci) : -1),
                                 (uint32_t)(f.first[t] ? f.c0[t] : f.seq[t]));
        ++gi;
        ci += f.complete[t];
    }
    // where the gradient row of every sorted position lives and what it is scaled by (one 8-byte record), resolved
    // through the sort permutation once, so that the reduce pass reads both with one coalesced load
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) {
        const int64_t i = f.i0 + t;
        if (i >= n || f.key[t] >= vocab) continue;
        const uint32_t r = rs.perm[i];
        const int32_t src = rs.src_row ? rs.src_row[r] : (int32_t)r;
        pmeta[i] = make_int2(src, __float_as_int(rs.scale ? rs.scale[src] : 1.f));
    }
}

struct RowGather {
    const float* grads; int64_t ld; const int2* pmeta;      // pmeta[p] = (source row, scale bits) of sorted position p
};

// What a lane knows about "its" group of a span: own rows [start, start + len), then zlen rows from zstart.
struct LaneGroup {
    uint32_t start, key, zstart;
    int slot, c0, len, zlen, items;      // items = rows the warp stages for the group (0: nothing to do)
    int seq;                             // number of the group among those of its image that the call completes
    bool first;
};

// Where the averages of the groups a call completes go when they bypass the ready queue: the caller's own lists
// (gear_accumulate_collect).  All null: the groups join the queue.  cap < 0: the host has checked that the queue is empty
// and that the lists can take every group the call could complete.  cap >= 0: the kernel decides: the lists are used if
// the queue is empty and the call completes at most cap groups, else the groups join the queue and the hand-over pass
// that the host has enqueued behind this kernel deals with them.
struct EmitTarget { int32_t* ids; int32_t* seq; float* avg; int64_t* d_n; int64_t cap; };

// One row to stage, as the copy side sees it (where the row starts; bit 0 of the address word is set if the item
// exists) and as the adding side sees it (what the row is scaled by and
// meta = group lane << 2 | last item of the group << 1 | last of the group's own rows).
struct ItemDesc { uint32_t addr_lo, addr_hi; float scale; int meta; };

// The reduce pass.  A warp takes spans of ACC_SPAN sorted positions, span w, w + W, w + 2W, ... (W = warps of
// the grid); the groups that start inside a span (at most ACC_SPAN, one per lane) are walked as one flat
// sequence of items -- for every group first the image's accumulator row if it holds anything, then its
// gradient rows in arrival order; the first group of an image, if it completes, is followed by the rows of
// the image's trailing open group, so that one warp alone reads and writes the image's accumulator row.
// Items are staged through a per-warp ring of S row-sized shared-memory slots with asynchronous copies
// (cp.async, 16 bytes per lane, whole rows): the copy of item i + S - 1 is issued before item i is added,
// across group boundaries, so a warp keeps S - 1 rows in flight whatever the group sizes are -- most
// groups hold a single row, and registers alone cannot keep enough of those in flight.  What to copy is
// worked out 32 items at a time, one item per lane (a search over the groups' item counts, the position
// record fetched by the lane), one batch ahead of the copies; the inner loop only broadcasts a lane's
// descriptor, copies and adds.  The group records of the next span are requested while the current span
// streams.  Sums are fp32, in arrival order, starting from the stored partial sum.
// FULL: a row is exactly NQ * 512 bytes, so no lane is ever idle.
template <int NQ, int S, bool FULL>
__global__ void __launch_bounds__(256, NQ <= 2 ? 3 : 2)
acc_reduce_kernel(const uint32_t* __restrict__ ks, RowGather rg, int D, int M, int64_t n_tiles, int64_t ready_cap,
                  const uint2* __restrict__ tile_cnt, const uint4* __restrict__ grp_rec,
                  const uint32_t* __restrict__ blk_first, const uint32_t* __restrict__ run_end,
                  float* __restrict__ gsum, int32_t* __restrict__ gcnt,
                  int32_t* __restrict__ q_id, float* __restrict__ q_avg, const EmitTarget direct,
                  DevState* __restrict__ state) {
    wait_for_predecessor();
    extern __shared__ float4 ring_mem[];                          // [warps][S][NQ * 32] float4
    const uint2 totals = tile_cnt[n_tiles];
    const int64_t n_groups = totals.x;
    // Averages go to the ready queue, or (the queue being empty, so that queue slot k is also entry k of the hand-over)
    // straight into the caller's lists, whose capacity the host has checked against the row count.
    const bool to_caller = direct.avg != nullptr &&
                           (direct.cap < 0 || (state->q_count == 0 && (int64_t)totals.y <= direct.cap));
    int32_t* __restrict__ e_id = to_caller ? direct.ids : q_id;
    float* __restrict__ e_avg = to_caller ? direct.avg : q_avg;
    // Step 6 of the plan (commit) is done by whichever block finishes last: by then every block has read the queue
    // length it started from.  Every block, also one of a dropped call, leaves through this.
    const bool dropped = !to_caller && state->q_count + (int64_t)totals.y > ready_cap;
    auto leave = [&]() {
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            unsigned int* ticket = reinterpret_cast<unsigned int*>(&state->pad[4]);
            if (atomicInc(ticket, gridDim.x - 1) == gridDim.x - 1) {
                state->n_complete = totals.y;
                state->direct_done = (to_caller && direct.cap >= 0) ? 1 : 0;
                if (to_caller) { if (direct.d_n) *direct.d_n = totals.y; }
                else if (dropped) atomicOr(&state->status, GEAR_DEV_READY_OVERFLOW);
                else if (totals.y > 0) { state->q_count += totals.y; state->q_calls += 1; }
            }
        }
    };
    if (dropped) { leave(); return; }                                // the whole call is dropped
    const int64_t n_valid = state->n_valid;
    const int lane = (int)lane_id(), warp = (int)(threadIdx.x >> 5);
    const int n_chunks = D / 4;
    const float m_f = (float)M;
    const int64_t W = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t n_spans = ceil_div(n_valid, ACC_SPAN);
    float4* my_ring = ring_mem + (size_t)warp * S * (NQ * 32);
    const uint32_t ring_addr = (uint32_t)__cvta_generic_to_shared(my_ring);
    constexpr uint32_t SLOT_BYTES = NQ * 32 * 16;

    // group range of a span: lane 0 holds the first group, lane 1 one past the last
    auto load_range = [&](int64_t span) -> uint32_t {
        uint32_t v = 0;
        if (span < n_spans && lane < 2) {
            const int64_t w = span + lane;
            v = w < n_spans ? __ldg(blk_first + w) : (uint32_t)n_groups;
        }
        return v;
    };
    auto load_group = [&](int64_t g_lo, int64_t g_hi) -> LaneGroup {
        LaneGroup r{0u, 0u, 0u, -1, 0, 0, 0, 0, 0, false};
        const int64_t g = g_lo + lane;
        if (g < g_hi) {
            const uint4 rec = __ldg(grp_rec + g);
            const uint32_t end = (g + 1 < n_groups) ? (__ldg(&grp_rec[g + 1].x) & 0x7fffffffu) : (uint32_t)n_valid;
            r.start = rec.x & 0x7fffffffu; r.first = rec.x >> 31; r.key = rec.y; r.slot = (int)rec.z;
            r.c0 = r.first ? (int)rec.w : 0;
            r.seq = r.first ? 0 : (int)rec.w;
            r.len = (int)(end - r.start);
        }
        return r;
    };

    int64_t span = (int64_t)blockIdx.x * (blockDim.x >> 5) + warp;
    uint32_t range_cur = load_range(span), range_nxt = load_range(span + W);
    LaneGroup G = load_group(__shfl_sync(0xffffffffu, range_cur, 0), __shfl_sync(0xffffffffu, range_cur, 1));

    for (; span < n_spans; span += W) {
        // ---- look-ahead: group records of the next span, group range of the one after it
        const LaneGroup G_nxt = load_group(__shfl_sync(0xffffffffu, range_nxt, 0), __shfl_sync(0xffffffffu, range_nxt, 1));
        const uint32_t range_nxt2 = load_range(span + 2 * W);

        // ---- complete this lane's group
        if (G.first && G.slot >= 0) {
            // what the image's remaining rows leave in the table: the rows of its trailing open group
            const uint32_t run_stop = __ldg(run_end + G.start);
            G.zlen = (int)(((int64_t)G.c0 + (int64_t)(run_stop - G.start)) % M);
            G.zstart = run_stop - (uint32_t)G.zlen;
        }
        // an image's trailing open group itself (not first, no queue slot) is skipped here
        if (G.len > 0 && (G.first || G.slot >= 0)) G.items = (G.c0 > 0 ? 1 : 0) + G.len + G.zlen;
        const int incl = (int)warp_inclusive_scan((uint32_t)G.items);      // items of the groups in lanes 0 .. lane
        const int total_items = __shfl_sync(0xffffffffu, incl, 31);
        if (total_items > 0) {
            // descriptor of item base + lane
            auto make_desc = [&](int base) -> ItemDesc {
                const int i = base + lane;
                int l = 0;                                      // group lane: the first one with incl > i
#pragma unroll
                for (int step = ACC_SPAN / 2; step >= 1; step >>= 1) {
                    const int v = __shfl_sync(0xffffffffu, incl, l + step - 1);
                    if (v <= i) l += step;
                }
                const int incl_l = __shfl_sync(0xffffffffu, incl, l), items_l = __shfl_sync(0xffffffffu, G.items, l);
                const int c0_l = __shfl_sync(0xffffffffu, G.c0, l), len_l = __shfl_sync(0xffffffffu, G.len, l);
                const uint32_t start_l = __shfl_sync(0xffffffffu, G.start, l);
                const uint32_t zstart_l = __shfl_sync(0xffffffffu, G.zstart, l);
                const uint32_t key_l = __shfl_sync(0xffffffffu, G.key, l);
                const int k = i - (incl_l - items_l);           // item number within the group
                const int tab = c0_l > 0 ? 1 : 0, own_end = tab + len_l;
                const bool ok = i < total_items, is_tab = k < tab;
                const int64_t p = k < own_end ? (int64_t)start_l + (k - tab) : (int64_t)zstart_l + (k - own_end);
                int2 pm = make_int2(0, __float_as_int(1.f));
                if (ok && !is_tab) pm = __ldg(rg.pmeta + p);
                const float* row = (ok && is_tab) ? gsum + (int64_t)key_l * D : rg.grads + (int64_t)pm.x * rg.ld;
                const uint64_t a = reinterpret_cast<uint64_t>(row) | (ok ? 1ull : 0ull);      // rows are 16-byte aligned
                ItemDesc d;
                d.addr_lo = (uint32_t)a; d.addr_hi = (uint32_t)(a >> 32);
                d.scale = __int_as_float(pm.y);
                d.meta = (l << 2) | (k + 1 == items_l ? 2 : 0) | (k + 1 == own_end ? 1 : 0);
                return d;
            };

            float4 acc[NQ];
#pragma unroll
            for (int q = 0; q < NQ; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);

            // acc holds the group's own rows (own_done) and/or everything the warp adds for it (all_done)
            auto settle = [&](int l, bool own_done, bool all_done) {
                const uint32_t key = __shfl_sync(0xffffffffu, G.key, l);
                const int slot = __shfl_sync(0xffffffffu, G.slot, l);
                float* srow = gsum + (int64_t)key * D;
                if (own_done && slot >= 0) {                    // the group reached M: its average joins the queue
                    float* qrow = e_avg + (int64_t)slot * D;
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        const int ch = lane + 32 * q;
                        if (FULL || ch < n_chunks)
                            st_f4(qrow + ch * 4, make_float4(acc[q].x / m_f, acc[q].y / m_f, acc[q].z / m_f, acc[q].w / m_f));
                        acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    if (lane == 0) e_id[slot] = (int32_t)key;
                    if (to_caller) {
                        const int seq = __shfl_sync(0xffffffffu, G.seq, l);
                        if (lane == 0) direct.seq[slot] = seq;
                    }
                }
                if (all_done) {
                    const int c0 = __shfl_sync(0xffffffffu, G.c0, l), len = __shfl_sync(0xffffffffu, G.len, l);
                    const int zlen = __shfl_sync(0xffffffffu, G.zlen, l);
                    const bool first = __shfl_sync(0xffffffffu, (int)G.first, l) != 0;
                    // the table row: the open group (this one if it did not complete, else the image's trailing one)
                    const bool write_row = first && (slot < 0 || zlen > 0 || c0 > 0);
                    if (write_row) {
#pragma unroll
                        for (int q = 0; q < NQ; ++q) {
                            const int ch = lane + 32 * q;
                            if (FULL || ch < n_chunks) st_f4(srow + ch * 4, acc[q]);
                        }
                        if (lane == 0) gcnt[key] = slot < 0 ? c0 + len : zlen;
                    }
#pragma unroll
                    for (int q = 0; q < NQ; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            };

            // cur / nxt: the items being added (base .. base + 31) and the batch after them; icur / inxt: the same for the
            // copies, which run S - 1 items ahead (lane j of icur is item base + j + S - 1)
            ItemDesc cur = make_desc(0), nxt = make_desc(32), icur = make_desc(S - 1), inxt = make_desc(32 + S - 1);
            int islot = 0, cslot = 0;
            auto advance = [](int slot) { return (S & (S - 1)) == 0 ? ((slot + 1) & (S - 1)) : (slot + 1 == S ? 0 : slot + 1); };
            // copy of the item in lane j of descriptor batch d (an empty copy if the item does not exist)
            auto issue = [&](const ItemDesc& d, int j) {
                const uint32_t lo = __shfl_sync(0xffffffffu, d.addr_lo, j), hi = __shfl_sync(0xffffffffu, d.addr_hi, j);
                const float* src = reinterpret_cast<const float*>(((uint64_t)hi << 32) | (lo & ~15u));
                const int bytes = (int)(lo & 1u) << 4;
                const uint32_t dst = ring_addr + (uint32_t)islot * SLOT_BYTES;
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const int ch = lane + 32 * q;
                    const bool on = FULL || ch < n_chunks;          // lanes past the end of a narrow row copy nothing
                    cp_async_16(dst + (uint32_t)ch * 16u, src + (on ? ch * 4 : 0), on ? bytes : 0);
                }
                cp_async_commit();
                islot = advance(islot);
            };

            // ---- the pipeline: S - 1 items ahead
            __syncwarp();
#pragma unroll
            for (int i = 0; i < S - 1; ++i) issue(cur, i);
            for (int base = 0; base < total_items; base += 32) {
                const int n_in = min(32, total_items - base);
                for (int j = 0; j < n_in; ++j) {
                    __syncwarp();                                 // every lane is done with the slot refilled next
                    issue(icur, j);
                    cp_async_wait<S - 1>();
                    __syncwarp();                                 // ... and sees the other lanes' copies of item base + j
                    const float scale = __shfl_sync(0xffffffffu, cur.scale, j);
                    const int meta = __shfl_sync(0xffffffffu, cur.meta, j);
                    const float4* row = my_ring + (size_t)cslot * (NQ * 32);
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        const float4 v = row[lane + 32 * q];
                        // in the indirect form the scaled row is never stored: the product joins the sum with one rounding
                        acc[q].x = fmaf(scale, v.x, acc[q].x); acc[q].y = fmaf(scale, v.y, acc[q].y);
                        acc[q].z = fmaf(scale, v.z, acc[q].z); acc[q].w = fmaf(scale, v.w, acc[q].w);
                    }
                    if (meta & 3) settle(meta >> 2, (meta & 1) != 0, (meta & 2) != 0);
                    cslot = advance(cslot);
                }
                cur = nxt; icur = inxt;
                nxt = make_desc(base + 64);
                inxt = make_desc(base + 64 + S - 1);
            }
            cp_async_wait<0>();
        }
        G = G_nxt; range_nxt = range_nxt2;
    }
    leave();
}

// Steps 2-4 of the plan over the sorted keys ks / permutation perm (flag pass, scan, plan pass).
static cudaError_t enqueue_plan(const gear_ctx_impl& c, const uint32_t* ks, const uint32_t* perm, int64_t n,
                                const int32_t* src_row, const float* scale, cudaStream_t st) {
    const int64_t vocab = c.cfg.img_vocab;
    const int M = c.cfg.M;
    DevState* state = c.state();
    const int64_t n_tiles = ceil_div(n, AF_TILE);
    uint2* tile_cnt = c.at<uint2>(c.ws.tile_cnt);
    { KernelScope k(&c.prof, "acc_flag", st);
    launch_dependent(acc_flag_kernel, dim3((unsigned)n_tiles), dim3(AF_THREADS), 0, st, ks, n, (uint32_t)vocab, M, c.buf.dfv_gcnt, tile_cnt, state); }
    scan_pairs(tile_cnt, n_tiles, tile_cnt + n_tiles, st, &c.prof);
    RowSource rs{perm, nullptr, 0, src_row, scale};
    { KernelScope k(&c.prof, "acc_plan", st);
    launch_dependent(acc_plan_kernel, dim3((unsigned)n_tiles), dim3(AF_THREADS), 0, st, ks, n, (uint32_t)vocab, M, c.buf.dfv_gcnt, tile_cnt,
                     c.at<uint4>(c.ws.grp_rec), rs, c.at<int2>(c.ws.pmeta), c.at<uint32_t>(c.ws.blk_first),
                     c.at<uint32_t>(c.ws.run_end), state); }
    return cudaGetLastError();
}

// The plan for the image occurrences of the batch gear_forward_backward has just sorted, enqueued ahead of the
// accumulate call that will use it (on the side stream, beside the head): it depends on the sorted IDs, the counts in
// the table and the queue length only, none of which changes before that call unless another accumulate or collect
// comes first -- those calls drop the plan.
cudaError_t launch_accumulate_plan_ahead(const gear_ctx_impl& c, int64_t n, const int32_t* src_row, const float* scale,
                                         cudaStream_t st) {
    c.plan_ready = false;
    if (n <= 0 || !c.img_sorted || !c.img_sort_valid || c.cfg.accum_mode != GEAR_ACC_SORT) return cudaSuccess;
    SortJob sb = c.sort_job(gear_ctx_impl::SORT_IMG);
    cudaError_t e = enqueue_plan(c, sb.keys[c.img_sorted_buf], sb.vals[c.img_sorted_buf], n, src_row, scale, st);
    if (e != cudaSuccess) return e;
    c.plan_ready = true; c.plan_n = n; c.plan_src_row = src_row; c.plan_scale = scale;
    return cudaSuccess;
}

// to_caller (optional): the caller's lists; only valid while the ready queue is known to be empty and the lists hold
// at least n entries (gear_accumulate_collect checks both on the host)
static cudaError_t launch_accumulate_to(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                                        const int32_t* src_row, const float* scale, int64_t n, const EmitTarget& to_caller,
                                        cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const int64_t vocab = c.cfg.img_vocab;
    const int D = c.cfg.dfv_dim, M = c.cfg.M;
    SortJob sb = c.sort_job(gear_ctx_impl::SORT_IMG);
    DevState* state = c.state();
    const bool planned = !img_id && c.plan_ready && c.plan_n == n && c.plan_src_row == src_row && c.plan_scale == scale;
    c.plan_ready = false;
    // "the batch of the last gear_forward_backward" after a call with explicit IDs has used the sort buffers: sort again
    const bool resort_batch = !img_id && !c.img_sort_valid;
    if (resort_batch) img_id = c.last_img_id;
    int cur = c.img_sorted_buf;
    if (img_id) {
        SortBatch batch = c.sort_batch();
        batch.n_jobs = 1;
        batch.job[0] = sb;
        batch.job[0].ids = img_id;
        batch.job[0].sentinel = (uint32_t)vocab;
        batch.job[0].n_max = n;
        batch.job[0].bits = bits_for(vocab);
        cudaError_t se;
        batch.name = "sort_img";
        cur = sort_jobs(batch, &c.gbs, st, &c.prof, &se);
        if (se != cudaSuccess) return se;
        c.img_sort_valid = resort_batch;
        if (resort_batch) c.img_sorted_buf = cur;
    }
    const uint32_t* ks = sb.keys[cur];
    const int64_t n_tiles = ceil_div(n, AF_TILE);
    uint2* tile_cnt = c.at<uint2>(c.ws.tile_cnt);
    if (!planned) {
        cudaError_t pe = enqueue_plan(c, ks, sb.vals[cur], n, src_row, scale, st);
        if (pe != cudaSuccess) return pe;
    }
    uint4* grp_rec = c.at<uint4>(c.ws.grp_rec);
    int2* pmeta = c.at<int2>(c.ws.pmeta);
    RowGather rg{grads, ld, pmeta};
    uint32_t* blk_first = c.at<uint32_t>(c.ws.blk_first);
    uint32_t* run_end = c.at<uint32_t>(c.ws.run_end);
    (void)vocab; (void)state;
    const int nq = (int)ceil_div(D / 4, 32);
    const int64_t want = ceil_div(ceil_div(n, ACC_SPAN), 8);
    const int resident = sm_count() * (nq <= 2 ? 3 : 2);          // every block stays resident
    const int grid = (int)(want < resident ? (want < 1 ? 1 : want) : resident);
    cudaError_t le = cudaSuccess;
    { KernelScope k(&c.prof, "acc_reduce", st);
    auto launch = [&](auto kernel, int slot_bytes, int slots) {
        const int smem = 8 * slots * slot_bytes;
        le = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (le != cudaSuccess) return;
        le = launch_dependent(kernel, dim3(grid), dim3(256), (size_t)smem, st, ks, rg, D, M, n_tiles, c.ws.ready_cap, tile_cnt, grp_rec, blk_first, run_end,
                                        c.buf.dfv_gsum, c.buf.dfv_gcnt, c.at<int32_t>(c.ws.q_id),
                                        c.at<float>(c.ws.q_avg), to_caller, state);
    };
    // ring depth: as many row slots as about 96 KB per block (two blocks per SM) allow, at most 8.
    // FULL only when a row fills the instantiated width exactly (D == NQ * 128): every lane then owns a chunk of every
    // row; any other width (also 384, 640, 768, 896, which round up to the next instantiation) keeps the per-chunk guard
#define GEAR_ACC_LAUNCH(NQ, S) \
    do { if (D == NQ * 128) launch(acc_reduce_kernel<NQ, S, true>, NQ * 512, S); else launch(acc_reduce_kernel<NQ, S, false>, NQ * 512, S); } while (0)
    if (nq <= 1) GEAR_ACC_LAUNCH(1, 8);
    else if (nq <= 2) GEAR_ACC_LAUNCH(2, 8);
    else if (nq <= 4) GEAR_ACC_LAUNCH(4, 5);
    else GEAR_ACC_LAUNCH(8, 3);
#undef GEAR_ACC_LAUNCH
    }
    if (le != cudaSuccess) return le;
    if (!to_caller.avg) ++c.acc_calls_pending;                    // a call that bypasses the queue leaves it empty (a call
                                                                  // that may or may not bypass it: see launch_accumulate_collect)
    return cudaGetLastError();
}

cudaError_t launch_accumulate(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                              const int32_t* src_row, const float* scale, int64_t n, cudaStream_t st) {
    return launch_accumulate_to(c, img_id, grads, ld, src_row, scale, n, EmitTarget{nullptr, nullptr, nullptr, nullptr, -1}, st);
}

// Events 5 and 6 in one call.  When the host knows the ready queue to be empty (no accumulate call since a collect that
// could not be refused) and the caller's lists can take every group the n rows could complete, the reduce pass writes
// ids, emission numbers and averages straight into the caller's lists and its last block reports the count: no
// hand-over pass, and the averages cross memory once.  Otherwise: accumulate into the queue, then hand the queue over.
cudaError_t launch_accumulate_collect(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                                      const int32_t* src_row, const float* scale, int64_t n, int32_t* ids, int32_t* seq,
                                      float* avg, int64_t cap, int64_t* d_n, cudaStream_t st) {
    const bool queue_empty = c.cfg.accum_mode == GEAR_ACC_SORT && c.acc_calls_pending == 0 && n > 0;
    if (queue_empty && cap >= n)
        return launch_accumulate_to(c, img_id, grads, ld, src_row, scale, n, EmitTarget{ids, seq, avg, d_n, -1}, st);
    if (queue_empty && cap > 0) {
        // the lists may or may not be long enough for what this call completes: the reduce pass finds out, and the
        // hand-over pass behind it moves the queue only if the reduce pass had to use it
        cudaError_t de = launch_accumulate_to(c, img_id, grads, ld, src_row, scale, n, EmitTarget{ids, seq, avg, d_n, cap}, st);
        if (de != cudaSuccess) return de;
        c.acc_calls_pending = 1;
        return launch_collect_ready(c, ids, seq, avg, cap, d_n, st);
    }
    cudaError_t e = cudaSuccess;
    if (n > 0)
        e = c.cfg.accum_mode == GEAR_ACC_ATOMIC
                ? launch_accumulate_atomic(c, img_id ? img_id : c.last_img_id, grads, ld, src_row, scale, n, st)
                : launch_accumulate(c, img_id, grads, ld, src_row, scale, n, st);
    if (e != cudaSuccess) return e;
    return launch_collect_ready(c, ids, seq, avg, cap, d_n, st);
}

// ---------------------------------------------------------------- GEAR_ACC_ATOMIC: the store without arrival order
// Rows are added to the accumulator rows with fp32 reductions in whatever order the hardware takes them, so
// which arrivals share a group is not defined; what is defined (and equal to the ordered path) is every
// image's count and its number of emissions.  After all rows of the call have been added, every image that
// was touched and now holds k >= M gradients emits floor(k / M) averages, each the mean of all k pooled
// gradients, and keeps k mod M gradients' worth of that mean, so that nothing is lost or counted twice.
// Under heavy skew the reductions of a hot image serialise on its accumulator row; that is the cost the
// sorted path avoids.
constexpr int32_t ACC_TOUCHED = 0x40000000;      // bit of dfv_gcnt[id] while a call is in flight: id is on the touched list

__global__ void __launch_bounds__(256)
acc_atomic_add_kernel(const int32_t* __restrict__ img_id, int64_t n, int64_t vocab, const float* __restrict__ grads,
                      int64_t ld, const int32_t* __restrict__ src_row, const float* __restrict__ scale, int D,
                      float* __restrict__ gsum, int32_t* __restrict__ gcnt, int32_t* __restrict__ touched,
                      int64_t ready_cap, DevState* __restrict__ state) {
    wait_for_predecessor();
    // a call completes at most n groups: refuse it whole if the queue could not take them
    const bool drop = state->q_count + n > ready_cap;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        state->pad[3] = drop ? 1 : 0;
        if (drop) atomicOr(&state->status, GEAR_DEV_READY_OVERFLOW);
    }
    if (drop) return;
    const unsigned lane = lane_id();
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    int flags = 0;
    for (int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < n; r += warps) {
        const int32_t id = img_id[r];
        if (id < 0 || id >= vocab) { flags |= GEAR_DEV_BAD_ID; continue; }
        const int64_t s = src_row ? src_row[r] : r;
        const float sc = scale ? scale[s] : 1.f;
        for (int ch = lane; ch < D / 4; ch += 32) {
            const float4 v = ld_stream_f4(grads + s * ld + ch * 4);
            red_add_f4(gsum + (int64_t)id * D + ch * 4, make_float4(sc * v.x, sc * v.y, sc * v.z, sc * v.w));
        }
        if (lane == 0) {
            const int32_t before = atomicOr(&gcnt[id], ACC_TOUCHED);
            if (!(before & ACC_TOUCHED)) {
                const unsigned long long pos = atomicAdd(reinterpret_cast<unsigned long long*>(&state->pad[2]), 1ull);
                touched[pos] = id;
            }
            atomicAdd(&gcnt[id], 1);
        }
    }
    if (flags) atomicOr(&state->status, flags);
}

__global__ void __launch_bounds__(256)
acc_atomic_settle_kernel(const int32_t* __restrict__ touched, int D, int M, float* __restrict__ gsum,
                         int32_t* __restrict__ gcnt, int32_t* __restrict__ q_id, float* __restrict__ q_avg,
                         DevState* __restrict__ state) {
    wait_for_predecessor();
    if (state->pad[3] != 0) return;                            // the call was dropped
    const int64_t n_touched = state->pad[2];
    const unsigned lane = lane_id();
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    if (blockIdx.x == 0 && threadIdx.x == 0)                   // emission order is not ID order: collect has to sort
        atomicAdd(reinterpret_cast<unsigned long long*>(&state->q_calls), 2ull);
    for (int64_t t = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); t < n_touched; t += warps) {
        const int32_t id = touched[t];
        const int32_t k = gcnt[id] & ~ACC_TOUCHED;
        const int32_t e = k / M, rest = k % M;
        float* row = gsum + (int64_t)id * D;
        if (e > 0) {
            unsigned long long slot0 = 0;
            if (lane == 0) slot0 = atomicAdd(reinterpret_cast<unsigned long long*>(&state->q_count), (unsigned long long)e);
            slot0 = __shfl_sync(0xffffffffu, slot0, 0);
            const float kf = (float)k, rf = (float)rest;
            for (int ch = lane; ch < D / 4; ch += 32) {
                const float4 sum = ld_f4(row + ch * 4);
                const float4 avg = make_float4(sum.x / kf, sum.y / kf, sum.z / kf, sum.w / kf);
                for (int32_t j = 0; j < e; ++j) st_f4(q_avg + (int64_t)(slot0 + j) * D + ch * 4, avg);
                st_f4(row + ch * 4, make_float4(avg.x * rf, avg.y * rf, avg.z * rf, avg.w * rf));
            }
            for (int32_t j = lane; j < e; j += 32) q_id[slot0 + j] = id;
        }
        if (lane == 0) gcnt[id] = rest;
    }
}

cudaError_t launch_accumulate_atomic(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                                     const int32_t* src_row, const float* scale, int64_t n, cudaStream_t st) {
    c.plan_ready = false;
    if (n <= 0) return cudaSuccess;
    DevState* state = c.state();
    int32_t* touched = c.at<int32_t>(c.ws.pmeta);               // the sorted path's scratch is free in this mode
    cudaError_t e = cudaMemsetAsync(&state->pad[2], 0, sizeof(int64_t), st);
    if (e != cudaSuccess) return e;
    const int64_t want = ceil_div(n, 8);
    const int resident = sm_count() * 8;
    const int grid = (int)(want < resident ? (want < 1 ? 1 : want) : resident);
    { KernelScope k(&c.prof, "acc_atomic_add", st);
    launch_dependent(acc_atomic_add_kernel, dim3(grid), dim3(256), 0, st, img_id, n, c.cfg.img_vocab, grads, ld, src_row, scale, c.cfg.dfv_dim,
                                                c.buf.dfv_gsum, c.buf.dfv_gcnt, touched, c.ws.ready_cap, state); }
    { KernelScope k(&c.prof, "acc_atomic_settle", st);
    launch_dependent(acc_atomic_settle_kernel, dim3(grid), dim3(256), 0, st, touched, c.cfg.dfv_dim, c.cfg.M, c.buf.dfv_gsum, c.buf.dfv_gcnt,
                                                   c.at<int32_t>(c.ws.q_id), c.at<float>(c.ws.q_avg), state); }
    c.acc_calls_pending += 2;
    return cudaGetLastError();
}

// ---------------------------------------------------------------- event 6b: hand the ready queue over
__global__ void collect_begin_kernel(DevState* __restrict__ state, int64_t cap, int64_t* __restrict__ d_n) {
    wait_for_predecessor();
    const int64_t n = state->q_count;
    if (d_n) *d_n = n;
    if (n > cap) { atomicOr(&state->status, GEAR_DEV_OUT_CAPACITY); state->collect_n = -1; state->sort_n = 0; }
    else {
        state->collect_n = n;
        // One accumulate call fills its slots in (id, group) order already; only a queue fed by several calls
        // has to be re-ordered.
        state->sort_n = state->q_calls <= 1 ? 0 : n;
    }
}

__global__ void __launch_bounds__(256)
collect_keys_kernel(const int32_t* __restrict__ q_id, const DevState* __restrict__ state, uint32_t* __restrict__ keys) {
    wait_for_predecessor();
    const int64_t n = state->sort_n;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        keys[i] = (uint32_t)q_id[i];
}

// Output entry k comes from queue slot perm[k] (or k itself when the queue is already in order); its emission
// number is its rank among equal IDs.  IDs and emission numbers: one thread per entry.  Rows: a warp copies
// eight rows at a time, 16 bytes per lane, all loads issued before the first store.
__global__ void __launch_bounds__(256)
collect_move_kernel(const uint32_t* __restrict__ sorted_keys, const uint32_t* __restrict__ sorted_perm,
                    const int32_t* __restrict__ q_id, const float* __restrict__ q_avg,
                    int D, DevState* __restrict__ state, int32_t* __restrict__ ids, int32_t* __restrict__ seq,
                    float* __restrict__ avg, int solo, int64_t cap, int64_t* __restrict__ d_n) {
    wait_for_predecessor();
    // solo: this launch is the whole hand-over (a queue fed by one accumulate call is in order already): it checks
    // the caller's capacity itself and the last block to finish empties the queue
    const int64_t n = solo ? state->q_count : state->collect_n;
    if (solo) {
        if (state->direct_done != 0) {
            // the reduce pass in front of this launch has written the caller's lists and the count itself: nothing to
            // move; the block that leaves last takes the mark down
            __shared__ int last_out;
            __syncthreads();
            if (threadIdx.x == 0) {
                __threadfence();
                last_out = atomicInc(&state->pad32, gridDim.x - 1) == gridDim.x - 1;
                if (last_out) state->direct_done = 0;
            }
            return;
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            if (d_n) *d_n = n;
            if (n > cap) atomicOr(&state->status, GEAR_DEV_OUT_CAPACITY);
        }
        if (n > cap) return;                            // nothing is consumed
    }
    const bool in_order = solo || state->sort_n == 0;  // the queue itself is sorted: no permutation
    const uint32_t* ks = in_order ? reinterpret_cast<const uint32_t*>(q_id) : sorted_keys;
    const int64_t threads = (int64_t)gridDim.x * blockDim.x;
    for (int64_t k = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += threads) {
        const uint32_t id = ks[k];
        // first index of this ID's run: gallop backwards, then bisect
        int64_t hi = k, step = 1, lo = k - 1;                  // ks[hi] == id
        while (lo >= 0 && ks[lo] == id) { hi = lo; step <<= 1; lo = max(hi - step, (int64_t)-1); }
        int64_t l = lo + 1, h = hi;                            // answer in [l, h]; ks[h] == id, ks[lo] != id
        while (l < h) {
            const int64_t mid = (l + h) >> 1;
            if (ks[mid] == id) h = mid; else l = mid + 1;
        }
        ids[k] = (int32_t)id;
        seq[k] = (int32_t)(k - l);
    }
    const unsigned lane = lane_id();
    const int64_t warps = threads >> 5;
    const int chunks = D / 4;
    constexpr int R = 8;
    for (int64_t k0 = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; k0 < n; k0 += R * warps) {
        int64_t src[R];
#pragma unroll
        for (int t = 0; t < R; ++t) {
            const int64_t k = k0 + t * warps;
            src[t] = k < n ? (in_order ? k : (int64_t)sorted_perm[k]) : -1;
        }
        for (int ch = lane; ch < chunks; ch += 32) {
            float4 v[R];
#pragma unroll
            for (int t = 0; t < R; ++t)
                v[t] = src[t] >= 0 ? ld_stream_f4(q_avg + src[t] * D + ch * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int t = 0; t < R; ++t)
                if (src[t] >= 0) st_f4(avg + (k0 + t * warps) * D + ch * 4, v[t]);
        }
    }
    if (solo) {
        __shared__ int is_last;
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            is_last = atomicInc(&state->pad32, gridDim.x - 1) == gridDim.x - 1;
            if (is_last) { state->q_count = 0; state->q_calls = 0; }
        }
    }
}

__global__ void collect_end_kernel(DevState* __restrict__ state) {
    wait_for_predecessor();
    if (state->collect_n >= 0) { state->q_count = 0; state->q_calls = 0; }
}

cudaError_t launch_collect_ready(const gear_ctx_impl& c, int32_t* ids, int32_t* seq, float* avg, int64_t cap,
                                 int64_t* d_n, cudaStream_t st) {
    DevState* state = c.state();
    c.plan_ready = false;                                    // a plan made ahead counted on the queue length of before
    SortJob sb = c.sort_job(gear_ctx_impl::SORT_READY);
    const int64_t n_max = c.ws.ready_cap;
    const int64_t resident = (int64_t)sm_count() * 8;       // blocks of 256 threads that fit the GPU at once
    const bool solo = c.acc_calls_pending <= 1;
    if (!solo) { KernelScope k(&c.prof, "collect_begin", st);
    launch_dependent(collect_begin_kernel, dim3(1), dim3(1), 0, st, state, cap, d_n); }
    int cur = 0;
    // A queue fed by at most one accumulate call is in (id, group) order already.  The host knows an upper bound
    // of the number of feeding calls; only when that exceeds one are the sort kernels enqueued at all (the device
    // then still decides from the exact count whether there is anything to re-order).
    if (c.acc_calls_pending > 1) {
        int64_t blocks = ceil_div(n_max, 256);
        { KernelScope k(&c.prof, "collect_keys", st);
        launch_dependent(collect_keys_kernel, dim3((unsigned)(blocks > resident ? resident : blocks)), dim3(256), 0, st, c.at<int32_t>(c.ws.q_id), state,
                                                                                     sb.keys[0]); }
        SortBatch batch = c.sort_batch();
        batch.n_jobs = 1;
        batch.job[0] = sb;
        batch.job[0].n_max = n_max;
        batch.job[0].n_dev = &state->sort_n;
        batch.job[0].bits = bits_for(c.cfg.img_vocab);
        cudaError_t se;
        batch.name = "sort_ready";
        cur = sort_jobs(batch, &c.gbs, st, &c.prof, &se);
        if (se != cudaSuccess) return se;
    }
    if (cap >= c.ws.ready_cap) c.acc_calls_pending = 0;      // this collect cannot be refused: the queue will be empty
    int64_t want = ceil_div(n_max, 8);
    { KernelScope k(&c.prof, "collect_move", st);
    launch_dependent(collect_move_kernel, dim3((unsigned)(want > resident ? resident : want)), dim3(256), 0, st, sb.keys[cur], sb.vals[cur],
                                                                            c.at<int32_t>(c.ws.q_id),
                                                                            c.at<float>(c.ws.q_avg), c.cfg.dfv_dim,
                                                                            state, ids, seq, avg, solo ? 1 : 0, cap, d_n); }
    if (!solo) { KernelScope k(&c.prof, "collect_end", st);
    launch_dependent(collect_end_kernel, dim3(1), dim3(1), 0, st, state); }
    return cudaGetLastError();
}

}  // namespace gear
