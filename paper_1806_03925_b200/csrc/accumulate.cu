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
//   5. reduce pass: one warp per group sums its rows (fp32, arrival order, 128-bit loads through the sort
//      permutation) and either writes the average to its queue slot or, for the open group, the running
//      sum and count back to the table.  The warp that owns the first group of an image also settles
//      what the image's last, still open group leaves in the table, so no two warps touch one table row.
//   6. commit: the queue length grows by the number of complete groups (or the call is dropped whole if
//      the queue would overflow).
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
    int64_t i0;                // first position owned by this thread
};

// smem: 34 words.  Every thread of the block must call this.
__device__ __forceinline__ void tile_flags(TileFlags& f, const uint32_t* __restrict__ ks, int64_t n, uint32_t vocab,
                                           int M, const int32_t* __restrict__ cnt, uint32_t* smem,
                                           DevState* __restrict__ state) {
    const int64_t tile0 = (int64_t)blockIdx.x * AF_TILE;
    f.i0 = tile0 + (int64_t)threadIdx.x * AF_ITEMS;
    uint32_t prev = vocab;   // key just before this thread's first position
    if (f.i0 < n && f.i0 > 0) prev = ks[f.i0 - 1];
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) f.key[t] = (f.i0 + t < n) ? ks[f.i0 + t] : vocab;

    // start of the image's run that covers the tile's first position (the run may begin in an earlier tile)
    if (threadIdx.x == 0) {
        uint32_t carry = (uint32_t)tile0;
        if (tile0 > 0 && tile0 < n && ks[tile0 - 1] == f.key[0]) {
            int64_t lo = 0, hi = tile0 - 1;       // first index whose key is >= key[0]; ks[hi] == key[0]
            while (lo < hi) {
                const int64_t mid = (lo + hi) >> 1;
                if (ks[mid] < f.key[0]) lo = mid + 1; else hi = mid;
            }
            carry = (uint32_t)lo;
        }
        smem[33] = carry;
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
        f.c0[t] = 0;
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
            const int64_t last = i + (M - rem) - 1;  // the row that brings the count to M
            f.complete[t] = last < n && ks[last] == f.key[t];
        }
        if (i + 1 == n || ks[i + 1] >= vocab) state->n_valid = i + 1;   // exactly one thread sees this
    }
    if (blockIdx.x == 0 && threadIdx.x == 0 && (n == 0 || ks[0] >= vocab)) state->n_valid = 0;   // no valid row at all
}

struct RowSource {
    const uint32_t* perm; const float* grads; int64_t ld; const int32_t* src_row; const float* scale;
};

__global__ void __launch_bounds__(AF_THREADS)
acc_flag_kernel(const uint32_t* __restrict__ ks, int64_t n, uint32_t vocab, int M, const int32_t* __restrict__ cnt,
                uint2* __restrict__ tile_cnt, DevState* __restrict__ state) {
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
                int32_t* __restrict__ psrc, float* __restrict__ pscale, DevState* __restrict__ state) {
    __shared__ uint32_t smem[34];
    TileFlags f;
    tile_flags(f, ks, n, vocab, M, cnt, smem, state);
    uint32_t g = 0, c = 0;
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) { g += f.head[t]; c += f.complete[t]; }
    const uint2 tile_base = tile_cnt[blockIdx.x];
    uint32_t gi = tile_base.x + block_exclusive_scan(g, smem, nullptr);
    uint32_t ci = tile_base.y + block_exclusive_scan(c, smem, nullptr);
    const int64_t q_base = state->q_count;
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) {
        if (!f.head[t]) continue;
        // one 16-byte record per group: start position (top bit: first group of its image in this call), image ID,
        // ready-queue slot (-1: the group stays open), rows the image already held
        grp_rec[gi] = make_uint4((uint32_t)(f.i0 + t) | (f.first[t] ? 0x80000000u : 0u), f.key[t],
                                 (uint32_t)(f.complete[t] ? (int32_t)(q_base + ci) : -1), (uint32_t)f.c0[t]);
        ++gi;
        ci += f.complete[t];
    }
    // where the gradient row of every sorted position lives and what it is scaled by, resolved through the sort
    // permutation once, so that the reduce pass reads both with coalesced loads
#pragma unroll
    for (int t = 0; t < AF_ITEMS; ++t) {
        const int64_t i = f.i0 + t;
        if (i >= n || f.key[t] >= vocab) continue;
        const uint32_t r = rs.perm[i];
        const int32_t src = rs.src_row ? rs.src_row[r] : (int32_t)r;
        psrc[i] = src;
        pscale[i] = rs.scale ? rs.scale[src] : 1.f;
    }
}

struct RowGather {
    const float* grads; int64_t ld; const int32_t* psrc; const float* pscale;
};

// Sum of the gradient rows at sorted positions [a, b), in order.  All 32 lanes call this together.
template <int NQ>
__device__ __forceinline__ void sum_rows(float4 (&acc)[NQ], const RowGather& rg, int64_t a, int64_t b, int n_chunks) {
    const unsigned lane = lane_id();
    for (int64_t p0 = a; p0 < b; p0 += 32) {
        const int m = (int)min((int64_t)32, b - p0);
        int my_s = 0;
        float my_scale = 1.f;
        if ((int)lane < m) { my_s = rg.psrc[p0 + lane]; my_scale = rg.pscale[p0 + lane]; }
        for (int t0 = 0; t0 < m; t0 += 4) {
            float4 v[4][NQ];
            float sc[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int64_t s = __shfl_sync(0xffffffffu, my_s, (t0 + t) & 31);
                sc[t] = __shfl_sync(0xffffffffu, my_scale, (t0 + t) & 31);
                const bool on = t0 + t < m;
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const int ch = lane + 32 * q;
                    v[t][q] = (on && ch < n_chunks) ? ld_stream_f4(rg.grads + s * rg.ld + ch * 4)
                                                    : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    acc[q].x = fmaf(sc[t], v[t][q].x, acc[q].x);
                    acc[q].y = fmaf(sc[t], v[t][q].y, acc[q].y);
                    acc[q].z = fmaf(sc[t], v[t][q].z, acc[q].z);
                    acc[q].w = fmaf(sc[t], v[t][q].w, acc[q].w);
                }
        }
    }
}

template <int NQ>
__global__ void __launch_bounds__(256, NQ <= 2 ? 4 : 2)
acc_reduce_kernel(const uint32_t* __restrict__ ks, RowGather rg, int D, int M, int64_t n_tiles, int64_t ready_cap,
                  const uint2* __restrict__ tile_cnt, const uint4* __restrict__ grp_rec,
                  float* __restrict__ gsum, int32_t* __restrict__ gcnt,
                  int32_t* __restrict__ q_id, float* __restrict__ q_avg, const DevState* __restrict__ state) {
    const uint2 totals = tile_cnt[n_tiles];
    const int64_t n_groups = totals.x;
    if (state->q_count + (int64_t)totals.y > ready_cap) return;      // the whole call is dropped
    const int64_t n_valid = state->n_valid;
    const unsigned lane = lane_id();
    const int n_chunks = D / 4;
    const float m_f = (float)M;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    int64_t g = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    // records of this group and the next one (its start is this group's end), fetched one iteration ahead
    uint4 rec = make_uint4(0u, 0u, 0u, 0u);
    uint32_t next_start = 0;
    if (g < n_groups) {
        rec = grp_rec[g];
        next_start = (g + 1 < n_groups) ? (grp_rec[g + 1].x & 0x7fffffffu) : (uint32_t)n_valid;
    }
    for (; g < n_groups; g += warps) {
        const uint4 cur = rec;
        const int64_t end = next_start;
        const int64_t gn = g + warps;
        if (gn < n_groups) {
            rec = grp_rec[gn];
            next_start = (gn + 1 < n_groups) ? (grp_rec[gn + 1].x & 0x7fffffffu) : (uint32_t)n_valid;
        }
        const bool first = cur.x >> 31;
        const int slot = (int)cur.z;
        if (!first && slot < 0) continue;      // an image's trailing open group: settled by its first group's warp
        const int64_t start = cur.x & 0x7fffffffu;
        const uint32_t key = cur.y;
        const int c0 = first ? (int)cur.w : 0;
        float4 acc[NQ];
#pragma unroll
        for (int q = 0; q < NQ; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        float* srow = gsum + (int64_t)key * D;
        if (c0 > 0) {
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int ch = lane + 32 * q;
                if (ch < n_chunks) acc[q] = ld_f4(srow + ch * 4);
            }
        }
        sum_rows<NQ>(acc, rg, start, end, n_chunks);
        if (slot >= 0) {
            float* qrow = q_avg + (int64_t)slot * D;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int ch = lane + 32 * q;
                if (ch < n_chunks)
                    st_f4(qrow + ch * 4, make_float4(acc[q].x / m_f, acc[q].y / m_f, acc[q].z / m_f, acc[q].w / m_f));
            }
            if (lane == 0) q_id[slot] = (int32_t)key;
            if (!first) continue;
            // what the image's remaining rows leave in the table
            int64_t rest = 0;
            if (end < n_valid && ks[end] == key) {
                int64_t lo = end, step = 1, hi = end + 1;          // ks[lo] == key
                while (hi < n_valid && ks[hi] == key) { lo = hi; step <<= 1; hi = min(lo + step, n_valid); }
                // first index in (lo, hi] whose key differs (hi == n_valid counts as differing)
                int64_t l = lo + 1, h = hi;
                while (l < h) {
                    const int64_t mid = (l + h) >> 1;
                    if (ks[mid] == key) l = mid + 1; else h = mid;
                }
                rest = (l - end) % M;
                if (rest > 0) {
#pragma unroll
                    for (int q = 0; q < NQ; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
                    sum_rows<NQ>(acc, rg, l - rest, l, n_chunks);
                }
            }
            if (rest > 0 || c0 > 0) {
#pragma unroll
                for (int q = 0; q < NQ; ++q) {
                    const int ch = lane + 32 * q;
                    if (ch < n_chunks) st_f4(srow + ch * 4, rest > 0 ? acc[q] : make_float4(0.f, 0.f, 0.f, 0.f));
                }
                if (lane == 0) gcnt[key] = (int32_t)rest;
            }
        } else {
            // the image's only group in this call, still open
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int ch = lane + 32 * q;
                if (ch < n_chunks) st_f4(srow + ch * 4, acc[q]);
            }
            if (lane == 0) gcnt[key] = c0 + (int32_t)(end - start);
        }
    }
}

__global__ void acc_commit_kernel(const uint2* __restrict__ tile_cnt, int64_t n_tiles, int64_t ready_cap,
                                  DevState* __restrict__ state) {
    const uint2 totals = tile_cnt[n_tiles];
    state->n_groups = totals.x;
    state->n_complete = totals.y;
    if (state->q_count + (int64_t)totals.y > ready_cap) atomicOr(&state->status, GEAR_DEV_READY_OVERFLOW);
    else if (totals.y > 0) { state->q_count += totals.y; state->q_calls += 1; }
}

static int reduce_grid() { return 148 * 8; }

cudaError_t launch_accumulate(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                              const int32_t* src_row, const float* scale, int64_t n, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const int64_t vocab = c.cfg.img_vocab;
    const int D = c.cfg.dfv_dim, M = c.cfg.M;
    SortJob sb = c.sort_job(gear_ctx_impl::SORT_IMG);
    DevState* state = c.state();
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
    }
    const uint32_t* ks = sb.keys[cur];
    const int64_t n_tiles = ceil_div(n, AF_TILE);
    uint2* tile_cnt = c.at<uint2>(c.ws.tile_cnt);
    { KernelScope k(&c.prof, "acc_flag", st);
    acc_flag_kernel<<<(unsigned)n_tiles, AF_THREADS, 0, st>>>(ks, n, (uint32_t)vocab, M, c.buf.dfv_gcnt, tile_cnt, state); }
    scan_pairs(tile_cnt, n_tiles, tile_cnt + n_tiles, st, &c.prof);
    uint4* grp_rec = c.at<uint4>(c.ws.grp_rec);
    int32_t* psrc = c.at<int32_t>(c.ws.psrc);
    float* pscale = c.at<float>(c.ws.pscale);
    RowSource rs{sb.vals[cur], grads, ld, src_row, scale};
    RowGather rg{grads, ld, psrc, pscale};
    { KernelScope k(&c.prof, "acc_plan", st);
    acc_plan_kernel<<<(unsigned)n_tiles, AF_THREADS, 0, st>>>(ks, n, (uint32_t)vocab, M, c.buf.dfv_gcnt, tile_cnt,
                                                            grp_rec, rs, psrc, pscale, state); }
    const int nq = (int)ceil_div(D / 4, 32);
    int64_t want = ceil_div(n, 8);
    const int grid = (int)(want < reduce_grid() ? (want < 1 ? 1 : want) : reduce_grid());
#define GEAR_ACC_LAUNCH(NQ) acc_reduce_kernel<NQ><<<grid, 256, 0, st>>>(ks, rg, D, M, n_tiles, c.ws.ready_cap, tile_cnt, \
        grp_rec, c.buf.dfv_gsum, c.buf.dfv_gcnt, c.at<int32_t>(c.ws.q_id), c.at<float>(c.ws.q_avg), state)
    { KernelScope k(&c.prof, "acc_reduce", st);
    if (nq <= 1) GEAR_ACC_LAUNCH(1);
    else if (nq <= 2) GEAR_ACC_LAUNCH(2);
    else if (nq <= 4) GEAR_ACC_LAUNCH(4);
    else GEAR_ACC_LAUNCH(8); }
#undef GEAR_ACC_LAUNCH
    { KernelScope k(&c.prof, "acc_commit", st);
    acc_commit_kernel<<<1, 1, 0, st>>>(tile_cnt, n_tiles, c.ws.ready_cap, state); }
    ++c.acc_calls_pending;
    return cudaGetLastError();
}

// ---------------------------------------------------------------- event 6b: hand the ready queue over
__global__ void collect_begin_kernel(DevState* __restrict__ state, int64_t cap, int64_t* __restrict__ d_n) {
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
    const int64_t n = state->sort_n;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        keys[i] = (uint32_t)q_id[i];
}

// One warp per output entry k: queue slot perm[k]; its emission number is its rank among equal IDs.
__global__ void __launch_bounds__(256)
collect_move_kernel(const uint32_t* __restrict__ sorted_keys, const uint32_t* __restrict__ sorted_perm,
                    const int32_t* __restrict__ q_id, const float* __restrict__ q_avg,
                    int D, const DevState* __restrict__ state, int32_t* __restrict__ ids, int32_t* __restrict__ seq,
                    float* __restrict__ avg) {
    const int64_t n = state->collect_n;
    const bool in_order = state->sort_n == 0;          // the queue itself is sorted: no permutation
    const uint32_t* ks = in_order ? reinterpret_cast<const uint32_t*>(q_id) : sorted_keys;
    const unsigned lane = lane_id();
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t k = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); k < n; k += warps) {
        const uint32_t id = ks[k];
        // first index of this ID's run: gallop backwards, then bisect
        int64_t hi = k, step = 1, lo = k - 1;                  // ks[hi] == id
        while (lo >= 0 && ks[lo] == id) { hi = lo; step <<= 1; lo = max(hi - step, (int64_t)-1); }
        int64_t l = lo + 1, h = hi;                            // answer in [l, h]; ks[h] == id, ks[lo] != id
        while (l < h) {
            const int64_t mid = (l + h) >> 1;
            if (ks[mid] == id) h = mid; else l = mid + 1;
        }
        const float* src = q_avg + (in_order ? k : (int64_t)sorted_perm[k]) * D;
        float* dst = avg + k * D;
        for (int ch = lane; ch < D / 4; ch += 32) st_f4(dst + ch * 4, ld_f4(src + ch * 4));
        if (lane == 0) { ids[k] = (int32_t)id; seq[k] = (int32_t)(k - l); }
    }
}

__global__ void collect_end_kernel(DevState* __restrict__ state) {
    if (state->collect_n >= 0) { state->q_count = 0; state->q_calls = 0; }
}

cudaError_t launch_collect_ready(const gear_ctx_impl& c, int32_t* ids, int32_t* seq, float* avg, int64_t cap,
                                 int64_t* d_n, cudaStream_t st) {
    DevState* state = c.state();
    SortJob sb = c.sort_job(gear_ctx_impl::SORT_READY);
    const int64_t n_max = c.ws.ready_cap;
    { KernelScope k(&c.prof, "collect_begin", st);
    collect_begin_kernel<<<1, 1, 0, st>>>(state, cap, d_n); }
    int cur = 0;
    // A queue fed by at most one accumulate call is in (id, group) order already.  The host knows an upper bound
    // of the number of feeding calls; only when that exceeds one are the sort kernels enqueued at all (the device
    // then still decides from the exact count whether there is anything to re-order).
    if (c.acc_calls_pending > 1) {
        int64_t blocks = ceil_div(n_max, 256);
        { KernelScope k(&c.prof, "collect_keys", st);
        collect_keys_kernel<<<(unsigned)(blocks > 1184 ? 1184 : blocks), 256, 0, st>>>(c.at<int32_t>(c.ws.q_id), state,
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
    collect_move_kernel<<<(unsigned)(want > 1184 ? 1184 : want), 256, 0, st>>>(sb.keys[cur], sb.vals[cur],
                                                                            c.at<int32_t>(c.ws.q_id),
                                                                            c.at<float>(c.ws.q_avg), c.cfg.dfv_dim,
                                                                            state, ids, seq, avg); }
    { KernelScope k(&c.prof, "collect_end", st);
    collect_end_kernel<<<1, 1, 0, st>>>(state); }
    return cudaGetLastError();
}

}  // namespace gear
