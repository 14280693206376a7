// Stable LSD radix sort of (key, value) pairs and small scan helpers.
//
// One cooperative, persistent kernel sorts up to three independent arrays ("jobs") in one launch.  Tiles of RS_TILE
// consecutive elements are dealt to the blocks round robin, in order.
//   histogram  one sweep over the keys gives the digit histogram of EVERY pass (the histograms do not depend on
//              the order of the elements), accumulated per block in shared memory and added to a small global
//              table; the same sweep clears the tiles' descriptors.  One grid barrier.
//   pass       (digits of up to 9 bits) a tile reads its keys once, ranks them (a warp owns 32 * RS_ITEMS
//              consecutive elements and ranks equal digits with match_any, which keeps equal keys in index order),
//              publishes its digit counts in the tile's descriptor and finds out how many elements of each digit
//              the tiles before it hold by looking back through their descriptors: a descriptor carries either
//              the tile's own counts (published at once) or, once known, the sum over all tiles up to and including
//              it, at which a look-back stops.  The pairs are put in digit order in shared memory and written out
//              position by position, so that neighbouring threads write neighbouring words.  One grid barrier
//              between passes.
// The first pass can read raw int32 IDs and map out-of-range ones to a sentinel key that sorts last, so no
// separate key-building launch is needed.  Arrays whose live size (known only on the device) fits a few
// tiles are sorted by block 0 alone, with block-level barriers only.
//
// The grid barrier is a monotonically increasing 64-bit arrival counter: barrier k of a launch completes
// when the counter reaches base + grid * (k + 1), where the host knows `base` (it adds up what every
// earlier launch contributes).  The kernel is launched cooperatively, so all blocks are resident and a tile's
// predecessors are always being worked on; the spins (barrier and look-back) are bounded all the same, and a block
// that gives up records an error and makes every later wait of the launch fall through.
#include <cstdlib>
#include "common.cuh"

namespace gear {

constexpr uint32_t GRID_SPIN_LIMIT = 1u << 22;
constexpr int RS_SOLO_TILES = 3;        // live tiles (all jobs) up to which block 0 sorts alone
// tile descriptor: the top two bits say what the low 30 hold (0: nothing yet; the tile's own count; the count of all tiles
// up to and including it)
enum : uint32_t { DESC_OWN = 1u << 30, DESC_UPTO = 2u << 30, DESC_COUNT = (1u << 30) - 1u };

__device__ __forceinline__ int64_t effective_n(int64_t n_max, const int64_t* n_dev) {
    if (!n_dev) return n_max;
    int64_t n = __ldcg(n_dev);
    return n < n_max ? (n < 0 ? 0 : n) : n_max;
}

// All threads of every participating block call this.  Returns false once the launch has been abandoned.
__device__ __forceinline__ bool grid_barrier(unsigned long long* ctr, unsigned long long target, int32_t* err) {
    __shared__ int ok_flag;
    __syncthreads();
    if (threadIdx.x == 0) {
        int ok = 1;
        __threadfence();
        atomicAdd(ctr, 1ull);
        uint32_t spin = 0;
        while (*reinterpret_cast<volatile unsigned long long*>(ctr) < target) {
            if (++spin > GRID_SPIN_LIMIT) { atomicCAS(err, 0, 100); ok = 0; break; }
            if ((spin & 1023u) == 1023u && *reinterpret_cast<volatile int32_t*>(err) != 0) { ok = 0; break; }
        }
        __threadfence();
        ok_flag = ok;
    }
    __syncthreads();
    return ok_flag != 0;
}

__device__ __forceinline__ uint32_t load_key(const SortJob& j, int pass, int64_t i, int src) {
    if (pass == 0 && j.ids) {
        const int32_t id = __ldcg(j.ids + i);
        return (id >= 0 && (uint32_t)id < j.sentinel) ? (uint32_t)id : j.sentinel;
    }
    return __ldcg(j.keys[src] + i);
}

// Dynamic shared memory of a block: during a pass the tile's (key, value) pairs in digit order on their way out;
// during the histogram sweep the block's digit histograms of every job and pass.
constexpr int RS_STAGE_BYTES = RS_TILE * 8;
static_assert(3 * RS_MAX_PASSES * RS_BUCKETS * 4 <= RS_STAGE_BYTES, "the histograms of three jobs fit the staging buffer");

// At most 80 registers per thread (three blocks' worth per SM): a sort block then leaves room for a CTA of the
// tensor-core head beside it, which matters because the ID sort of a step runs next to the gather and the head.
__global__ void __launch_bounds__(RS_THREADS, 3)
coop_sort_kernel(const SortBatch batch) {
    extern __shared__ uint32_t stage[];                // [RS_TILE] keys, then [RS_TILE] values
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t base[RS_BUCKETS];              // where each digit of this tile starts in the output
    __shared__ uint32_t lstart[RS_BUCKETS];            // ... and in the tile's own digit order
    __shared__ uint32_t wcnt[RS_THREADS / 32][RS_BUCKETS];
    __shared__ uint32_t gstart[3][RS_BUCKETS];        // per job: where each digit of the current pass starts in the output
    __shared__ int live_tiles[3];
    __shared__ int64_t live_n[3];
    __shared__ int give_up;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    constexpr int DPT = RS_BUCKETS / RS_THREADS;       // adjacent digits owned by a thread

    if (threadIdx.x == 0) {
        for (int j = 0; j < batch.n_jobs; ++j) {
            live_n[j] = effective_n(batch.job[j].n_max, batch.job[j].n_dev);
            live_tiles[j] = (int)ceil_div(live_n[j], RS_TILE);
        }
        give_up = 0;
    }
    __syncthreads();
    int total_tiles = 0;
    for (int j = 0; j < batch.n_jobs; ++j) total_tiles += live_tiles[j];
    // Small problems need no grid barrier (block 0 still advances the arrival counter on behalf of all):
    //   every array fits one tile -> block b sorts array b by itself;  a few tiles in all -> block 0 sorts everything.
    bool one_tile_each = batch.n_jobs > 1 && (int)gridDim.x >= batch.n_jobs;
    for (int j = 0; j < batch.n_jobs; ++j) one_tile_each = one_tile_each && live_tiles[j] <= 1;
    const bool per_job = one_tile_each;
    const bool solo = per_job || total_tiles <= RS_SOLO_TILES;          // this block works alone
    if (solo && (int)blockIdx.x >= (per_job ? batch.n_jobs : 1)) return;
    const int nblk = solo ? 1 : gridDim.x, blk = solo ? 0 : (int)blockIdx.x;
    // the tiles this block walks (with stride nblk, in increasing order)
    int w_begin = blk, w_end = total_tiles;
    if (per_job) {
        w_begin = 0;
        for (int j = 0; j < (int)blockIdx.x; ++j) w_begin += live_tiles[j];
        w_end = w_begin + live_tiles[blockIdx.x];
    }
    unsigned long long target = batch.barrier_base;
    auto sync_all = [&]() -> bool {
        if (solo) { __syncthreads(); return true; }
        target += gridDim.x;
        return grid_barrier(batch.barrier_ctr, target, batch.err);
    };
    auto job_of = [&](int w, int& t) -> int {
        int jj = 0;
        t = w;
        while (t >= live_tiles[jj]) { t -= live_tiles[jj]; ++jj; }
        return jj;
    };

    // ---- histogram sweep: digit histograms of every pass, descriptors of my tiles cleared
    {
        uint32_t* hist = stage;                        // [job][pass][digit]
        for (int i = threadIdx.x; i < 3 * RS_MAX_PASSES * RS_BUCKETS; i += RS_THREADS) hist[i] = 0;
        __syncthreads();
        for (int w = w_begin; w < w_end; w += nblk) {
            int t;
            const int jj = job_of(w, t);
            const SortJob& j = batch.job[jj];
            const int64_t n = live_n[jj];
            const uint32_t mask = (1u << j.width) - 1u;
            for (int p = 0; p < batch.passes; ++p)
                for (int d = threadIdx.x; d < RS_BUCKETS; d += RS_THREADS)
                    __stcg(j.hist + ((int64_t)p * j.n_tiles + t) * RS_BUCKETS + d, 0u);
            const int64_t tile0 = (int64_t)t * RS_TILE;
            bool bad = false;
            uint32_t hk[RS_ITEMS];
#pragma unroll
            for (int it = 0; it < RS_ITEMS; ++it) {                 // all loads of the tile in flight before the first is used
                const int64_t i = tile0 + it * RS_THREADS + threadIdx.x;
                hk[it] = i < n ? load_key(j, 0, i, 0) : 0u;
            }
#pragma unroll
            for (int it = 0; it < RS_ITEMS; ++it) {
                const int64_t i = tile0 + it * RS_THREADS + threadIdx.x;
                if (i < n) {
                    const uint32_t k = hk[it];
                    bad |= (k == j.sentinel);
                    for (int p = 0; p < batch.passes; ++p)
                        atomicAdd(&hist[(jj * RS_MAX_PASSES + p) * RS_BUCKETS + ((k >> (p * j.width)) & mask)], 1u);
                }
            }
            if (bad && j.ids && j.status) atomicOr(j.status, GEAR_DEV_BAD_ID);
        }
        __syncthreads();
        for (int jj = 0; jj < batch.n_jobs; ++jj)
            for (int i = threadIdx.x; i < batch.passes * RS_BUCKETS; i += RS_THREADS) {
                const uint32_t v = hist[jj * RS_MAX_PASSES * RS_BUCKETS + i];
                if (v) atomicAdd(batch.job[jj].tot + i, v);        // tot: [pass][digit], zeroed by the host before the launch
            }
        __threadfence();
    }
    bool ok = sync_all();

    for (int pass = 0; pass < batch.passes && ok; ++pass) {
        const int src = pass & 1, dst = src ^ 1;
        // where each digit starts in the output: digits before it, all tiles (the histogram of the pass), per job
        for (int jj = 0; jj < batch.n_jobs; ++jj) {
            const SortJob& j = batch.job[jj];
            const uint32_t mask = (1u << j.width) - 1u;
            uint32_t gtot[DPT], mine = 0;
#pragma unroll
            for (int q = 0; q < DPT; ++q) {
                const int d = threadIdx.x * DPT + q;
                gtot[q] = d <= (int)mask ? __ldcg(j.tot + pass * RS_BUCKETS + d) : 0u;
                mine += gtot[q];
            }
            uint32_t ex = block_exclusive_scan(mine, scratch, nullptr);
#pragma unroll
            for (int q = 0; q < DPT; ++q) { gstart[jj][threadIdx.x * DPT + q] = ex; ex += gtot[q]; }
        }
        __syncthreads();
        for (int w = w_begin; w < w_end && ok; w += nblk) {
            int t;
            const int jj = job_of(w, t);
            const SortJob& j = batch.job[jj];
            const int64_t n = live_n[jj];
            const int64_t tile0 = (int64_t)t * RS_TILE;
            const int shift = pass * j.width;
            const uint32_t mask = (1u << j.width) - 1u;
            uint32_t* desc = j.hist + ((int64_t)pass * j.n_tiles) * RS_BUCKETS;      // [tile][digit] of this pass
            for (int d = threadIdx.x; d < RS_BUCKETS; d += RS_THREADS)
#pragma unroll
                for (int w2 = 0; w2 < RS_THREADS / 32; ++w2) wcnt[w2][d] = 0;
            __syncthreads();
            uint32_t key[RS_ITEMS], rank[RS_ITEMS], val[RS_ITEMS];
            const int64_t seg0 = tile0 + (int64_t)warp * (32 * RS_ITEMS);
            const bool identity = (pass == 0 && j.identity_vals);
#pragma unroll
            for (int it = 0; it < RS_ITEMS; ++it) {                 // keys and values of the tile: one trip to memory
                const int64_t i = seg0 + it * 32 + lane;
                key[it] = i < n ? load_key(j, pass, i, src) : 0u;
                val[it] = identity ? (uint32_t)i : (i < n ? __ldcg(j.vals[src] + i) : 0u);
            }
#pragma unroll
            for (int it = 0; it < RS_ITEMS; ++it) {
                const int64_t i = seg0 + it * 32 + lane;
                const bool valid = i < n;
                const uint32_t d = valid ? ((key[it] >> shift) & mask) : 0xffffu;
                const uint32_t peers = __match_any_sync(0xffffffffu, d);
                const int leader = __ffs(peers) - 1;
                uint32_t old = 0;
                if (valid && (int)lane == leader) {
                    old = wcnt[warp][d];
                    wcnt[warp][d] = old + __popc(peers);
                }
                old = __shfl_sync(0xffffffffu, old, leader);
                rank[it] = old + __popc(peers & ((1u << lane) - 1u));
                __syncwarp();
            }
            __syncthreads();
            // per digit: the warps' counts become running offsets; the tile's digit counts are published, scanned into
            // lstart (a thread owns adjacent digits), and completed by the counts of the tiles before this one
            uint32_t tot[DPT];
            {
                uint32_t mine = 0;
#pragma unroll
                for (int q = 0; q < DPT; ++q) {
                    const int d = threadIdx.x * DPT + q;
                    uint32_t run = 0;
#pragma unroll
                    for (int w2 = 0; w2 < RS_THREADS / 32; ++w2) {
                        const uint32_t c = wcnt[w2][d];
                        wcnt[w2][d] = run;
                        run += c;
                    }
                    tot[q] = run;
                    mine += run;
                    if (d <= (int)mask) __stcg(desc + (int64_t)t * RS_BUCKETS + d, (t == 0 ? DESC_UPTO : DESC_OWN) | run);
                }
                uint32_t ex = block_exclusive_scan(mine, scratch, nullptr);
#pragma unroll
                for (int q = 0; q < DPT; ++q) {
                    lstart[threadIdx.x * DPT + q] = ex;
                    ex += tot[q];
                }
            }
            // look back: elements of my digits in the tiles before this one
#pragma unroll
            for (int q = 0; q < DPT; ++q) {
                const int d = threadIdx.x * DPT + q;
                uint32_t before = 0;
                if (t > 0 && d <= (int)mask) {
                    // a window of LOOK descriptors is read at once (independent loads, one trip to the L2), then taken in
                    // order: counts are added until a descriptor that covers everything before it, or one that has not
                    // been published yet, where the next window starts
                    constexpr int LOOK = 8;
                    int look = t - 1;
                    uint32_t spin = 0;
                    bool done = false;
                    while (!done) {
                        uint32_t v[LOOK];
#pragma unroll
                        for (int k = 0; k < LOOK; ++k)
                            v[k] = look - k >= 0 ? *reinterpret_cast<volatile uint32_t*>(desc + (int64_t)(look - k) * RS_BUCKETS + d)
                                                 : DESC_UPTO;      // before tile 0: nothing
                        int used = 0;
#pragma unroll
                        for (int k = 0; k < LOOK; ++k) {
                            if (done || used != k) continue;
                            const uint32_t flag = v[k] & ~DESC_COUNT;
                            if (flag == 0u) continue;          // not published yet: the next window starts here
                            before += v[k] & DESC_COUNT;
                            used = k + 1;
                            done = flag == DESC_UPTO;
                        }
                        look -= used;
                        if (!done && used == 0) {
                            if (++spin > GRID_SPIN_LIMIT) { atomicCAS(batch.err, 0, 101); give_up = 1; break; }
                            if ((spin & 1023u) == 1023u && *reinterpret_cast<volatile int32_t*>(batch.err) != 0) { give_up = 1; break; }
                        }
                    }
                    __stcg(desc + (int64_t)t * RS_BUCKETS + d, DESC_UPTO | (before + tot[q]));
                }
                base[d] = gstart[jj][d] + before;
            }
            __syncthreads();
            if (give_up) { ok = false; break; }
            // The pairs are first put in digit order inside the tile (shared memory), then written out position by
            // position: neighbouring threads write neighbouring words of a digit's run, so the stores of a warp fall
            // into a few full sectors instead of 32 different ones.
            uint32_t* skey = stage;
            uint32_t* sval = stage + RS_TILE;
#pragma unroll
            for (int it = 0; it < RS_ITEMS; ++it) {
                const int64_t i = seg0 + it * 32 + lane;
                if (i < n) {
                    const uint32_t d = (key[it] >> shift) & mask;
                    const uint32_t lp = lstart[d] + wcnt[warp][d] + rank[it];
                    skey[lp] = key[it];
                    sval[lp] = val[it];
                }
            }
            __syncthreads();
            const int in_tile = (int)min((int64_t)RS_TILE, n - tile0);
            for (int lp = threadIdx.x; lp < in_tile; lp += RS_THREADS) {
                const uint32_t k = skey[lp];
                const uint32_t d = (k >> shift) & mask;
                const uint32_t pos = base[d] + ((uint32_t)lp - lstart[d]);
                __stcg(j.keys[dst] + pos, k);
                __stcg(j.vals[dst] + pos, sval[lp]);
            }
            __syncthreads();
        }
        if (pass + 1 < batch.passes && !(ok = sync_all() && ok)) break;
    }
    if (solo && blockIdx.x == 0 && threadIdx.x == 0) {
        // the host has already booked this launch's arrivals: deliver them
        __threadfence();
        atomicAdd(batch.barrier_ctr, (unsigned long long)gridDim.x * (unsigned long long)batch.n_barriers);
    }
}

static int coop_grid_limit() {
    static int limit = 0;
    if (!limit) {
        int dev = 0, sms = 0, per_sm = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        cudaFuncSetAttribute(coop_sort_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, RS_STAGE_BYTES);
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, coop_sort_kernel, RS_THREADS, RS_STAGE_BYTES);
        if (sms <= 0) sms = 148;
        if (per_sm <= 0) per_sm = 1;
        if (per_sm > 3) per_sm = 3;
        if (getenv("GEAR_SORT_PER_SM")) per_sm = atoi(getenv("GEAR_SORT_PER_SM"));
        limit = sms * per_sm;
    }
    return limit;
}

int sort_jobs(SortBatch& batch, GridBarrierState* gbs, cudaStream_t st, Profiler* prof, cudaError_t* err_out) {
    *err_out = cudaSuccess;
    int passes = 1, total_tiles = 0;
    for (int j = 0; j < batch.n_jobs; ++j) {
        const int p = (batch.job[j].bits + RS_RADIX_BITS - 1) / RS_RADIX_BITS;
        if (p > passes) passes = p;
    }
    for (int j = 0; j < batch.n_jobs; ++j) {
        SortJob& job = batch.job[j];
        job.width = (job.bits + passes - 1) / passes;
        job.n_tiles = (int)sort_tiles(job.n_max);
        total_tiles += job.n_tiles;
        // the per-pass digit histograms start from zero
        *err_out = cudaMemsetAsync(job.tot, 0, sizeof(uint32_t) * RS_MAX_PASSES * RS_BUCKETS, st);
        if (*err_out != cudaSuccess) return 0;
    }
    batch.passes = passes;
    int grid = total_tiles < coop_grid_limit() ? total_tiles : coop_grid_limit();
    if (grid < 1) grid = 1;
    batch.n_barriers = passes;                          // one after the histogram sweep, one between passes
    batch.barrier_ctr = gbs->device_counter;
    batch.barrier_base = gbs->host_base;
    gbs->host_base += (unsigned long long)grid * (unsigned long long)batch.n_barriers;
    KernelScope k(prof, batch.name ? batch.name : "coop_sort", st);
    void* args[] = {&batch};
    *err_out = cudaLaunchCooperativeKernel((const void*)coop_sort_kernel, dim3(grid), dim3(RS_THREADS), args, RS_STAGE_BYTES, st);
    return passes & 1;
}

// ---------------------------------------------------------------- scan of counter pairs
__global__ void __launch_bounds__(1024)
scan_pairs_kernel(uint2* __restrict__ data, int64_t m, uint2* __restrict__ total) {
    wait_for_predecessor();
    __shared__ uint32_t scratch[33];
    uint32_t ca = 0, cb = 0;
    for (int64_t base = 0; base < m; base += blockDim.x) {
        int64_t i = base + threadIdx.x;
        uint2 v = i < m ? data[i] : make_uint2(0u, 0u);
        uint32_t ta, tb;
        uint32_t ea = block_exclusive_scan(v.x, scratch, &ta);
        uint32_t eb = block_exclusive_scan(v.y, scratch, &tb);
        if (i < m) data[i] = make_uint2(ca + ea, cb + eb);
        ca += ta;
        cb += tb;
    }
    if (threadIdx.x == 0) *total = make_uint2(ca, cb);
}

void scan_pairs(uint2* data, int64_t m, uint2* total, cudaStream_t st, Profiler* prof) {
    KernelScope k(prof, "scan_pairs", st);
    launch_dependent(scan_pairs_kernel, dim3(1), dim3(1024), 0, st, data, m, total);
}

}  // namespace gear
