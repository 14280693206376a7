// Stable LSD radix sort of (key, value) pairs and small scan helpers.
//
// One cooperative, persistent kernel sorts up to three independent arrays ("jobs") in one launch.  A pass
// (digits of up to 9 bits) has three phases over tiles of RS_TILE consecutive elements, separated by
// grid-wide barriers:
//   count    per-tile digit histogram -> hist[digit][tile]
//   scan     one warp per digit: exclusive scan of that digit's per-tile counts, digit total
//   scatter  each tile looks up where its digits start, ranks its elements and writes them out.  A warp owns
//            32 * RS_ITEMS consecutive elements of a tile and ranks equal digits with match_any, which
//            keeps equal keys in index order.
// The first pass can read raw int32 IDs and map out-of-range ones to a sentinel key that sorts last, so no
// separate key-building launch is needed.  Arrays whose live size (known only on the device) fits a few
// tiles are sorted by block 0 alone, with block-level barriers only.
//
// The grid barrier is a monotonically increasing 64-bit arrival counter: barrier k of a launch completes
// when the counter reaches base + grid * (k + 1), where the host knows `base` (it adds up what every
// earlier launch contributes).  The kernel is launched cooperatively, so all blocks are resident; the
// spin is bounded all the same, and a block that gives up records an error and makes every later barrier
// of the launch fall through.
#include "common.cuh"

namespace gear {

constexpr uint32_t GRID_SPIN_LIMIT = 1u << 22;
constexpr int RS_SOLO_TILES = 3;        // live tiles (all jobs) up to which block 0 sorts alone

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

// At most 80 registers per thread (three blocks' worth per SM): a sort block then leaves room for a CTA of the
// tensor-core head beside it, which matters because the ID sort of a step runs next to the gather and the head.
__global__ void __launch_bounds__(RS_THREADS, 3)
coop_sort_kernel(const SortBatch batch) {
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t base[RS_BUCKETS];
    __shared__ uint32_t wcnt[RS_THREADS / 32][RS_BUCKETS];
    __shared__ int live_tiles[3];
    __shared__ int64_t live_n[3];
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;

    if (threadIdx.x == 0) {
        for (int j = 0; j < batch.n_jobs; ++j) {
            live_n[j] = effective_n(batch.job[j].n_max, batch.job[j].n_dev);
            live_tiles[j] = (int)ceil_div(live_n[j], RS_TILE);
        }
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
    // the tiles and the digit rows this block walks (with stride nblk)
    int w_begin = blk, w_end = total_tiles, r_begin = 0, r_end = batch.n_jobs * RS_BUCKETS;
    if (per_job) {
        w_begin = 0;
        for (int j = 0; j < (int)blockIdx.x; ++j) w_begin += live_tiles[j];
        w_end = w_begin + live_tiles[blockIdx.x];
        r_begin = (int)blockIdx.x * RS_BUCKETS; r_end = r_begin + RS_BUCKETS;
    }
    unsigned long long target = batch.barrier_base;
    auto sync_all = [&]() -> bool {
        if (solo) { __syncthreads(); return true; }
        target += gridDim.x;
        return grid_barrier(batch.barrier_ctr, target, batch.err);
    };
    bool ok = true;

    for (int pass = 0; pass < batch.passes && ok; ++pass) {
        const int src = pass & 1, dst = src ^ 1;

        // ---- count: digit histogram of every live tile
        for (int w = w_begin; w < w_end; w += nblk) {
            int jj = 0, t = w;
            while (t >= live_tiles[jj]) { t -= live_tiles[jj]; ++jj; }
            const SortJob& j = batch.job[jj];
            const int64_t n = live_n[jj];
            const int shift = pass * j.width;
            const uint32_t mask = (1u << j.width) - 1u;
            for (int d = threadIdx.x; d < RS_BUCKETS; d += RS_THREADS) base[d] = 0;
            __syncthreads();
            const int64_t tile0 = (int64_t)t * RS_TILE;
            bool bad = false;
#pragma unroll 4
            for (int it = 0; it < RS_ITEMS; ++it) {
                const int64_t i = tile0 + it * RS_THREADS + threadIdx.x;
                if (i < n) {
                    const uint32_t k = load_key(j, pass, i, src);
                    bad |= (k == j.sentinel);
                    atomicAdd(&base[(k >> shift) & mask], 1u);
                }
            }
            if (bad && pass == 0 && j.ids && j.status) atomicOr(j.status, GEAR_DEV_BAD_ID);
            __syncthreads();
            for (int d = threadIdx.x; d <= (int)mask; d += RS_THREADS)
                __stcg(j.hist + (int64_t)d * j.n_tiles + t, base[d]);
            __syncthreads();
        }
        if (!(ok = sync_all())) break;

        // ---- scan: per digit, exclusive scan of the per-tile counts; digit totals.  Jobs of few tiles: one thread per
        //      digit row (its loads are independent, so the rows of all digits cost one trip to the L2 together);
        //      jobs of many tiles: one warp per row.
        constexpr int RS_ROW_THREAD_TILES = 32;
        for (int r = r_begin + blk * RS_THREADS + threadIdx.x; r < r_end; r += nblk * RS_THREADS) {
            const int jj = r / RS_BUCKETS, d = r % RS_BUCKETS;
            const SortJob& j = batch.job[jj];
            const int nt = live_tiles[jj];
            if (d >= (1 << j.width) || nt > RS_ROW_THREAD_TILES) continue;
            uint32_t* row = j.hist + (int64_t)d * j.n_tiles;
            uint32_t carry = 0;
            for (int b0 = 0; b0 < nt; b0 += 8) {
                uint32_t v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q) v[q] = b0 + q < nt ? __ldcg(row + b0 + q) : 0u;
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    if (b0 + q < nt) __stcg(row + b0 + q, carry);
                    carry += v[q];
                }
            }
            __stcg(j.tot + d, carry);
        }
        for (int r = r_begin + blk * (RS_THREADS / 32) + warp; r < r_end; r += nblk * (RS_THREADS / 32)) {
            const int jj = r / RS_BUCKETS, d = r % RS_BUCKETS;
            const SortJob& j = batch.job[jj];
            if (d >= (1 << j.width) || live_tiles[jj] <= RS_ROW_THREAD_TILES) continue;
            uint32_t* row = j.hist + (int64_t)d * j.n_tiles;
            uint32_t carry = 0;
            for (int b0 = 0; b0 < live_tiles[jj]; b0 += 32) {
                const int i = b0 + lane;
                const uint32_t v = i < live_tiles[jj] ? __ldcg(row + i) : 0u;
                const uint32_t inc = warp_inclusive_scan(v);
                if (i < live_tiles[jj]) __stcg(row + i, carry + inc - v);
                carry += __shfl_sync(0xffffffffu, inc, 31);
            }
            if (lane == 0) __stcg(j.tot + d, carry);
        }
        if (!(ok = sync_all())) break;

        // ---- scatter
        for (int w = w_begin; w < w_end; w += nblk) {
            int jj = 0, t = w;
            while (t >= live_tiles[jj]) { t -= live_tiles[jj]; ++jj; }
            const SortJob& j = batch.job[jj];
            const int64_t n = live_n[jj];
            const int64_t tile0 = (int64_t)t * RS_TILE;
            const int shift = pass * j.width;
            const uint32_t mask = (1u << j.width) - 1u;
            {   // where each digit of this tile starts in the output
                uint32_t tot[RS_BUCKETS / RS_THREADS], before[RS_BUCKETS / RS_THREADS];
#pragma unroll
                for (int q = 0; q < RS_BUCKETS / RS_THREADS; ++q) {
                    const int d = threadIdx.x * (RS_BUCKETS / RS_THREADS) + q;     // a thread owns adjacent digits
                    tot[q] = before[q] = 0;
                    if (d <= (int)mask) {
                        tot[q] = __ldcg(j.tot + d);
                        before[q] = __ldcg(j.hist + (int64_t)d * j.n_tiles + t);
                    }
                }
                uint32_t mine = 0;
#pragma unroll
                for (int q = 0; q < RS_BUCKETS / RS_THREADS; ++q) mine += tot[q];
                uint32_t ex = block_exclusive_scan(mine, scratch, nullptr);
#pragma unroll
                for (int q = 0; q < RS_BUCKETS / RS_THREADS; ++q) {
                    base[threadIdx.x * (RS_BUCKETS / RS_THREADS) + q] = ex + before[q];
                    ex += tot[q];
                }
            }
            for (int d = threadIdx.x; d < RS_BUCKETS; d += RS_THREADS)
#pragma unroll
                for (int w2 = 0; w2 < RS_THREADS / 32; ++w2) wcnt[w2][d] = 0;
            __syncthreads();
            uint32_t key[RS_ITEMS], rank[RS_ITEMS];
            const int64_t seg0 = tile0 + (int64_t)warp * (32 * RS_ITEMS);
#pragma unroll
            for (int it = 0; it < RS_ITEMS; ++it) {
                const int64_t i = seg0 + it * 32 + lane;
                key[it] = i < n ? load_key(j, pass, i, src) : 0u;
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
            for (int d = threadIdx.x; d < RS_BUCKETS; d += RS_THREADS) {
                uint32_t run = 0;
#pragma unroll
                for (int w2 = 0; w2 < RS_THREADS / 32; ++w2) {
                    const uint32_t c = wcnt[w2][d];
                    wcnt[w2][d] = run;
                    run += c;
                }
            }
            __syncthreads();
            const bool identity = (pass == 0 && j.identity_vals);
#pragma unroll
            for (int it = 0; it < RS_ITEMS; ++it) {
                const int64_t i = seg0 + it * 32 + lane;
                if (i < n) {
                    const uint32_t d = (key[it] >> shift) & mask;
                    const uint32_t pos = base[d] + wcnt[warp][d] + rank[it];
                    __stcg(j.keys[dst] + pos, key[it]);
                    __stcg(j.vals[dst] + pos, identity ? (uint32_t)i : __ldcg(j.vals[src] + i));
                }
            }
            __syncthreads();
        }
        if (pass + 1 < batch.passes && !(ok = sync_all())) break;
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
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, coop_sort_kernel, RS_THREADS, 0);
        if (sms <= 0) sms = 148;
        if (per_sm <= 0) per_sm = 1;
        if (per_sm > 3) per_sm = 3;
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
    }
    batch.passes = passes;
    int grid = total_tiles < coop_grid_limit() ? total_tiles : coop_grid_limit();
    if (grid < 1) grid = 1;
    batch.n_barriers = 3 * passes - 1;
    batch.barrier_ctr = gbs->device_counter;
    batch.barrier_base = gbs->host_base;
    gbs->host_base += (unsigned long long)grid * (unsigned long long)batch.n_barriers;
    KernelScope k(prof, batch.name ? batch.name : "coop_sort", st);
    void* args[] = {&batch};
    *err_out = cudaLaunchCooperativeKernel((const void*)coop_sort_kernel, dim3(grid), dim3(RS_THREADS), args, 0, st);
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
