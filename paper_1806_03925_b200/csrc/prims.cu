// Stable LSD radix sort of (key, value) pairs and small scan helpers.
//
// Every pass is three kernels -- per-tile digit histogram, per-digit scan over tiles, stable scatter --
// so no kernel ever waits on another block.  A tile is RS_TILE consecutive elements; a warp owns
// 32 * RS_ITEMS consecutive elements of it and ranks equal digits with match_any, which keeps equal keys
// in index order.
#include "common.cuh"

namespace gear {

__device__ __forceinline__ int64_t effective_n(int64_t n_max, const int64_t* n_dev) {
    if (!n_dev) return n_max;
    int64_t n = *n_dev;
    return n < n_max ? (n < 0 ? 0 : n) : n_max;
}

__global__ void __launch_bounds__(RS_THREADS)
radix_hist_kernel(const uint32_t* __restrict__ keys, int64_t n_max, const int64_t* __restrict__ n_dev,
                  int shift, uint32_t mask, uint32_t* __restrict__ hist, int n_tiles) {
    __shared__ uint32_t h[RS_BUCKETS];
    const int64_t n = effective_n(n_max, n_dev);
    h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * RS_TILE;
#pragma unroll 4
    for (int it = 0; it < RS_ITEMS; ++it) {
        int64_t i = base + it * RS_THREADS + threadIdx.x;
        if (i < n) atomicAdd(&h[(keys[i] >> shift) & mask], 1u);
    }
    __syncthreads();
    hist[(int64_t)threadIdx.x * n_tiles + blockIdx.x] = h[threadIdx.x];
}

// One block per digit: exclusive scan of that digit's per-tile counts; the digit total goes to tot[d].
__global__ void __launch_bounds__(RS_THREADS)
radix_scan_rows_kernel(uint32_t* __restrict__ hist, uint32_t* __restrict__ tot, int n_tiles) {
    __shared__ uint32_t scratch[33];
    uint32_t* row = hist + (int64_t)blockIdx.x * n_tiles;
    uint32_t carry = 0;
    for (int base = 0; base < n_tiles; base += RS_THREADS) {
        int i = base + threadIdx.x;
        uint32_t v = i < n_tiles ? row[i] : 0u;
        uint32_t total;
        uint32_t ex = block_exclusive_scan(v, scratch, &total);
        if (i < n_tiles) row[i] = carry + ex;
        carry += total;
    }
    if (threadIdx.x == 0) tot[blockIdx.x] = carry;
}

__global__ void __launch_bounds__(RS_THREADS)
radix_scatter_kernel(const uint32_t* __restrict__ kin, const uint32_t* __restrict__ vin,
                     uint32_t* __restrict__ kout, uint32_t* __restrict__ vout,
                     int64_t n_max, const int64_t* __restrict__ n_dev, int shift, uint32_t mask,
                     const uint32_t* __restrict__ hist, const uint32_t* __restrict__ tot, int n_tiles) {
    __shared__ uint32_t scratch[33];
    __shared__ uint32_t base[RS_BUCKETS];
    __shared__ uint32_t wcnt[RS_THREADS / 32][RS_BUCKETS];
    const int64_t n = effective_n(n_max, n_dev);
    const int64_t tile0 = (int64_t)blockIdx.x * RS_TILE;
    if (tile0 >= n) return;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;

    {   // global start of every digit, plus what earlier tiles put into it
        uint32_t t = tot[threadIdx.x];
        uint32_t ex = block_exclusive_scan(t, scratch, nullptr);
        base[threadIdx.x] = ex + hist[(int64_t)threadIdx.x * n_tiles + blockIdx.x];
    }
    for (int w = 0; w < RS_THREADS / 32; ++w) wcnt[w][threadIdx.x] = 0;
    __syncthreads();

    uint32_t key[RS_ITEMS], rank[RS_ITEMS];
    const int64_t seg0 = tile0 + (int64_t)warp * (32 * RS_ITEMS);
#pragma unroll
    for (int it = 0; it < RS_ITEMS; ++it) {
        int64_t i = seg0 + it * 32 + lane;
        key[it] = i < n ? kin[i] : 0u;
    }
#pragma unroll
    for (int it = 0; it < RS_ITEMS; ++it) {
        int64_t i = seg0 + it * 32 + lane;
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
    {   // turn the per-warp digit counts into exclusive offsets across the warps of this tile
        uint32_t run = 0;
#pragma unroll
        for (int w = 0; w < RS_THREADS / 32; ++w) {
            uint32_t c = wcnt[w][threadIdx.x];
            wcnt[w][threadIdx.x] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int it = 0; it < RS_ITEMS; ++it) {
        int64_t i = seg0 + it * 32 + lane;
        if (i < n) {
            const uint32_t d = (key[it] >> shift) & mask;
            const uint32_t pos = base[d] + wcnt[warp][d] + rank[it];
            kout[pos] = key[it];
            vout[pos] = vin ? vin[i] : (uint32_t)i;
        }
    }
}

int radix_sort_pairs(const SortBufs& b, int64_t n_max, const int64_t* n_dev, int bits, bool identity_vals,
                     cudaStream_t st, Profiler* prof) {
    if (n_max <= 0) return 0;
    const int n_tiles = (int)sort_tiles(n_max);
    const int passes = (bits + 7) / 8;
    const int width = (bits + passes - 1) / passes;
    int cur = 0;
    for (int p = 0; p < passes; ++p) {
        const int shift = p * width;
        const uint32_t mask = (1u << width) - 1u;
        { KernelScope k(prof, "radix_hist", st);
        radix_hist_kernel<<<n_tiles, RS_THREADS, 0, st>>>(b.keys[cur], n_max, n_dev, shift, mask, b.hist, n_tiles); }
        { KernelScope k(prof, "radix_scan_rows", st);
        radix_scan_rows_kernel<<<RS_BUCKETS, RS_THREADS, 0, st>>>(b.hist, b.tot, n_tiles); }
        const uint32_t* vin = (p == 0 && identity_vals) ? nullptr : b.vals[cur];
        { KernelScope k(prof, "radix_scatter", st);
        radix_scatter_kernel<<<n_tiles, RS_THREADS, 0, st>>>(b.keys[cur], vin, b.keys[cur ^ 1], b.vals[cur ^ 1],
                                                             n_max, n_dev, shift, mask, b.hist, b.tot, n_tiles); }
        cur ^= 1;
    }
    return cur;
}

// ---------------------------------------------------------------- scan of counter pairs
__global__ void __launch_bounds__(1024)
scan_pairs_kernel(uint2* __restrict__ data, int64_t m, uint2* __restrict__ total) {
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
    scan_pairs_kernel<<<1, 1024, 0, st>>>(data, m, total);
}

}  // namespace gear
