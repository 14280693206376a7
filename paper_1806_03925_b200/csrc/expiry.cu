// Inference-expired time (Section 1, second point; Section 3: the workers drop expired inference
// results continuously): list every image whose cached DFV is older than the expiry time.
//
// Three launches, none waits on another block:
//   mark   streams the int64 timestamp table once (the only HBM-sized traffic: 8 bytes per image),
//          evaluates now - ts >= expire, packs the predicate 32 entries to a word with a warp ballot and
//          counts per 2048-entry tile;
//   scan   one block scans the tile counts;
//   write  checks the caller's capacity, re-reads only the bitmap (1 bit per image), ranks the set bits
//          with popc + block scan and writes the ascending ID list; listed entries are restamped on request.
#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int EXP_THREADS = 256;
constexpr int EXP_MARK_ITEMS = EXP_MARK_TILE / EXP_THREADS;
static_assert(EXP_TILE == EXP_THREADS * 32, "one bitmap word per thread in the write pass");
static_assert(EXP_MARK_TILE % (EXP_THREADS * 1) == 0 && EXP_TILE % EXP_MARK_TILE == 0, "mark tiles nest in write tiles");

// One block per EXP_MARK_TILE timestamps.  All of a thread's loads are issued before the first ballot, so a
// block keeps its whole 16 KB tile in flight; the small tiles leave the balancing to the block scheduler.
__global__ void __launch_bounds__(EXP_THREADS)
expiry_mark_kernel(const int64_t* __restrict__ ts, int64_t vocab, int64_t now, int64_t expire,
                   uint32_t* __restrict__ bits, uint2* __restrict__ tile_cnt) {
    wait_for_predecessor();
    __shared__ uint32_t warp_cnt[EXP_THREADS / 32];
    const int64_t tile0 = (int64_t)blockIdx.x * EXP_MARK_TILE;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    int64_t t[EXP_MARK_ITEMS];
#pragma unroll
    for (int it = 0; it < EXP_MARK_ITEMS; ++it) {
        const int64_t i = tile0 + (int64_t)it * EXP_THREADS + threadIdx.x;
        t[it] = i < vocab ? __ldcs(reinterpret_cast<const long long*>(ts) + i) : 0;
    }
    uint32_t count = 0;
#pragma unroll
    for (int it = 0; it < EXP_MARK_ITEMS; ++it) {
        const int64_t i = tile0 + (int64_t)it * EXP_THREADS + threadIdx.x;
        const bool expired = i < vocab && now - t[it] >= expire;
        const uint32_t word = __ballot_sync(0xffffffffu, expired);
        if (lane == 0) {
            const int64_t w = (tile0 + (int64_t)it * EXP_THREADS) / 32 + warp;
            if (w * 32 < vocab) bits[w] = word;
            count += __popc(word);
        }
    }
    if (lane == 0) warp_cnt[warp] = count;
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t total = 0;
#pragma unroll
        for (int w = 0; w < EXP_THREADS / 32; ++w) total += warp_cnt[w];
        tile_cnt[blockIdx.x] = make_uint2(total, 0u);
    }
}

// One block per EXP_TILE entries: re-reads the bitmap only.  Every block compares the total with the
// caller's capacity itself; block 0 reports the count and raises the status bit.
__global__ void __launch_bounds__(EXP_THREADS)
expiry_write_kernel(const uint32_t* __restrict__ bits, int64_t vocab, const uint2* __restrict__ tile_cnt,
                    int64_t n_mark_tiles, int64_t cap, int64_t* __restrict__ d_n, DevState* __restrict__ state,
                    int64_t now, int restamp, int64_t* __restrict__ ts, int32_t* __restrict__ ids) {
    wait_for_predecessor();
    __shared__ uint32_t scratch[33];
    const int64_t total = tile_cnt[n_mark_tiles].x;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (d_n) *d_n = total;
        state->exp_total = total > cap ? -1 : total;
        if (total > cap) atomicOr(&state->status, GEAR_DEV_OUT_CAPACITY);
    }
    if (total > cap) return;                                // capacity too small: nothing listed, nothing restamped
    const int64_t w = (int64_t)blockIdx.x * EXP_THREADS + threadIdx.x;
    uint32_t word = (w * 32 < vocab) ? bits[w] : 0u;
    const uint32_t ex = block_exclusive_scan(__popc(word), scratch, nullptr);
    int64_t out = (int64_t)tile_cnt[(int64_t)blockIdx.x * (EXP_TILE / EXP_MARK_TILE)].x + ex;
    while (word) {
        const int bit = __ffs(word) - 1;
        word &= word - 1;
        const int64_t id = w * 32 + bit;
        ids[out++] = (int32_t)id;
        if (restamp) ts[id] = now;
    }
}

// The three launches of one scan over scratch (bits, tile_cnt, state).  prof may be null.
static cudaError_t enqueue_expiry_scan(int64_t* ts, int64_t vocab, int64_t expire, int64_t now, int restamp,
                                       int32_t* ids, int64_t cap, int64_t* d_n, uint32_t* bits, uint2* tile_cnt,
                                       DevState* state, Profiler* prof, cudaStream_t st) {
    const int64_t n_mark = ceil_div(vocab, EXP_MARK_TILE), n_write = ceil_div(vocab, EXP_TILE);
    { KernelScope k(prof, "expiry_mark", st);
    launch_dependent(expiry_mark_kernel, dim3((unsigned)n_mark), dim3(EXP_THREADS), 0, st, ts, vocab, now, expire, bits, tile_cnt); }
    scan_pairs(tile_cnt, n_mark, tile_cnt + n_mark, st, prof);
    { KernelScope k(prof, "expiry_write", st);
    launch_dependent(expiry_write_kernel, dim3((unsigned)n_write), dim3(EXP_THREADS), 0, st, bits, vocab, tile_cnt, n_mark, cap, d_n, state, now,
                                                                  restamp, ts, ids); }
    return cudaGetLastError();
}

cudaError_t launch_collect_expired(const gear_ctx_impl& c, int64_t now, int restamp, int32_t* ids, int64_t cap,
                                   int64_t* d_n, cudaStream_t st) {
    return enqueue_expiry_scan(c.buf.dfv_ts, c.cfg.img_vocab, c.cfg.expire, now, restamp, ids, cap, d_n,
                               c.at<uint32_t>(c.ws.exp_bits), c.at<uint2>(c.ws.exp_cnt), c.state(), &c.prof, st);
}

}  // namespace gear

// ---------------------------------------------------------------------------------------------------
// gear_collect_expired_static: the same scan for callers that cannot allocate device memory.
//
// Some hosts of this library run it where cudaMalloc is off limits: inside a serving process whose memory
// pool was carved up at start-up and is policed, from a plug-in that is handed buffers but no allocator,
// or on a path that must not touch the allocator because an allocation may synchronise the device.  Such a
// caller cannot provide the workspace a gear_ctx needs.  This entry point therefore keeps the scan's
// scratch (expired bitmap, per-tile counts, a small state block) in a fixed array that is part of the
// library image: every GPU that loads libgear holds GEAR_STATIC_EXPIRY_SCRATCH_BYTES of it until the
// process exits.  The price is a bound on the table size and one shared scratch per device.
// ---------------------------------------------------------------------------------------------------
#include <mutex>

namespace gear {

constexpr int64_t STATIC_MAX_VOCAB = GEAR_STATIC_EXPIRY_MAX_VOCAB;
constexpr size_t STATIC_STATE_BYTES = 256;
constexpr size_t STATIC_BITS_BYTES = (size_t)(STATIC_MAX_VOCAB / 32) * 4;
constexpr size_t STATIC_CNT_BYTES = ((size_t)(STATIC_MAX_VOCAB / EXP_MARK_TILE) + 1) * sizeof(uint2);
constexpr size_t STATIC_SCRATCH_BYTES = STATIC_STATE_BYTES + STATIC_BITS_BYTES + ((STATIC_CNT_BYTES + 255) / 256) * 256;
static_assert(sizeof(DevState) <= STATIC_STATE_BYTES, "state block");
static_assert(STATIC_SCRATCH_BYTES == GEAR_STATIC_EXPIRY_SCRATCH_BYTES, "the header states the size of the array");

// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_expiry_scratch[STATIC_SCRATCH_BYTES];

constexpr int STATIC_MAX_DEVICES = 64;
static std::mutex g_static_mutex;
static unsigned char* g_static_ptr[STATIC_MAX_DEVICES];     // device address of the scratch, per device ordinal

// Device address of the scratch on the current device (looked up once per device).
static cudaError_t static_scratch(unsigned char** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= STATIC_MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_expiry_scratch);
        if (e != cudaSuccess) return e;
        g_static_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}

}  // namespace gear

extern "C" int gear_collect_expired_static(int64_t* dfv_ts, int64_t img_vocab, int64_t expire, int64_t now, int restamp,
                                           int32_t* ids, int64_t cap, int64_t* d_n, int64_t* h_n, void* stream) {
    using namespace gear;
    if (!dfv_ts || img_vocab < 1 || expire < 0 || cap < 0 || (cap > 0 && !ids)) return GEAR_ERR_ARG;
    if (img_vocab > STATIC_MAX_VOCAB) return GEAR_ERR_CAPACITY;      // the fixed scratch cannot hold the bitmap
    unsigned char* base = nullptr;
    if (static_scratch(&base) != cudaSuccess) return GEAR_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    DevState* state = reinterpret_cast<DevState*>(base);
    uint32_t* bits = reinterpret_cast<uint32_t*>(base + STATIC_STATE_BYTES);
    uint2* tile_cnt = reinterpret_cast<uint2*>(base + STATIC_STATE_BYTES + STATIC_BITS_BYTES);

    // the array keeps what the previous call left: the state block has to start from zero, the bitmap words
    // and tile counts of this table size are all rewritten by the mark pass
    if (cudaMemsetAsync(state, 0, STATIC_STATE_BYTES, st) != cudaSuccess) return GEAR_ERR_CUDA;
    int64_t* d_cnt = d_n ? d_n : &state->pad[1];
    if (enqueue_expiry_scan(dfv_ts, img_vocab, expire, now, restamp, ids, cap, d_cnt, bits, tile_cnt, state, nullptr, st) !=
        cudaSuccess)
        return GEAR_ERR_CUDA;
    if (h_n) {
        if (cudaMemcpyAsync(h_n, d_cnt, sizeof(int64_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return GEAR_ERR_CUDA;
        if (*h_n > cap) return GEAR_ERR_CAPACITY;
    }
    return GEAR_OK;
}
