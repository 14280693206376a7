// Inference-expired time (Section 1, second point; Section 3: the workers drop expired inference
// results continuously): list every image whose cached DFV is older than the expiry time.
//
// Three launches, none waits on another block:
//   mark   streams the int64 timestamp table once (the only HBM-sized traffic: 8 bytes per image),
//          evaluates now - ts >= expire, packs the predicate 32 entries to a word with a warp ballot and
//          counts per tile;
//   scan   one block scans the tile counts and checks the caller's capacity;
//   write  re-reads only the bitmap (1 bit per image), ranks the set bits with popc + block scan
//          and writes the ascending ID list; listed entries are restamped on request.
#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int EXP_THREADS = 256;
static_assert(EXP_TILE == EXP_THREADS * 32, "one bitmap word per thread in the write pass");

__global__ void __launch_bounds__(EXP_THREADS)
expiry_mark_kernel(const int64_t* __restrict__ ts, int64_t vocab, int64_t now, int64_t expire,
                   uint32_t* __restrict__ bits, uint2* __restrict__ tile_cnt) {
    __shared__ uint32_t scratch[33];
    const int64_t tile0 = (int64_t)blockIdx.x * EXP_TILE;
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    uint32_t count = 0;
#pragma unroll 8
    for (int it = 0; it < EXP_TILE / EXP_THREADS; ++it) {
        const int64_t i = tile0 + (int64_t)it * EXP_THREADS + threadIdx.x;
        bool expired = false;
        if (i < vocab) {
            int64_t t;
            asm volatile("ld.global.nc.L1::no_allocate.s64 %0, [%1];" : "=l"(t) : "l"(ts + i));
            expired = now - t >= expire;
        }
        const uint32_t word = __ballot_sync(0xffffffffu, expired);
        if (lane == 0) {
            const int64_t w = (tile0 + (int64_t)it * EXP_THREADS) / 32 + warp;
            if (w * 32 < vocab) bits[w] = word;
            count += __popc(word);
        }
    }
    uint32_t total;
    block_exclusive_scan(count, scratch, &total);
    if (threadIdx.x == 0) tile_cnt[blockIdx.x] = make_uint2(total, 0u);
}

__global__ void expiry_check_kernel(const uint2* __restrict__ tile_cnt, int64_t n_tiles, int64_t cap,
                                    int64_t* __restrict__ d_n, DevState* __restrict__ state) {
    const int64_t total = tile_cnt[n_tiles].x;
    if (d_n) *d_n = total;
    if (total > cap) { atomicOr(&state->status, GEAR_DEV_OUT_CAPACITY); state->exp_total = -1; }
    else state->exp_total = total;
}

__global__ void __launch_bounds__(EXP_THREADS)
expiry_write_kernel(const uint32_t* __restrict__ bits, int64_t vocab, const uint2* __restrict__ tile_cnt,
                    const DevState* __restrict__ state, int64_t now, int restamp, int64_t* __restrict__ ts,
                    int32_t* __restrict__ ids) {
    __shared__ uint32_t scratch[33];
    if (state->exp_total < 0) return;                       // capacity too small: nothing listed, nothing restamped
    const int64_t w = (int64_t)blockIdx.x * EXP_THREADS + threadIdx.x;
    uint32_t word = (w * 32 < vocab) ? bits[w] : 0u;
    const uint32_t ex = block_exclusive_scan(__popc(word), scratch, nullptr);
    int64_t out = (int64_t)tile_cnt[blockIdx.x].x + ex;
    while (word) {
        const int bit = __ffs(word) - 1;
        word &= word - 1;
        const int64_t id = w * 32 + bit;
        ids[out++] = (int32_t)id;
        if (restamp) ts[id] = now;
    }
}

cudaError_t launch_collect_expired(const gear_ctx_impl& c, int64_t now, int restamp, int32_t* ids, int64_t cap,
                                   int64_t* d_n, cudaStream_t st) {
    const int64_t vocab = c.cfg.img_vocab;
    const int64_t n_tiles = ceil_div(vocab, EXP_TILE);
    uint32_t* bits = c.at<uint32_t>(c.ws.exp_bits);
    uint2* tile_cnt = c.at<uint2>(c.ws.exp_cnt);
    { KernelScope k(&c.prof, "expiry_mark", st);
    expiry_mark_kernel<<<(unsigned)n_tiles, EXP_THREADS, 0, st>>>(c.buf.dfv_ts, vocab, now, c.cfg.expire, bits, tile_cnt); }
    scan_pairs(tile_cnt, n_tiles, tile_cnt + n_tiles, st, &c.prof);
    { KernelScope k(&c.prof, "expiry_check", st);
    expiry_check_kernel<<<1, 1, 0, st>>>(tile_cnt, n_tiles, cap, d_n, c.state()); }
    { KernelScope k(&c.prof, "expiry_write", st);
    expiry_write_kernel<<<(unsigned)n_tiles, EXP_THREADS, 0, st>>>(bits, vocab, tile_cnt, c.state(), now, restamp,
                                                                  c.buf.dfv_ts, ids); }
    return cudaGetLastError();
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
constexpr size_t STATIC_CNT_BYTES = ((size_t)(STATIC_MAX_VOCAB / EXP_TILE) + 1) * sizeof(uint2);
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
    const int64_t n_tiles = ceil_div(img_vocab, EXP_TILE);

    // the array keeps what the previous call left: the state block has to start from zero, the bitmap words
    // and tile counts of this table size are all rewritten by the mark pass
    if (cudaMemsetAsync(state, 0, STATIC_STATE_BYTES, st) != cudaSuccess) return GEAR_ERR_CUDA;
    expiry_mark_kernel<<<(unsigned)n_tiles, EXP_THREADS, 0, st>>>(dfv_ts, img_vocab, now, expire, bits, tile_cnt);
    scan_pairs(tile_cnt, n_tiles, tile_cnt + n_tiles, st, nullptr);
    int64_t* d_cnt = d_n ? d_n : &state->pad[1];
    expiry_check_kernel<<<1, 1, 0, st>>>(tile_cnt, n_tiles, cap, d_cnt, state);
    expiry_write_kernel<<<(unsigned)n_tiles, EXP_THREADS, 0, st>>>(bits, img_vocab, tile_cnt, state, now, restamp, dfv_ts, ids);
    if (cudaGetLastError() != cudaSuccess) return GEAR_ERR_CUDA;
    if (h_n) {
        if (cudaMemcpyAsync(h_n, d_cnt, sizeof(int64_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return GEAR_ERR_CUDA;
        if (*h_n > cap) return GEAR_ERR_CAPACITY;
    }
    return GEAR_OK;
}
