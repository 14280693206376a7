// Shared device helpers and the internal host-side declarations of libgear.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/gear.h"

namespace gear {

// ---------------------------------------------------------------- device state
// Lives at the start of the workspace.  Counters are device-resident so that no
// call has to synchronise to learn a size produced by an earlier kernel.
struct DevState {
    int32_t status;        // GEAR_DEV_* bits, sticky
    int32_t tc_error;      // non-zero: a bounded wait of the tensor-core head gave up (code of the wait)
    int64_t q_count;       // averages waiting in the ready queue
    int64_t n_valid;       // accumulate: rows with an in-range ID (sorted prefix length)
    int64_t direct_done;   // accumulate + collect as one call: 1 while the hand-over pass that follows has nothing to do
                           // (the reduce pass wrote the averages straight into the caller's lists)
    int64_t n_complete;    // accumulate: groups of this call that reached M
    int64_t exp_total;     // expiry scan: entries found
    int64_t collect_n;     // collect_ready: entries moved by the running call
    unsigned long long grid_barrier;   // arrival counter of the cooperative sort's grid barrier
    unsigned int colsum_ticket;        // blocks of head_out_kernel that have delivered their partial loss (wraps to 0)
    unsigned int pad32;                // blocks of a solo collect_move_kernel that have finished (wraps to 0)
    int64_t q_calls;       // accumulate calls that added to the ready queue since the last collect
    int64_t sort_n;        // collect_ready: entries the queue sort has to order (0: the queue is already in order)
    int64_t pad[5];
};
static_assert(sizeof(DevState) == 128, "DevState layout");

// ---------------------------------------------------------------- small helpers
__host__ __device__ inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// SMs of the current device (host side; 148 on a B200)
inline int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

__device__ __forceinline__ unsigned lane_id() { return threadIdx.x & 31u; }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ uint32_t warp_inclusive_scan(uint32_t v) {
    const unsigned lane = lane_id();
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= (unsigned)o) v += t;
    }
    return v;
}

// Exclusive scan over the threads of a block (blockDim.x a multiple of 32, <= 1024).
// `scratch` needs 33 words of shared memory.  Returns the exclusive prefix; *total gets the block sum.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* scratch, uint32_t* total) {
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    uint32_t inc = warp_inclusive_scan(v);
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t w = lane < nwarp ? scratch[lane] : 0u;
        uint32_t winc = warp_inclusive_scan(w);
        scratch[lane] = winc - w;
        if (lane == 31) scratch[32] = winc;
    }
    __syncthreads();
    uint32_t res = scratch[warp] + inc - v;
    if (total) *total = scratch[32];
    __syncthreads();
    return res;
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float((uint32_t)b << 16); }

__device__ __forceinline__ float4 ld_f4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ void st_f4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }

// 128-bit load that does not allocate in L1 (streamed data read once)
__device__ __forceinline__ float4 ld_stream_f4(const float* p) {
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// vector reduction: *p += v without a return value (sm_90+)
__device__ __forceinline__ void red_add_f4(float* p, float4 v) {
    asm volatile("red.global.add.v4.f32 [%0], {%1,%2,%3,%4};"
                 :: "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// L2 eviction priorities: data that is read again soon is kept (evict_last), data touched once is let go first
// (evict_first), so that a streamed table does not push a reused matrix out of the L2.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void st_f4_hint(float* p, float4 v, uint64_t policy) {
    asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1,%2,%3,%4}, %5;"
                 :: "l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "l"(policy) : "memory");
}

// 16-byte asynchronous copy global -> shared; src_bytes = 0 reads nothing and fills the 16 bytes with zeros
__device__ __forceinline__ void cp_async_16(uint32_t smem_dst, const void* gsrc, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" :: "r"(smem_dst), "l"(gsrc), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" :: "n"(N) : "memory");
}

// ---------------------------------------------------------------- programmatic dependent launch
// The step is a chain of two dozen short kernels on one stream.  Launched this way, the blocks of a kernel may be
// set up on SMs that the previous kernel in the stream has already left while its last blocks still run; every
// such kernel calls wait_for_predecessor() before it touches memory, which returns once the previous kernel has
// completed and its writes are visible.  That takes the launch latency out of the gaps between kernels.  Every
// block of such a kernel must make the call, first thing, or the chain of completions would break.
__device__ __forceinline__ void wait_for_predecessor() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---------------------------------------------------------------- launch accounting / per-kernel timing
// Every kernel launch of the library goes through a KernelScope: it counts the launch and, when profiling
// is on, brackets it with a pair of CUDA events on the caller's stream (read back by gear_profile_read).
struct Profiler {
    struct Rec { const char* name; cudaEvent_t start, stop; };
    bool on = false;
    bool keep_streams = false;     // timeline mode: events are recorded but the library keeps its side stream
    int64_t launches = 0;
    std::vector<Rec> recs;
    std::vector<cudaEvent_t> pool;
    cudaEvent_t get() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
    void clear() {
        for (auto& r : recs) { pool.push_back(r.start); pool.push_back(r.stop); }
        recs.clear();
    }
    ~Profiler() {
        clear();
        for (auto e : pool) cudaEventDestroy(e);
    }
};

struct KernelScope {
    Profiler* p; cudaStream_t st; cudaEvent_t stop = nullptr;
    KernelScope(Profiler* prof, const char* name, cudaStream_t s) : p(prof), st(s) {
        if (!p) return;
        ++p->launches;
        if (p->on) {
            Profiler::Rec r{name, p->get(), p->get()};
            stop = r.stop;
            cudaEventRecord(r.start, st);
            p->recs.push_back(r);
        }
    }
    ~KernelScope() { if (stop) cudaEventRecord(stop, st); }
};

// sorted positions per unit of work of the accumulate's reduce pass (at most 32); the workspace holds one word per span
constexpr int ACC_SPAN = 16;

// ---------------------------------------------------------------- radix sort / scans (prims.cu)
constexpr int RS_THREADS = 256;
constexpr int RS_ITEMS = 16;
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;
constexpr int RS_RADIX_BITS = 9;
constexpr int RS_BUCKETS = 1 << RS_RADIX_BITS;
constexpr int RS_MAX_PASSES = 4;          // 32-bit keys in digits of 9 bits

inline int64_t sort_tiles(int64_t n_max) { return n_max > 0 ? ceil_div(n_max, RS_TILE) : 1; }

// One array to sort: (key, value) pairs ordered by the low `bits` bits of the key, equal keys in input order.
struct SortJob {
    const int32_t* ids;     // if set, pass 0 reads these: key = id if 0 <= id < sentinel, else sentinel
    uint32_t sentinel;      // key of out-of-range IDs (sorts last when bits covers it)
    int32_t* status;        // device status word that gets GEAR_DEV_BAD_ID when a sentinel key is met (may be null)
    uint32_t* keys[2];      // without ids the input keys are keys[0]
    uint32_t* vals[2];      // with identity_vals the value of element i is i, else vals[0][i]
    uint32_t* hist;         // [RS_MAX_PASSES][n_tiles][RS_BUCKETS] tile descriptors: per pass and tile, how many of the
                            // tile's elements (or of all tiles up to it) carry each digit; top two bits say which
    uint32_t* tot;          // [RS_MAX_PASSES][RS_BUCKETS] digit histogram of every pass
    int64_t n_max;          // element count (or its upper bound when n_dev is given)
    const int64_t* n_dev;   // optional device-resident count, capped at n_max
    int bits;
    int identity_vals;
    int width, n_tiles;     // filled in by sort_jobs
};

struct SortBatch {
    SortJob job[3];
    int n_jobs;
    const char* name;                 // host only: the name the launch is timed under
    int passes, n_barriers;           // filled in by sort_jobs
    unsigned long long* barrier_ctr;  // filled in by sort_jobs
    unsigned long long barrier_base;
    int32_t* err;                     // device word that receives a non-zero code when a grid barrier gives up
};

// Arrival counter of the grid barrier (device) and what all launches so far will have added to it (host).
struct GridBarrierState {
    unsigned long long* device_counter;
    unsigned long long host_base;
};

// Sorts every job of the batch in one cooperative launch.  Returns the index (0 or 1) of the keys/vals
// buffer pair that holds the sorted result of every job.
int sort_jobs(SortBatch& batch, GridBarrierState* gbs, cudaStream_t st, Profiler* prof, cudaError_t* err_out);

// In-place exclusive scan of m (a, b) counter pairs by one block; the totals go to total[0..1].
void scan_pairs(uint2* data, int64_t m, uint2* total, cudaStream_t st, Profiler* prof);

inline int bits_for(int64_t max_key_inclusive) {
    int b = 1;
    while (b < 32 && (int64_t(1) << b) <= max_key_inclusive) ++b;
    return b;
}

}  // namespace gear
