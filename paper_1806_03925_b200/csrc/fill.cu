// Procedural table fill: counter-based SplitMix64 streams, one draw per element, so any element can be
// regenerated without the rest of the table.  Pure streaming writes (HBM write bound).
#include "common.cuh"
#include "internal.h"

namespace gear {

__host__ __device__ __forceinline__ uint64_t mix64(uint64_t z) {
    z ^= z >> 30; z *= 0xbf58476d1ce4e5b9ull;
    z ^= z >> 27; z *= 0x94d049bb133111ebull;
    z ^= z >> 31;
    return z;
}
constexpr uint64_t kGamma = 0x9e3779b97f4a7c15ull;

__host__ __device__ __forceinline__ uint64_t stream_key(uint64_t seed, uint64_t tag) {
    return mix64(seed + kGamma * (tag + 1));
}
__device__ __forceinline__ uint64_t draw(uint64_t key, uint64_t idx) { return mix64(key + kGamma * (idx + 1)); }

__device__ __forceinline__ float grid_value(uint64_t key, uint64_t idx, float step) {
    const int32_t k = (int32_t)(draw(key, idx) >> 40) - 8388608;
    return __fmul_rn((float)k, step);
}

// each thread writes 16 bytes: 4 floats or 8 bf16
template <bool BF16>
__global__ void __launch_bounds__(256)
fill_uniform_kernel(void* __restrict__ dst, int64_t n_elems, uint64_t key, float step) {
    constexpr int PER = BF16 ? 8 : 4;
    const int64_t n_chunks = (n_elems + PER - 1) / PER;
    for (int64_t ch = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; ch < n_chunks;
         ch += (int64_t)gridDim.x * blockDim.x) {
        const int64_t e0 = ch * PER;
        float v[PER];
#pragma unroll
        for (int k = 0; k < PER; ++k) v[k] = grid_value(key, (uint64_t)(e0 + k), step);
        if (e0 + PER <= n_elems) {
            if (BF16) {
                uint4 pk;
                uint32_t* w = reinterpret_cast<uint32_t*>(&pk);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
                    w[k] = *reinterpret_cast<uint32_t*>(&h);
                }
                reinterpret_cast<uint4*>(dst)[ch] = pk;
            } else {
                reinterpret_cast<float4*>(dst)[ch] = make_float4(v[0], v[1], v[2], v[3]);
            }
        } else {
            for (int k = 0; e0 + k < n_elems; ++k) {
                if (BF16) reinterpret_cast<__nv_bfloat16*>(dst)[e0 + k] = __float2bfloat16_rn(v[k]);
                else reinterpret_cast<float*>(dst)[e0 + k] = v[k];
            }
        }
    }
}

__global__ void __launch_bounds__(256)
fill_ts_kernel(int64_t* __restrict__ ts, int64_t n, uint64_t key, uint64_t span, int64_t now) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        ts[i] = now - (int64_t)(draw(key, (uint64_t)i) % span);
}

static int grid_for(int64_t work_items) {
    int64_t blocks = ceil_div(work_items, 256);
    const int64_t cap = 148 * 16;
    return (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

cudaError_t launch_fill_uniform(void* dst, int dtype, int64_t n_elems, uint64_t seed, uint64_t tag, double amp,
                                cudaStream_t st) {
    if (n_elems <= 0) return cudaSuccess;
    const float step = (float)(amp / 8388608.0);
    const uint64_t key = stream_key(seed, tag);
    if (dtype == GEAR_BF16)
        fill_uniform_kernel<true><<<grid_for(ceil_div(n_elems, 8)), 256, 0, st>>>(dst, n_elems, key, step);
    else
        fill_uniform_kernel<false><<<grid_for(ceil_div(n_elems, 4)), 256, 0, st>>>(dst, n_elems, key, step);
    return cudaGetLastError();
}

cudaError_t launch_fill_ts(int64_t* ts, int64_t n, uint64_t seed, int64_t expire, int64_t now, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const uint64_t span = expire > 1 ? (uint64_t)expire : 1u;
    fill_ts_kernel<<<grid_for(n), 256, 0, st>>>(ts, n, stream_key(seed, GEAR_TAG_TS), span, now);
    return cudaGetLastError();
}

}  // namespace gear
