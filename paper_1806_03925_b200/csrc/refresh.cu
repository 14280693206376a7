// Refresh of cached inference results (Section 1, second point; Section 3: a Dense Feature Vector whose cached
// copy has expired is computed again): the new vectors replace the cached rows and restart their clocks.
//
// A warp takes four refreshed images per pass.  A lane owns 16-byte chunks of the table row: for a bf16 table it
// reads 32 bytes of the fp32 source row, rounds to nearest even and writes 16 bytes; for an fp32 table it copies
// 16 bytes.  The loads of the four rows are issued before the first store.  HBM bound: n * D * (4 + sizeof(dfv)) bytes
// plus 12 bytes of ID and timestamp per image; the table rows are random 256-1024 byte writes.
#include "common.cuh"
#include "internal.h"

namespace gear {

template <typename TD> struct RefreshChunk;                 // one 16-byte chunk of a table row and its fp32 source
template <> struct RefreshChunk<float> {
    static constexpr int PER = 4;
    float4 a;
    __device__ __forceinline__ void load(const float* src) { a = ld_stream_f4(src); }
    __device__ __forceinline__ void store(float* dst) const { st_f4(dst, a); }
};
template <> struct RefreshChunk<__nv_bfloat16> {
    static constexpr int PER = 8;
    float4 a, b;
    __device__ __forceinline__ void load(const float* src) { a = ld_stream_f4(src); b = ld_stream_f4(src + 4); }
    __device__ __forceinline__ void store(__nv_bfloat16* dst) const {
        __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
        __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
        *reinterpret_cast<uint4*>(dst) = make_uint4(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1),
                                                    *reinterpret_cast<uint32_t*>(&h2), *reinterpret_cast<uint32_t*>(&h3));
    }
};

constexpr int RF_ROWS = 4;       // images a warp takes per pass: their loads are all in flight before the first store

// d_n (optional): a count on the device that bounds n, e.g. the one the expiry scan has just written.
template <typename TD>
__global__ void __launch_bounds__(256)
refresh_dfv_kernel(const int32_t* __restrict__ ids, const float* __restrict__ rows, int64_t ld, int64_t n,
                   const int64_t* __restrict__ d_n, int64_t now, TD* __restrict__ dfv, int64_t* __restrict__ ts,
                   int64_t vocab, int D, DevState* __restrict__ state) {
    wait_for_predecessor();
    constexpr int PER = RefreshChunk<TD>::PER;
    if (d_n) { const int64_t m = *d_n; if (m < n) n = m < 0 ? 0 : m; }
    const int lane = (int)lane_id();
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int n_chunks = D / PER;
    bool bad = false;
    for (int64_t k0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * RF_ROWS; k0 < n; k0 += warps * RF_ROWS) {
        int64_t id[RF_ROWS];
#pragma unroll
        for (int t = 0; t < RF_ROWS; ++t) {
            id[t] = k0 + t < n ? (int64_t)__ldg(ids + k0 + t) : -1;        // every lane reads the same word
            if (k0 + t < n && (id[t] < 0 || id[t] >= vocab)) { bad = true; id[t] = -1; }
        }
        for (int ch = lane; ch < n_chunks; ch += 32) {
            RefreshChunk<TD> c[RF_ROWS];
#pragma unroll
            for (int t = 0; t < RF_ROWS; ++t)
                if (id[t] >= 0) c[t].load(rows + (k0 + t) * ld + ch * PER);
#pragma unroll
            for (int t = 0; t < RF_ROWS; ++t)
                if (id[t] >= 0) c[t].store(dfv + id[t] * (int64_t)D + ch * PER);
        }
        if (lane < RF_ROWS) {
            int64_t mine = id[0];
#pragma unroll
            for (int t = 1; t < RF_ROWS; ++t) if (lane == t) mine = id[t];
            if (mine >= 0) ts[mine] = now;
        }
    }
    if (bad && lane == 0) atomicOr(&state->status, GEAR_DEV_BAD_ID);
}

cudaError_t launch_refresh_dfv(const gear_ctx_impl& c, const int32_t* ids, const float* rows, int64_t ld, int64_t n,
                               const int64_t* d_n, int64_t now, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const int64_t want = ceil_div(n, 8 * RF_ROWS);
    const int64_t cap = (int64_t)sm_count() * 8;                          // eight resident blocks per SM
    const int grid = (int)(want < cap ? want : cap);
    KernelScope k(&c.prof, "refresh_dfv", st);
    if (c.cfg.dfv_dtype == GEAR_BF16)
        return launch_dependent(refresh_dfv_kernel<__nv_bfloat16>, dim3(grid), dim3(256), 0, st, ids, rows, ld, n, d_n, now,
                                static_cast<__nv_bfloat16*>(c.buf.dfv), c.buf.dfv_ts, (int64_t)c.cfg.img_vocab, c.cfg.dfv_dim,
                                c.state());
    return launch_dependent(refresh_dfv_kernel<float>, dim3(grid), dim3(256), 0, st, ids, rows, ld, n, d_n, now,
                            static_cast<float*>(c.buf.dfv), c.buf.dfv_ts, (int64_t)c.cfg.img_vocab, c.cfg.dfv_dim, c.state());
}

}  // namespace gear
