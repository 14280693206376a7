// Events 1-3 of the step: build the head input X[b] = [user row | url row | mean of the view's DFVs].
//
// One warp per page view.  Every lane owns 16-byte chunks of the rows (128-bit loads, a full row is read
// by consecutive lanes), so each table row is fetched with fully used 32-byte sectors.  The pooled sum is
// fp32, taken in slot order, divided once by n_b.  HBM bound: the kernel moves
// B*(2E*4) + nnz*D*sizeof(dfv) bytes of table rows and writes B*Din*sizeof(x).
#include "common.cuh"
#include "internal.h"

namespace gear {

template <typename T> struct Chunk;                         // 16 bytes of a table row as floats
template <> struct Chunk<float> {
    static constexpr int PER = 4;
    __device__ static void load(const float* row, int ch, float* v) {
        float4 t = ld_f4(row + ch * 4);
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
};
template <> struct Chunk<__nv_bfloat16> {
    static constexpr int PER = 8;
    __device__ static void load(const __nv_bfloat16* row, int ch, float* v) {
        uint4 t = *reinterpret_cast<const uint4*>(row + ch * 8);
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            v[2 * k] = __uint_as_float(w[k] << 16);
            v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
        }
    }
};

template <int N> __device__ __forceinline__ void store_x(float* dst, const float* v) {
#pragma unroll
    for (int k = 0; k < N; k += 4) st_f4(dst + k, make_float4(v[k], v[k + 1], v[k + 2], v[k + 3]));
}
template <int N> __device__ __forceinline__ void store_x(__nv_bfloat16* dst, const float* v) {
    uint32_t w[N / 2];
#pragma unroll
    for (int k = 0; k < N / 2; ++k) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
        w[k] = *reinterpret_cast<uint32_t*>(&h);
    }
    if constexpr (N == 8) *reinterpret_cast<uint4*>(dst) = make_uint4(w[0], w[1], w[2], w[3]);
    else *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);
}

struct GatherArgs {
    const float* user_emb; const float* url_emb; const void* dfv;
    int64_t user_vocab, url_vocab, img_vocab;
    int E, D, B;
    int64_t nnz;
    const int32_t* user_id; const int32_t* url_id; const int32_t* img_off; const int32_t* img_id;
    void* X; void* x_debug;
    int32_t* row_view; float* inv_n;
    DevState* state;
};

// NQ = 16-byte chunks of a DFV row per lane
template <typename TD, typename TX, int NQ>
__global__ void __launch_bounds__(256)
gather_pool_kernel(const GatherArgs a) {
    constexpr int PER = Chunk<TD>::PER;
    const unsigned lane = lane_id();
    const int warps_per_block = blockDim.x >> 5;
    const int Din = 2 * a.E + a.D;
    const int n_chunks = a.D / PER;
    const TD* dfv = static_cast<const TD*>(a.dfv);
    int flags = 0;

    for (int b = blockIdx.x * warps_per_block + (threadIdx.x >> 5); b < a.B; b += gridDim.x * warps_per_block) {
        TX* x = static_cast<TX*>(a.X) + (int64_t)b * Din;
        TX* xd = a.x_debug ? static_cast<TX*>(a.x_debug) + (int64_t)b * Din : nullptr;

        // user and URL-hash embedding rows: plain copies
        const int u = a.user_id[b], h = a.url_id[b];
        const bool u_ok = u >= 0 && u < a.user_vocab, h_ok = h >= 0 && h < a.url_vocab;
        if (!u_ok || !h_ok) flags |= GEAR_DEV_BAD_ID;
        for (int ch = lane; ch < a.E / 4; ch += 32) {
            float v[4] = {0.f, 0.f, 0.f, 0.f}, w[4] = {0.f, 0.f, 0.f, 0.f};
            if (u_ok) Chunk<float>::load(a.user_emb + (int64_t)u * a.E, ch, v);
            if (h_ok) Chunk<float>::load(a.url_emb + (int64_t)h * a.E, ch, w);
            store_x<4>(x + ch * 4, v);
            store_x<4>(x + a.E + ch * 4, w);
            if (xd) { store_x<4>(xd + ch * 4, v); store_x<4>(xd + a.E + ch * 4, w); }
        }

        // DFV rows of the view, summed in slot order
        int s = a.img_off[b], e = a.img_off[b + 1];
        if (s < 0 || e < s || e > a.nnz) { flags |= GEAR_DEV_BAD_CSR; e = s = 0; }
        const int n = e - s;
        float acc[NQ][PER];
#pragma unroll
        for (int q = 0; q < NQ; ++q)
#pragma unroll
            for (int k = 0; k < PER; ++k) acc[q][k] = 0.f;

        for (int j0 = 0; j0 < n; j0 += 32) {
            const int m = min(32, n - j0);
            int my_id = -1;
            if ((int)lane < m) {
                my_id = a.img_id[s + j0 + lane];
                if (a.row_view) a.row_view[s + j0 + lane] = b;
                if (my_id < 0 || my_id >= a.img_vocab) { flags |= GEAR_DEV_BAD_ID; my_id = -1; }
            }
            for (int j = 0; j < m; j += 4) {
                float v[4][NQ][PER];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int id = __shfl_sync(0xffffffffu, my_id, (j + t) & 31);
                    const bool on = (j + t) < m && id >= 0;
#pragma unroll
                    for (int q = 0; q < NQ; ++q) {
                        const int ch = lane + 32 * q;
                        if (on && ch < n_chunks) Chunk<TD>::load(dfv + (int64_t)id * a.D, ch, v[t][q]);
                        else {
#pragma unroll
                            for (int k = 0; k < PER; ++k) v[t][q][k] = 0.f;
                        }
                    }
                }
#pragma unroll
                for (int t = 0; t < 4; ++t)
#pragma unroll
                    for (int q = 0; q < NQ; ++q)
#pragma unroll
                        for (int k = 0; k < PER; ++k) acc[q][k] += v[t][q][k];
            }
        }
        const float nf = (float)n;
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int ch = lane + 32 * q;
            if (ch < n_chunks) {
                float o[PER];
#pragma unroll
                for (int k = 0; k < PER; ++k) o[k] = n > 0 ? acc[q][k] / nf : 0.f;
                store_x<PER>(x + 2 * a.E + ch * PER, o);
                if (xd) store_x<PER>(xd + 2 * a.E + ch * PER, o);
            }
        }
        if (a.inv_n && lane == 0) a.inv_n[b] = n > 0 ? 1.0f / nf : 0.f;
    }
    if (flags) atomicOr(&a.state->status, flags);
}

template <typename TD, typename TX>
static cudaError_t dispatch_nq(const GatherArgs& a, cudaStream_t st, Profiler* prof) {
    constexpr int PER = Chunk<TD>::PER;
    const int n_chunks = a.D / PER;
    const int nq = (n_chunks + 31) / 32;
    const int warps = 8;
    int grid = (int)ceil_div(a.B, warps);
    if (grid < 1) grid = 1;
    KernelScope ks(prof, "gather_pool", st);
    if (nq <= 1) gather_pool_kernel<TD, TX, 1><<<grid, warps * 32, 0, st>>>(a);
    else if (nq <= 2) gather_pool_kernel<TD, TX, 2><<<grid, warps * 32, 0, st>>>(a);
    else if (nq <= 4) gather_pool_kernel<TD, TX, 4><<<grid, warps * 32, 0, st>>>(a);
    else gather_pool_kernel<TD, TX, 8><<<grid, warps * 32, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_gather(const gear_ctx_impl& c, const gear_batch& b, int32_t* row_view, float* inv_n,
                          void* x_debug, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    GatherArgs a;
    a.user_emb = c.buf.user_emb; a.url_emb = c.buf.url_emb; a.dfv = c.buf.dfv;
    a.user_vocab = c.cfg.user_vocab; a.url_vocab = c.cfg.url_vocab; a.img_vocab = c.cfg.img_vocab;
    a.E = c.cfg.emb_dim; a.D = c.cfg.dfv_dim; a.B = b.B; a.nnz = b.nnz;
    a.user_id = b.user_id; a.url_id = b.url_id; a.img_off = b.img_off; a.img_id = b.img_id;
    a.X = c.at<void>(c.ws.x); a.x_debug = x_debug; a.row_view = row_view; a.inv_n = inv_n;
    a.state = c.state();
    const bool dbf = c.cfg.dfv_dtype == GEAR_BF16, xbf = c.cfg.head_dtype == GEAR_BF16;
    if (dbf && xbf) return dispatch_nq<__nv_bfloat16, __nv_bfloat16>(a, st, &c.prof);
    if (dbf && !xbf) return dispatch_nq<__nv_bfloat16, float>(a, st, &c.prof);
    if (!dbf && xbf) return dispatch_nq<float, __nv_bfloat16>(a, st, &c.prof);
    return dispatch_nq<float, float>(a, st, &c.prof);
}

}  // namespace gear
