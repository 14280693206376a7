// What a table shard's owner and a worker need when the tables are partitioned by ID across devices (Section 3: the
// Slowgear Workers serve requests "by partition of Image ID"; Section 4: N Fastgear and N Slowgear workers):
//   fetch rows     the owner's answer to a request for rows by ID (event 3: "sends inference result back"): plain
//                  copies of table rows, in the table's storage type, into a dense buffer that is then sent;
//   gradient rows  event 5 in its materialised form: one (Image ID, gradient) pair per image occurrence,
//                  g_r = dLoss/d(pooled DFV)[view of r] * 1/n_view, as a dense [nnz][D] array that can be sent.
// Both are HBM-bound row copies: a warp takes eight rows per pass, a lane owns 16-byte chunks, all loads of a pass
// are issued before the first store.
#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int SH_ROWS = 8;

__global__ void __launch_bounds__(256)
fetch_rows_kernel(const uint4* __restrict__ table, int64_t vocab, int chunks, const int32_t* __restrict__ ids, int64_t n,
                  uint4* __restrict__ out, DevState* __restrict__ state) {
    wait_for_predecessor();
    const int lane = (int)lane_id();
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    bool bad = false;
    for (int64_t k0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * SH_ROWS; k0 < n; k0 += warps * SH_ROWS) {
        int64_t id[SH_ROWS];
#pragma unroll
        for (int t = 0; t < SH_ROWS; ++t) {
            id[t] = k0 + t < n ? (int64_t)__ldg(ids + k0 + t) : -1;
            if (k0 + t < n && (id[t] < 0 || id[t] >= vocab)) { bad = true; id[t] = -2; }     // -2: a zero row is written
        }
        for (int ch = lane; ch < chunks; ch += 32) {
            uint4 v[SH_ROWS];
#pragma unroll
            for (int t = 0; t < SH_ROWS; ++t)
                v[t] = id[t] >= 0 ? __ldg(table + id[t] * chunks + ch) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
            for (int t = 0; t < SH_ROWS; ++t)
                if (id[t] != -1) out[(k0 + t) * chunks + ch] = v[t];
        }
    }
    if (bad && lane == 0) atomicOr(&state->status, GEAR_DEV_BAD_ID);
}

cudaError_t launch_fetch_rows(const gear_ctx_impl& c, int which, const int32_t* ids, int64_t n, void* out, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const void* table; int64_t vocab; int row_bytes;
    if (which == GEAR_TABLE_USER) { table = c.buf.user_emb; vocab = c.cfg.user_vocab; row_bytes = c.cfg.emb_dim * 4; }
    else if (which == GEAR_TABLE_URL) { table = c.buf.url_emb; vocab = c.cfg.url_vocab; row_bytes = c.cfg.emb_dim * 4; }
    else { table = c.buf.dfv; vocab = c.cfg.img_vocab; row_bytes = c.cfg.dfv_dim * (c.cfg.dfv_dtype == GEAR_BF16 ? 2 : 4); }
    const int64_t want = ceil_div(n, 8 * SH_ROWS), cap = (int64_t)sm_count() * 8;
    KernelScope k(&c.prof, "fetch_rows", st);
    return launch_dependent(fetch_rows_kernel, dim3((unsigned)(want < cap ? want : cap)), dim3(256), 0, st,
                            static_cast<const uint4*>(table), vocab, row_bytes / 16, ids, n, static_cast<uint4*>(out), c.state());
}

// out[r][c] = dX[row_view[r]][col0 + c] * inv_n[row_view[r]],  r < nnz,  c < D
__global__ void __launch_bounds__(256)
dfv_grad_rows_kernel(const float* __restrict__ dX, int64_t ldx, int col0, int D, const int32_t* __restrict__ row_view,
                     const float* __restrict__ inv_n, int64_t nnz, float* __restrict__ out) {
    wait_for_predecessor();
    const int lane = (int)lane_id();
    const int chunks = D / 4;
    const int64_t warps = (int64_t)gridDim.x * (blockDim.x >> 5);
    for (int64_t k0 = ((int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5)) * SH_ROWS; k0 < nnz; k0 += warps * SH_ROWS) {
        int view[SH_ROWS];
        float s[SH_ROWS];
#pragma unroll
        for (int t = 0; t < SH_ROWS; ++t) {
            view[t] = k0 + t < nnz ? __ldg(row_view + k0 + t) : -1;
            s[t] = view[t] >= 0 ? __ldg(inv_n + view[t]) : 0.f;
        }
        for (int ch = lane; ch < chunks; ch += 32) {
            float4 v[SH_ROWS];
#pragma unroll
            for (int t = 0; t < SH_ROWS; ++t)
                v[t] = view[t] >= 0 ? ld_f4(dX + (int64_t)view[t] * ldx + col0 + ch * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int t = 0; t < SH_ROWS; ++t)
                if (view[t] >= 0)
                    st_f4(out + (k0 + t) * (int64_t)D + ch * 4, make_float4(v[t].x * s[t], v[t].y * s[t], v[t].z * s[t], v[t].w * s[t]));
        }
    }
}

cudaError_t launch_dfv_grad_rows(const gear_ctx_impl& c, const float* dX, const int32_t* row_view, const float* inv_n,
                                 int64_t nnz, float* out, cudaStream_t st) {
    if (nnz <= 0) return cudaSuccess;
    const int64_t want = ceil_div(nnz, 8 * SH_ROWS), cap = (int64_t)sm_count() * 8;
    KernelScope k(&c.prof, "dfv_grad_rows", st);
    return launch_dependent(dfv_grad_rows_kernel, dim3((unsigned)(want < cap ? want : cap)), dim3(256), 0, st, dX, (int64_t)c.d_in,
                            2 * c.cfg.emb_dim, c.cfg.dfv_dim, row_view, inv_n, nnz, out);
}

}  // namespace gear
