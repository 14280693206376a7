// The Slowgear side beyond the gradient store: a linear Dense Part and the optimiser of the paper's experiments.
//
//   dense forward   Section 3, events 2 and 3: the Dense Part turns an image's raw data into its Dense Feature Vector.
//                   Here the smallest Dense Part there is: DFV[id] = raw[id] . Wd  (raw [img_vocab][R], Wd [R][D]).
//   dense backward  Section 3, event 6, second half; Eq. 1, right factor: the averaged gradient of every completed
//                   group goes back through the Dense Part.  For the linear map dDFV[id][c] / dWd[r][c] = raw[id][r]:
//                   G[r][c] += sum over emissions e of raw[id_e][r] * avg_e[c].
//   Adam            Section 4: the optimiser of the paper's experiments, for dense parameter vectors (head, Wd) and for
//                   the rows of an embedding table that received a gradient in this step.
//
// The two products are fp32 FMA products with one operand gathered by Image ID (the tolerance is 1e-5; reductions of
// a few dozen to a few hundred terms).  64 x 64 x 16 tiles through shared memory, 4 x 4 outputs per thread.
#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int DT = 64;     // tile edge
constexpr int DK = 16;     // tile depth

// rows[k][c] = sum_r raw[ids[k]][r] * Wd[r][c],  k < min(n, *d_n),  c < D.  An ID outside [0, vocab) gives a zero row.
__global__ void __launch_bounds__(256)
dense_forward_kernel(const float* __restrict__ raw, int64_t vocab, int R, const float* __restrict__ Wd, int D,
                     const int32_t* __restrict__ ids, int64_t n, const int64_t* __restrict__ d_n,
                     float* __restrict__ rows, int64_t ld, DevState* __restrict__ state) {
    wait_for_predecessor();
    if (d_n) { const int64_t live = *d_n; n = live < n ? (live < 0 ? 0 : live) : n; }
    const int64_t m0 = (int64_t)blockIdx.x * DT;           // row tiles along x: an expiry list can hold millions of IDs
    if (m0 >= n) return;
    __shared__ float As[DK][DT + 4];
    __shared__ float Bs[DK][DT + 4];
    __shared__ int64_t row_of[DT];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int n0 = blockIdx.y * DT;
    if (tid < DT) {
        int64_t id = -1;
        if (m0 + tid < n) {
            id = ids[m0 + tid];
            if (id < 0 || id >= vocab) { id = -1; atomicOr(&state->status, GEAR_DEV_BAD_ID); }
        }
        row_of[tid] = id;
    }
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int k0 = 0; k0 < R; k0 += DK) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int idx = tid + r * 256;
            const int m = idx >> 4, k = idx & 15;                  // A: the reduction index is the fast one
            const int64_t id = row_of[m];
            As[k][m] = (id >= 0 && k0 + k < R) ? __ldg(raw + id * R + k0 + k) : 0.f;
            const int kb = idx >> 6, c = idx & 63;                 // B: the column is the fast one
            Bs[kb][c] = (k0 + kb < R && n0 + c < D) ? __ldg(Wd + (int64_t)(k0 + kb) * D + n0 + c) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < DK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int64_t m = m0 + ty * 4 + i;
        if (m >= n) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = n0 + tx * 4 + j;
            if (c < D) rows[m * ld + c] = acc[i][j];
        }
    }
}

// G[r][c] += sum over e in this block's slice of raw[ids[e]][r] * avg[e][c].  blockIdx.z walks slices of e_chunk emissions.
__global__ void __launch_bounds__(256)
dense_backward_kernel(const float* __restrict__ raw, int64_t vocab, int R, int D, const int32_t* __restrict__ ids,
                      const float* __restrict__ avg, int64_t ld_avg, int64_t n, const int64_t* __restrict__ d_n,
                      int e_chunk, float* __restrict__ G, DevState* __restrict__ state) {
    wait_for_predecessor();
    if (d_n) { const int64_t live = *d_n; n = live < n ? (live < 0 ? 0 : live) : n; }
    const int64_t e_begin = (int64_t)blockIdx.z * e_chunk;
    if (e_begin >= n) return;
    const int64_t e_end = min(n, e_begin + (int64_t)e_chunk);
    __shared__ float As[DK][DT + 4];       // [emission][r]
    __shared__ float Bs[DK][DT + 4];       // [emission][c]
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int r0 = blockIdx.y * DT, c0 = blockIdx.x * DT;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    int flags = 0;
    for (int64_t e0 = e_begin; e0 < e_end; e0 += DK) {
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int idx = tid + q * 256;
            const int k = idx >> 6, x = idx & 63;                  // both operands: emission slow, row / column fast
            const int64_t e = e0 + k;
            int64_t id = -1;
            if (e < e_end) {
                id = ids[e];
                if (id < 0 || id >= vocab) { id = -1; flags |= GEAR_DEV_BAD_ID; }
            }
            As[k][x] = (id >= 0 && r0 + x < R) ? __ldg(raw + id * R + r0 + x) : 0.f;
            Bs[k][x] = (id >= 0 && c0 + x < D) ? __ldg(avg + e * ld_avg + c0 + x) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < DK; ++k) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[k][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
    if (flags) atomicOr(&state->status, flags);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = r0 + ty * 4 + i;
        if (r >= R) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int c = c0 + tx * 4 + j;
            if (c < D) atomicAdd(G + (int64_t)r * D + c, acc[i][j]);
        }
    }
}

cudaError_t launch_dense_forward(const gear_ctx_impl& c, const float* raw, int R, const float* Wd, const int32_t* ids,
                                 int64_t n, const int64_t* d_n, float* rows, int64_t ld, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    KernelScope k(&c.prof, "dense_forward", st);
    const dim3 grid((unsigned)ceil_div(n, DT), (unsigned)ceil_div(c.cfg.dfv_dim, DT));
    return launch_dependent(dense_forward_kernel, grid, dim3(256), 0, st, raw, c.cfg.img_vocab, R, Wd, c.cfg.dfv_dim, ids, n, d_n,
                            rows, ld, c.state());
}

cudaError_t launch_dense_backward(const gear_ctx_impl& c, const float* raw, int R, const int32_t* ids, const float* avg,
                                  int64_t ld_avg, int64_t n, const int64_t* d_n, float* G, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    KernelScope k(&c.prof, "dense_backward", st);
    // slices of the emission list: enough of them to fill the GPU a few times over, each at least 256 emissions long
    const int64_t tiles = ceil_div(c.cfg.dfv_dim, DT) * ceil_div(R, DT);
    int64_t slices = ceil_div((int64_t)sm_count() * 8, tiles);
    const int64_t max_slices = ceil_div(n, 256);
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    if (slices > 65535) slices = 65535;
    const int e_chunk = (int)(ceil_div(ceil_div(n, slices), DK) * DK);
    const dim3 grid((unsigned)ceil_div(c.cfg.dfv_dim, DT), (unsigned)ceil_div(R, DT), (unsigned)ceil_div(n, e_chunk));
    return launch_dependent(dense_backward_kernel, grid, dim3(256), 0, st, raw, c.cfg.img_vocab, R, c.cfg.dfv_dim, ids, avg, ld_avg,
                            n, d_n, e_chunk, G, c.state());
}

// ---------------------------------------------------------------- Adam (Kingma and Ba 2015, Algorithm 1)
struct AdamCoef { float lr, b1, b2, eps, inv_c1, inv_c2; };      // inv_c1 = 1 / (1 - b1^t), inv_c2 = 1 / (1 - b2^t)

__device__ __forceinline__ void adam_update(float& p, float g, float& m, float& v, const AdamCoef& a) {
    m = a.b1 * m + (1.f - a.b1) * g;
    v = a.b2 * v + (1.f - a.b2) * g * g;
    p -= a.lr * (m * a.inv_c1) / (sqrtf(v * a.inv_c2) + a.eps);
}

__global__ void __launch_bounds__(256)
adam_dense_kernel(float* __restrict__ p, const float* __restrict__ g, float* __restrict__ m, float* __restrict__ v,
                  int64_t n, const AdamCoef a) {
    wait_for_predecessor();
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        float pi = p[i], mi = m[i], vi = v[i];
        adam_update(pi, g[i], mi, vi, a);
        p[i] = pi; m[i] = mi; v[i] = vi;
    }
}

static AdamCoef adam_coef(const gear_adam& cfg, int64_t t) {
    const double c1 = 1.0 - pow((double)cfg.beta1, (double)t), c2 = 1.0 - pow((double)cfg.beta2, (double)t);
    return AdamCoef{cfg.lr, cfg.beta1, cfg.beta2, cfg.eps, (float)(1.0 / c1), (float)(1.0 / c2)};
}

cudaError_t launch_adam_dense(Profiler* prof, float* p, const float* g, float* m, float* v, int64_t n, int64_t t,
                              const gear_adam& cfg, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    KernelScope k(prof, "adam_dense", st);
    const int64_t want = ceil_div(n, 256), cap = (int64_t)sm_count() * 8;
    return launch_dependent(adam_dense_kernel, dim3((unsigned)(want < cap ? want : cap)), dim3(256), 0, st, p, g, m, v, n,
                            adam_coef(cfg, t));
}

// ---------------------------------------------------------------- Adam on the embedding rows a step touched
// The summed gradient of every distinct ID of the batch sits in a compact buffer, in the row of the sorted position
// at which the ID's run starts (emb_scatter.cu).  One lane group per sorted position: a position that starts a run
// takes the Adam step of its ID's table row and moment rows; the others have nothing to do.
template <int NQ>
__global__ void __launch_bounds__(256)
emb_adam_rows_kernel(const EmbAdamTable t0, const EmbAdamTable t1, int n, int E, int lpr, const AdamCoef a) {
    wait_for_predecessor();
    const EmbAdamTable& t = blockIdx.y == 0 ? t0 : t1;
    const int64_t gthread = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t p = gthread / lpr;
    const int c = (int)(gthread % lpr);
    if (p >= n) return;
    const uint32_t key = t.ks[p];
    if (key >= t.vocab || (p > 0 && t.ks[p - 1] == key)) return;
    const int n_chunks = E / 4;
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const int ch = c + q * lpr;
        if (ch >= n_chunks) continue;
        const float4 g = ld_f4(t.gsum + p * (int64_t)E + ch * 4);
        float* prow = t.table + (int64_t)key * E + ch * 4;
        float* mrow = t.m + (int64_t)key * E + ch * 4;
        float* vrow = t.v + (int64_t)key * E + ch * 4;
        float4 pv = ld_f4(prow), mv = ld_f4(mrow), vv = ld_f4(vrow);
        adam_update(pv.x, g.x, mv.x, vv.x, a); adam_update(pv.y, g.y, mv.y, vv.y, a);
        adam_update(pv.z, g.z, mv.z, vv.z, a); adam_update(pv.w, g.w, mv.w, vv.w, a);
        st_f4(prow, pv); st_f4(mrow, mv); st_f4(vrow, vv);
    }
}

cudaError_t launch_emb_adam_rows(const gear_ctx_impl& c, const EmbAdamTable& t0, const EmbAdamTable& t1, int32_t B,
                                 int64_t t, const gear_adam& cfg, cudaStream_t st) {
    if (B <= 0) return cudaSuccess;
    const int E = c.cfg.emb_dim, n_chunks = E / 4;
    int lpr = 1;
    while (lpr < n_chunks && lpr < 32) lpr <<= 1;
    const int nq = (int)ceil_div(n_chunks, lpr);
    const dim3 grid((unsigned)ceil_div((int64_t)B * lpr, 256), 2);
    const AdamCoef a = adam_coef(cfg, t);
    KernelScope ks(&c.prof, "emb_adam_rows", st);
#define GEAR_EA_LAUNCH(NQ) launch_dependent(emb_adam_rows_kernel<NQ>, grid, dim3(256), 0, st, t0, t1, (int)B, E, lpr, a)
    if (nq <= 1) return GEAR_EA_LAUNCH(1);
    if (nq <= 2) return GEAR_EA_LAUNCH(2);
    if (nq <= 4) return GEAR_EA_LAUNCH(4);
    return GEAR_EA_LAUNCH(8);
#undef GEAR_EA_LAUNCH
}

}  // namespace gear
