// Event 4, "push the Sparse Part's gradients": table[id] += alpha * sum of the dX rows of the views
// that share id.
//
// The batch's IDs are key-sorted (stable radix sort, value = view index), so that views sharing an ID
// sit next to each other.  A group of lanes then walks a short run of sorted positions, sums the rows
// that share a key in registers and issues one 128-bit reduction per 16 bytes of table row at every key
// change.  Hot IDs (Zipf) therefore cost one reduction per run instead of one per view.  HBM/L2 bound:
// B rows of E floats read, about one table row read-modify-written per distinct ID.
#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int ES_SEG = 8;    // sorted positions walked by one lane group

// LPR lanes share a row: lane c of the group owns the float4 chunks c, c + LPR, ... (NQ of them)
template <int NQ>
__global__ void __launch_bounds__(256)
emb_reduce_kernel(const uint32_t* __restrict__ ks, const uint32_t* __restrict__ perm, int n, uint32_t vocab,
                  int E, int lpr, const float* __restrict__ dX, int64_t ldx, int col0,
                  float* __restrict__ table, float alpha) {
    wait_for_predecessor();
    const int64_t gthread = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t group = gthread / lpr;
    const int c = (int)(gthread % lpr);
    const int64_t p0 = group * ES_SEG;
    if (p0 >= n) return;
    const int n_chunks = E / 4;

    uint32_t key[ES_SEG], row[ES_SEG];
#pragma unroll
    for (int t = 0; t < ES_SEG; ++t) {
        const int64_t p = p0 + t;
        key[t] = p < n ? ks[p] : vocab;
        row[t] = p < n ? perm[p] : 0u;
    }
    float4 v[ES_SEG][NQ];
#pragma unroll
    for (int t = 0; t < ES_SEG; ++t)
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int ch = c + q * lpr;
            v[t][q] = (key[t] < vocab && ch < n_chunks) ? ld_f4(dX + (int64_t)row[t] * ldx + col0 + ch * 4)
                                                        : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    float4 acc[NQ];
#pragma unroll
    for (int q = 0; q < NQ; ++q) acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int t = 0; t < ES_SEG; ++t) {
        if (key[t] >= vocab) break;
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            acc[q].x += v[t][q].x; acc[q].y += v[t][q].y; acc[q].z += v[t][q].z; acc[q].w += v[t][q].w;
        }
        const bool last = (t == ES_SEG - 1) || key[t + 1] != key[t];
        if (last) {
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int ch = c + q * lpr;
                if (ch < n_chunks)
                    red_add_f4(table + (int64_t)key[t] * E + ch * 4,
                               make_float4(alpha * acc[q].x, alpha * acc[q].y, alpha * acc[q].z, alpha * acc[q].w));
                acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
    }
}

cudaError_t launch_emb_reduce(const gear_ctx_impl& c, int which, int cur, int32_t B, int64_t vocab, float* table,
                              const float* dX, int ldx, int col0, float alpha, cudaStream_t st) {
    if (B <= 0) return cudaSuccess;
    SortJob sb = c.sort_job(which);
    const int E = c.cfg.emb_dim, n_chunks = E / 4;
    int lpr = 1;
    while (lpr < n_chunks && lpr < 32) lpr <<= 1;
    const int nq = (int)ceil_div(n_chunks, lpr);
    const int64_t groups = ceil_div(B, ES_SEG);
    const unsigned grid = (unsigned)ceil_div(groups * lpr, 256);
#define GEAR_ES_LAUNCH(NQ) launch_dependent(emb_reduce_kernel<NQ>, dim3(grid), dim3(256), 0, st, sb.keys[cur], sb.vals[cur], B, (uint32_t)vocab, \
                                                                        E, lpr, dX, ldx, col0, table, alpha)
    KernelScope ks(&c.prof, "emb_reduce", st);
    if (nq <= 1) GEAR_ES_LAUNCH(1);
    else if (nq <= 2) GEAR_ES_LAUNCH(2);
    else if (nq <= 4) GEAR_ES_LAUNCH(4);
    else GEAR_ES_LAUNCH(8);
#undef GEAR_ES_LAUNCH
    return cudaGetLastError();
}

}  // namespace gear
