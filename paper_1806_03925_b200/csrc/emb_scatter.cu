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
// One of the two tables of a launch (blockIdx.y picks it).
struct EmbTable { const uint32_t* ks; const uint32_t* perm; uint32_t vocab; int col0; float* table; };

// COMPACT: the sums do not go to the table but to a buffer with one row per sorted position: an ID's sum lands in the
// row of the position at which its run starts (table then points to that buffer, alpha is 1).  The optimiser's row
// kernel (dense.cu) picks the sums up from there: a non-linear update needs an ID's whole sum before it can start.
template <int NQ, bool COMPACT>
__global__ void __launch_bounds__(256)
emb_reduce_kernel(const EmbTable t0, const EmbTable t1, int n, int E, int lpr, const float* __restrict__ dX, int64_t ldx,
                  float alpha) {
    wait_for_predecessor();
    const EmbTable& t = blockIdx.y == 0 ? t0 : t1;
    const uint32_t* __restrict__ ks = t.ks;
    const uint32_t* __restrict__ perm = t.perm;
    const uint32_t vocab = t.vocab;
    const int col0 = t.col0;
    float* __restrict__ table = t.table;
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
    // COMPACT: where the run that covers position p0 starts (it may start in an earlier segment: gallop back, then bisect)
    int64_t head = p0;
    if (COMPACT && p0 > 0 && key[0] < vocab && ks[p0 - 1] == key[0]) {
        int64_t hi = p0 - 1, step = 1, lo = hi - 1;            // ks[hi] == key[0]
        while (lo >= 0 && ks[lo] == key[0]) { hi = lo; step <<= 1; lo = max(hi - step, (int64_t)-1); }
        int64_t l = lo + 1, h = hi;                            // answer in [l, h]; ks[h] == key[0], ks[lo] != key[0]
        while (l < h) {
            const int64_t mid = (l + h) >> 1;
            if (ks[mid] == key[0]) h = mid; else l = mid + 1;
        }
        head = l;
    }
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
                    red_add_f4(table + (COMPACT ? head : (int64_t)key[t]) * E + ch * 4,
                               make_float4(alpha * acc[q].x, alpha * acc[q].y, alpha * acc[q].z, alpha * acc[q].w));
                acc[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            head = p0 + t + 1;                                 // the next position starts a run
        }
    }
}

// both tables of a step in one launch: user rows (columns 0 .. E) and URL-hash rows (columns E .. 2E) of dX
cudaError_t launch_emb_reduce(const gear_ctx_impl& c, int cur, int32_t B, float* user_table, float* url_table,
                              const float* dX, int ldx, float alpha, cudaStream_t st) {
    if (B <= 0) return cudaSuccess;
    SortJob su = c.sort_job(gear_ctx_impl::SORT_USER), sh = c.sort_job(gear_ctx_impl::SORT_URL);
    const int E = c.cfg.emb_dim, n_chunks = E / 4;
    int lpr = 1;
    while (lpr < n_chunks && lpr < 32) lpr <<= 1;
    const int nq = (int)ceil_div(n_chunks, lpr);
    const int64_t groups = ceil_div(B, ES_SEG);
    const dim3 grid((unsigned)ceil_div(groups * lpr, 256), 2);
    const EmbTable t0{su.keys[cur], su.vals[cur], (uint32_t)c.cfg.user_vocab, 0, user_table};
    const EmbTable t1{sh.keys[cur], sh.vals[cur], (uint32_t)c.cfg.url_vocab, E, url_table};
#define GEAR_ES_LAUNCH(NQ) launch_dependent(emb_reduce_kernel<NQ, false>, grid, dim3(256), 0, st, t0, t1, B, E, lpr, dX, (int64_t)ldx, alpha)
    KernelScope ks(&c.prof, "emb_reduce", st);
    if (nq <= 1) GEAR_ES_LAUNCH(1);
    else if (nq <= 2) GEAR_ES_LAUNCH(2);
    else if (nq <= 4) GEAR_ES_LAUNCH(4);
    else GEAR_ES_LAUNCH(8);
#undef GEAR_ES_LAUNCH
    return cudaGetLastError();
}

// Section 4's optimiser on the rows of both embedding tables that the batch touched: the per-ID sums go to the compact
// buffers (zeroed first), then every distinct ID's row takes one Adam step.
cudaError_t launch_emb_adam(const gear_ctx_impl& c, int cur, int32_t B, const float* dX, int ldx, const gear_adam& cfg,
                            int64_t t, float* user_m, float* user_v, float* url_m, float* url_v, cudaStream_t st) {
    if (B <= 0) return cudaSuccess;
    SortJob su = c.sort_job(gear_ctx_impl::SORT_USER), sh = c.sort_job(gear_ctx_impl::SORT_URL);
    const int E = c.cfg.emb_dim, n_chunks = E / 4;
    float* gu = c.at<float>(c.ws.emb_gsum[0]);
    float* gh = c.at<float>(c.ws.emb_gsum[1]);
    cudaError_t e = cudaMemsetAsync(gu, 0, sizeof(float) * (size_t)B * E, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(gh, 0, sizeof(float) * (size_t)B * E, st);
    if (e != cudaSuccess) return e;
    int lpr = 1;
    while (lpr < n_chunks && lpr < 32) lpr <<= 1;
    const int nq = (int)ceil_div(n_chunks, lpr);
    const int64_t groups = ceil_div(B, ES_SEG);
    const dim3 grid((unsigned)ceil_div(groups * lpr, 256), 2);
    const EmbTable t0{su.keys[cur], su.vals[cur], (uint32_t)c.cfg.user_vocab, 0, gu};
    const EmbTable t1{sh.keys[cur], sh.vals[cur], (uint32_t)c.cfg.url_vocab, E, gh};
    {
#define GEAR_ES_LAUNCH(NQ) launch_dependent(emb_reduce_kernel<NQ, true>, grid, dim3(256), 0, st, t0, t1, B, E, lpr, dX, (int64_t)ldx, 1.0f)
        KernelScope ks(&c.prof, "emb_reduce", st);
        if (nq <= 1) GEAR_ES_LAUNCH(1);
        else if (nq <= 2) GEAR_ES_LAUNCH(2);
        else if (nq <= 4) GEAR_ES_LAUNCH(4);
        else GEAR_ES_LAUNCH(8);
#undef GEAR_ES_LAUNCH
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const EmbAdamTable a0{su.keys[cur], (uint32_t)c.cfg.user_vocab, c.buf.user_emb, user_m, user_v, gu};
    const EmbAdamTable a1{sh.keys[cur], (uint32_t)c.cfg.url_vocab, c.buf.url_emb, url_m, url_v, gh};
    return launch_emb_adam_rows(c, a0, a1, B, t, cfg, st);
}

}  // namespace gear

namespace gear {

// The owner of a table shard applies gradient rows that arrive with their IDs (from its own step or from other devices):
// stable key sort of the IDs, then the segmented sum and scatter above on that one table.
cudaError_t launch_apply_emb_grad(const gear_ctx_impl& c, int which, const int32_t* ids, const float* rows, int64_t ld,
                                  int64_t n, float alpha, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const bool user = which == GEAR_TABLE_USER;
    const int64_t vocab = user ? c.cfg.user_vocab : c.cfg.url_vocab;
    SortBatch batch = c.sort_batch();
    batch.n_jobs = 1;
    batch.job[0] = c.sort_job(user ? gear_ctx_impl::SORT_USER : gear_ctx_impl::SORT_URL);
    batch.job[0].ids = ids; batch.job[0].sentinel = (uint32_t)vocab;
    batch.job[0].n_max = n; batch.job[0].bits = bits_for(vocab);
    batch.name = "sort_emb";
    cudaError_t se;
    const int cur = sort_jobs(batch, &c.gbs, st, &c.prof, &se);
    if (se != cudaSuccess) return se;
    const int E = c.cfg.emb_dim, n_chunks = E / 4;
    int lpr = 1;
    while (lpr < n_chunks && lpr < 32) lpr <<= 1;
    const int nq = (int)ceil_div(n_chunks, lpr);
    const int64_t groups = ceil_div(n, ES_SEG);
    const dim3 grid((unsigned)ceil_div(groups * lpr, 256), 1);
    const EmbTable t0{batch.job[0].keys[cur], batch.job[0].vals[cur], (uint32_t)vocab, 0, user ? c.buf.user_emb : c.buf.url_emb};
#define GEAR_ES_LAUNCH(NQ) launch_dependent(emb_reduce_kernel<NQ, false>, grid, dim3(256), 0, st, t0, t0, (int)n, E, lpr, rows, ld, alpha)
    KernelScope ks(&c.prof, "emb_reduce", st);
    if (nq <= 1) GEAR_ES_LAUNCH(1);
    else if (nq <= 2) GEAR_ES_LAUNCH(2);
    else if (nq <= 4) GEAR_ES_LAUNCH(4);
    else GEAR_ES_LAUNCH(8);
#undef GEAR_ES_LAUNCH
    return cudaGetLastError();
}

}  // namespace gear
