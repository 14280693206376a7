// Events 1-3 of the step: build the head input X[b] = [user row | url row | mean of the view's DFVs].
//
// One warp per page view at a time.  Every lane owns 16-byte chunks of a row (128-bit loads; consecutive lanes read
// a row end to end, so each fetch uses full 32-byte sectors).  The loads of up to eight DFV rows of the
// view, and of its two embedding rows, are issued back to back before the first one is used; the code for
// each row count is straight-line (one dispatch per view on the number of rows), which keeps the
// instruction count per byte low enough for the memory system to be the limit.  The pooled sum is fp32,
// taken in slot order, divided once by n_b.  HBM bound: the kernel moves B*(2E*4) + nnz*D*sizeof(dfv)
// bytes of table rows and writes B*Din*sizeof(x).
#include <algorithm>
#include <cfloat>

#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int GP_WARPS = 8;      // warps (views) per block

template <typename T> struct Chunk;                         // 16 bytes of a table row
template <> struct Chunk<float> {
    static constexpr int PER = 4;
    __device__ static __forceinline__ void add(float* acc, const uint4& t) {
        acc[0] += __uint_as_float(t.x); acc[1] += __uint_as_float(t.y);
        acc[2] += __uint_as_float(t.z); acc[3] += __uint_as_float(t.w);
    }
};
template <> struct Chunk<__nv_bfloat16> {
    static constexpr int PER = 8;
    __device__ static __forceinline__ void add(float* acc, const uint4& t) {
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            acc[2 * k] += __uint_as_float(w[k] << 16);
            acc[2 * k + 1] += __uint_as_float(w[k] & 0xffff0000u);
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

// x / n for a small positive integer n held as nf, with rinv = 1 / nf: the product x * rinv corrected by one
// exact residual step, which yields the correctly rounded quotient (infinities and NaNs pass through).
__device__ __forceinline__ float div_by_count(float x, float nf, float rinv) {
    const float q = x * rinv;
    const float q2 = fmaf(fmaf(-q, nf, x), rinv, q);
    return fabsf(q) <= FLT_MAX ? q2 : q;
}

struct GatherArgs {
    const float* user_emb; const float* url_emb; const void* dfv;
    int64_t user_vocab, url_vocab, img_vocab;
    int E, D, B, F;
    const float* fast;          // [B][F] the views' own dense input (F > 0)
    int64_t nnz;
    const int32_t* user_id; const int32_t* url_id; const int32_t* img_off; const int32_t* img_id;
    void* X; void* x_debug;
    int32_t* row_view; float* inv_n;
    DevState* state;
};

// Adds rows j .. j + K - 1 of the view to acc, in order; their IDs, all valid, sit in lanes (j + t) % 32 of my_id.
// All K loads are issued before the first addition.  FULL: every lane owns a chunk of every row (the row is NQ * 512
// bytes), so the loads carry no predicate at all -- the kernel is bound by its integer instructions, and the
// compare-and-clear around a guarded 128-bit load costs as much as the row's additions.
template <typename TD, int NQ, int K, bool FULL>
__device__ __forceinline__ void add_rows(float (&acc)[NQ][Chunk<TD>::PER], const TD* __restrict__ dfv, int D,
                                         int n_chunks, int my_id, int j, int lane) {
    uint4 v[K][NQ];
#pragma unroll
    for (int t = 0; t < K; ++t) {
        const int id = __shfl_sync(0xffffffffu, my_id, (j + t) & 31);
        const uint4* __restrict__ row = reinterpret_cast<const uint4*>(dfv + (int64_t)id * D);
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int ch = lane + 32 * q;
            v[t][q] = (FULL || ch < n_chunks) ? __ldg(row + ch) : make_uint4(0u, 0u, 0u, 0u);
        }
    }
#pragma unroll
    for (int t = 0; t < K; ++t)
#pragma unroll
        for (int q = 0; q < NQ; ++q) Chunk<TD>::add(acc[q], v[t][q]);
}

// The same for a stretch of the view that holds an invalid ID (-1: the row counts as zeros): one row at a time.
template <typename TD, int NQ>
__device__ __forceinline__ void add_rows_checked(float (&acc)[NQ][Chunk<TD>::PER], const TD* __restrict__ dfv, int D,
                                              int n_chunks, int my_id, int j, int count, int lane) {
#pragma unroll 1
    for (int t = 0; t < count; ++t) {
        const int id = __shfl_sync(0xffffffffu, my_id, (j + t) & 31);
        const uint4* __restrict__ row = reinterpret_cast<const uint4*>(dfv + (int64_t)(id < 0 ? 0 : id) * D);
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int ch = lane + 32 * q;
            const uint4 v = (id >= 0 && ch < n_chunks) ? __ldg(row + ch) : make_uint4(0u, 0u, 0u, 0u);
            Chunk<TD>::add(acc[q], v);
        }
    }
}

struct ViewRec { int uid, hid, s, n; };

// The record of view b as every lane of the warp reads it (same words: one transaction each).
// Out-of-range views read as empty.
__device__ __forceinline__ ViewRec load_view(const GatherArgs& a, int b) {
    ViewRec r{-1, -1, 0, 0};
    if (b < a.B) {
        r.uid = __ldg(a.user_id + b); r.hid = __ldg(a.url_id + b);
        r.s = __ldg(a.img_off + b);
        r.n = __ldg(a.img_off + b + 1) - r.s;                 // validated when the view is processed
    }
    return r;
}

// NQ = 16-byte chunks of a DFV row per lane.  A warp walks views b, b + W, b + 2W, ... (W = warps of the grid)
// and keeps two stages of look-ahead in registers: the record of the view after next and the image IDs of
// the next view are requested before the current view's rows are summed, so that per view only one memory
// round trip (the rows themselves) is exposed.
template <typename TD, typename TX, int NQ, bool FULL>
__global__ void __launch_bounds__(GP_WARPS * 32, NQ <= 2 ? 3 : 2)
gather_pool_kernel(const GatherArgs a) {
    wait_for_predecessor();
    constexpr int PER = Chunk<TD>::PER;
    constexpr int KMAX = NQ >= 8 ? 1 : 8 / NQ;               // rows in flight per warp
    const int lane = (int)lane_id();
    const int W = gridDim.x * GP_WARPS;
    const int Din = 2 * a.E + a.D + a.F;
    const int n_chunks = a.D / PER;
    const int ce = a.E / 4;                                    // 16-byte chunks per embedding row
    const TD* __restrict__ dfv = static_cast<const TD*>(a.dfv);
    int flags = 0;

    auto load_ids = [&](const ViewRec& r, int j0) -> int {     // IDs j0 + lane of the view (unchecked), -1 past its end
        const bool ok = r.s >= 0 && r.n >= 0 && (int64_t)r.s + r.n <= a.nnz;
        return (ok && j0 + lane < r.n) ? __ldg(a.img_id + r.s + j0 + lane) : -1;
    };

    int b = blockIdx.x * GP_WARPS + (int)(threadIdx.x >> 5);
    ViewRec cur = load_view(a, b), nxt = load_view(a, b + W);
    int ids_cur = load_ids(cur, 0);

    for (; b < a.B; b += W) {
        // ---- look-ahead: IDs of the next view, record of the one after it
        const int ids_nxt = load_ids(nxt, 0);
        const ViewRec nxt2 = load_view(a, b + 2 * W);

        TX* __restrict__ x = static_cast<TX*>(a.X) + (int64_t)b * Din;
        TX* __restrict__ xd = a.x_debug ? static_cast<TX*>(a.x_debug) + (int64_t)b * Din : nullptr;
        int uid = cur.uid, hid = cur.hid, s = cur.s, n = cur.n;
        if (uid < 0 || uid >= a.user_vocab) { uid = -1; flags |= GEAR_DEV_BAD_ID; }
        if (hid < 0 || hid >= a.url_vocab) { hid = -1; flags |= GEAR_DEV_BAD_ID; }
        if (s < 0 || n < 0 || (int64_t)s + n > a.nnz) { flags |= GEAR_DEV_BAD_CSR; s = 0; n = 0; }
        int my_id = ids_cur;
        if (lane < n) {
            if (my_id < 0 || my_id >= a.img_vocab) { my_id = -1; flags |= GEAR_DEV_BAD_ID; }
            if (a.row_view) a.row_view[s + lane] = b;
        } else my_id = -1;
        // every ID among the (up to 32) held now is valid: the straight-line code may load without looking
        bool clean = !__any_sync(0xffffffffu, lane < n && my_id < 0);

        // ---- user and URL-hash rows: the first 2E columns of X are the two rows end to end.  The common case
        //      (at most 32 chunks) is loaded here and stored after the DFV loads have been issued.
        float4 emb = make_float4(0.f, 0.f, 0.f, 0.f);
        {
            const bool is_url = lane >= ce;
            const int id = is_url ? hid : uid;
            const float* __restrict__ table = is_url ? a.url_emb : a.user_emb;
            if (lane < 2 * ce && id >= 0)
                emb = __ldg(reinterpret_cast<const float4*>(table + (int64_t)id * a.E + (is_url ? lane - ce : lane) * 4));
        }

        // ---- DFV rows, summed in slot order
        float acc[NQ][PER];
#pragma unroll
        for (int q = 0; q < NQ; ++q)
#pragma unroll
            for (int k = 0; k < PER; ++k) acc[q][k] = 0.f;
        int j = 0;
        auto next_ids = [&]() {                                    // IDs 32.. of a long view
            if (j >= 32 && (j & 31) == 0) {
                my_id = load_ids(cur, j);
                if (j + lane < n) {
                    if (my_id < 0 || my_id >= a.img_vocab) { my_id = -1; flags |= GEAR_DEV_BAD_ID; }
                    if (a.row_view) a.row_view[s + j + lane] = b;
                } else my_id = -1;
                clean = !__any_sync(0xffffffffu, j + lane < n && my_id < 0);
            }
        };
        while (n - j >= KMAX) {
            next_ids();
            if (clean) add_rows<TD, NQ, KMAX, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane);
            else add_rows_checked<TD, NQ>(acc, dfv, a.D, n_chunks, my_id, j, KMAX, lane);
            j += KMAX;
        }
        if (KMAX > 1 && j < n) {
            next_ids();
            if (!clean) add_rows_checked<TD, NQ>(acc, dfv, a.D, n_chunks, my_id, j, n - j, lane);
            else switch (n - j) {                                  // 1 .. KMAX - 1 rows left: straight-line code for each count
            case 1: add_rows<TD, NQ, 1, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane); break;
            case 2: if constexpr (KMAX > 2) add_rows<TD, NQ, 2, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane); break;
            case 3: if constexpr (KMAX > 3) add_rows<TD, NQ, 3, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane); break;
            case 4: if constexpr (KMAX > 4) add_rows<TD, NQ, 4, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane); break;
            case 5: if constexpr (KMAX > 5) add_rows<TD, NQ, 5, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane); break;
            case 6: if constexpr (KMAX > 6) add_rows<TD, NQ, 6, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane); break;
            default: if constexpr (KMAX > 7) add_rows<TD, NQ, 7, FULL>(acc, dfv, a.D, n_chunks, my_id, j, lane); break;
            }
        }

        // ---- write the row of X
        if (lane < 2 * ce) {
            const float f[4] = {emb.x, emb.y, emb.z, emb.w};
            store_x<4>(x + lane * 4, f);
            if (xd) store_x<4>(xd + lane * 4, f);
        }
        for (int c = 32 + lane; c < 2 * ce; c += 32) {             // embedding rows wider than 32 chunks in total
            const bool is_url = c >= ce;
            const int id = is_url ? hid : uid;
            const float* __restrict__ table = is_url ? a.url_emb : a.user_emb;
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            if (id >= 0) t = __ldg(reinterpret_cast<const float4*>(table + (int64_t)id * a.E + (is_url ? c - ce : c) * 4));
            const float f[4] = {t.x, t.y, t.z, t.w};
            store_x<4>(x + c * 4, f);
            if (xd) store_x<4>(xd + c * 4, f);
        }
        const float nf = (float)n, rinv = n > 0 ? 1.0f / nf : 0.f;
#pragma unroll
        for (int q = 0; q < NQ; ++q) {
            const int ch = lane + 32 * q;
            if (ch < n_chunks) {
                float o[PER];
#pragma unroll
                for (int k = 0; k < PER; ++k) o[k] = n > 0 ? div_by_count(acc[q][k], nf, rinv) : 0.f;
                store_x<PER>(x + 2 * a.E + ch * PER, o);
                if (xd) store_x<PER>(xd + 2 * a.E + ch * PER, o);
            }
        }
        if (a.inv_n && lane == 0) a.inv_n[b] = rinv;
        // ---- the view's own dense input (the part of the image the Fastgear side keeps), eight columns per lane and pass
        for (int c = lane * 8; c < a.F; c += 256) {
            const float4 f0 = ld_stream_f4(a.fast + (int64_t)b * a.F + c), f1 = ld_stream_f4(a.fast + (int64_t)b * a.F + c + 4);
            const float f[8] = {f0.x, f0.y, f0.z, f0.w, f1.x, f1.y, f1.z, f1.w};
            store_x<8>(x + 2 * a.E + a.D + c, f);
            if (xd) store_x<8>(xd + 2 * a.E + a.D + c, f);
        }

        cur = nxt; nxt = nxt2; ids_cur = ids_nxt;
    }
    if (flags) atomicOr(&a.state->status, flags);
}

template <typename TD, typename TX>
static cudaError_t dispatch_nq(const GatherArgs& a, cudaStream_t st, Profiler* prof) {
    constexpr int PER = Chunk<TD>::PER;
    const int n_chunks = a.D / PER;
    const int nq = (n_chunks + 31) / 32;
    // every block stays resident: three (two for wide rows) per SM
    const int64_t resident = (int64_t)sm_count() * (nq <= 2 ? 3 : 2);
    const int grid = (int)std::min<int64_t>(ceil_div(a.B, GP_WARPS), resident);
    KernelScope ks(prof, "gather_pool", st);
    // FULL only when a row fills the instantiated width exactly (n_chunks == NQ * 32): every lane then owns a chunk of
    // every DFV row; widths that round up to the next instantiation (3, 5, 6, 7 chunks per lane) keep the guard
#define GEAR_GATHER(NQ) do { \
        if (n_chunks == NQ * 32) launch_dependent(gather_pool_kernel<TD, TX, NQ, true>, dim3(grid), dim3(GP_WARPS * 32), 0, st, a); \
        else launch_dependent(gather_pool_kernel<TD, TX, NQ, false>, dim3(grid), dim3(GP_WARPS * 32), 0, st, a); } while (0)
    if (nq <= 1) GEAR_GATHER(1);
    else if (nq <= 2) GEAR_GATHER(2);
    else if (nq <= 4) GEAR_GATHER(4);
    else GEAR_GATHER(8);
#undef GEAR_GATHER
    return cudaGetLastError();
}

cudaError_t launch_gather(const gear_ctx_impl& c, const gear_batch& b, int32_t* row_view, float* inv_n,
                          void* x_debug, cudaStream_t st) {
    if (b.B <= 0) return cudaSuccess;
    GatherArgs a;
    a.user_emb = c.buf.user_emb; a.url_emb = c.buf.url_emb; a.dfv = c.buf.dfv;
    a.user_vocab = c.cfg.user_vocab; a.url_vocab = c.cfg.url_vocab; a.img_vocab = c.cfg.img_vocab;
    a.E = c.cfg.emb_dim; a.D = c.cfg.dfv_dim; a.B = b.B; a.nnz = b.nnz; a.F = c.cfg.fast_dim; a.fast = b.fast;
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
