// The Sparse Part's head (event 4) with fp32 FMA matrix products.
//
// Used for GEAR_F32 heads, where the 1e-5 tolerance rules out tf32/bf16 tensor-core products, and as the
// plain-ALU version of the GEAR_BF16 head (operands rounded to bf16, fp32 accumulation).  One generic
// shared-memory tiled GEMM with strided operands covers the three product shapes of the step:
//   forward        H_l    = ReLU(H_{l-1} W_l + b_l)
//   input gradient dH_{l-1} = (dA_l W_l^T) masked by H_{l-1} > 0
//   weight gradient dW_l  = H_{l-1}^T dA_l           (reduction over the batch, split over blocks)
#include <type_traits>

#include "common.cuh"
#include "internal.h"

namespace gear {

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

enum { EPI_NONE = 0, EPI_BIAS_RELU = 1, EPI_MASK = 2, EPI_ATOMIC = 3 };

constexpr int GT = 64;    // tile edge in M and N
constexpr int GK = 16;    // tile depth

// C[m][n] (+)= epi( sum_k A(m,k) * B(k,n) ),  A(m,k) = A[m*sam + k*sak],  B(k,n) = B[k*sbk + n*sbn].
// blockIdx.z selects a k-range of k_chunk elements (EPI_ATOMIC adds the partial products into C).
template <typename TA, typename TB, typename TC, typename TM, int EPI>
__global__ void __launch_bounds__(256)
gemm_kernel(int M, int N, int K, const TA* __restrict__ A, int64_t sam, int64_t sak,
            const TB* __restrict__ Bm, int64_t sbk, int64_t sbn, TC* __restrict__ C, int64_t ldc,
            const float* __restrict__ bias, const TM* __restrict__ mask, int64_t ldm, int k_chunk) {
    wait_for_predecessor();
    __shared__ float As[GK][GT + 4];
    __shared__ float Bs[GK][GT + 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * GT, n0 = blockIdx.x * GT;
    const int k_begin = blockIdx.z * k_chunk, k_end = min(K, k_begin + k_chunk);
    const bool a_kfast = (sak == 1), b_kfast = (sbk == 1);
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

    for (int k0 = k_begin; k0 < k_end; k0 += GK) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int idx = tid + r * 256;
            int m, k;
            if (a_kfast) { m = idx >> 4; k = idx & 15; } else { k = idx >> 6; m = idx & 63; }
            const int gm = m0 + m, gk = k0 + k;
            As[k][m] = (gm < M && gk < k_end) ? to_f(A[gm * sam + gk * sak]) : 0.f;
            int n, kb;
            if (b_kfast) { n = idx >> 4; kb = idx & 15; } else { kb = idx >> 6; n = idx & 63; }
            const int gn = n0 + n, gkb = k0 + kb;
            Bs[kb][n] = (gn < N && gkb < k_end) ? to_f(Bm[gkb * sbk + gn * sbn]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < GK; ++k) {
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
        const int gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            float v = acc[i][j];
            if (EPI == EPI_BIAS_RELU) v = fmaxf(v + bias[gn], 0.f);
            if (EPI == EPI_MASK) v = to_f(mask[gm * ldm + gn]) > 0.f ? v : 0.f;
            if (EPI == EPI_ATOMIC) atomicAdd(reinterpret_cast<float*>(C) + gm * ldc + gn, v);
            else C[gm * ldc + gn] = from_f<TC>(v);
        }
    }
}

// ---------------------------------------------------------------------------------------------------
// The same product for fp32 operands of at least 128 x 128 outputs: 128 x 128 x 8 tiles, 8 x 8 outputs per
// thread (two 4-wide strips in each direction, 64 apart, so that shared-memory reads are 128-bit and free of
// bank conflicts), operand tiles fetched with 128-bit loads one tile ahead into registers and passed through two
// shared-memory buffers (one __syncthreads per tile).  Either operand may be contiguous along the reduction
// (K_FAST) or along its other index; leading dimensions must be multiples of 4 and the pointers 16-byte
// aligned (the launcher falls back to the 64 x 64 kernel otherwise).  16 FMAs per 128-bit shared-memory read.
// ---------------------------------------------------------------------------------------------------
constexpr int BT = 128;   // tile edge in M and N
constexpr int BK = 8;     // tile depth

// The 128-bit piece of an operand tile that thread `tid` fetches: K_FAST: row (tid / 2) of the tile, reduction
// indices 4 * (tid % 2) .. + 3; else reduction index tid / 32, rows 4 * (tid % 32) .. + 3.  Out-of-range parts are
// zero (whole pieces: the extents are multiples of 4 where it matters, see the launcher).
template <bool K_FAST>
__device__ __forceinline__ float4 fetch_piece(const float* __restrict__ base, int64_t ld, int row0, int rows, int k0,
                                              int k_end, int tid) {
    if (K_FAST) {
        const int r = row0 + (tid >> 1), k = k0 + 4 * (tid & 1);
        if (r < rows && k + 3 < k_end) return __ldg(reinterpret_cast<const float4*>(base + (int64_t)r * ld + k));
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < rows) {
            const float* p = base + (int64_t)r * ld;
            if (k < k_end) v.x = __ldg(p + k);
            if (k + 1 < k_end) v.y = __ldg(p + k + 1);
            if (k + 2 < k_end) v.z = __ldg(p + k + 2);
        }
        return v;
    } else {
        const int k = k0 + (tid >> 5), r = row0 + 4 * (tid & 31);
        if (k < k_end && r + 3 < rows) return __ldg(reinterpret_cast<const float4*>(base + (int64_t)k * ld + r));
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (k < k_end) {
            const float* p = base + (int64_t)k * ld;
            if (r < rows) v.x = __ldg(p + r);
            if (r + 1 < rows) v.y = __ldg(p + r + 1);
            if (r + 2 < rows) v.z = __ldg(p + r + 2);
        }
        return v;
    }
}
// ... and where it goes in the [BK][BT + 4] shared-memory tile
template <bool K_FAST>
__device__ __forceinline__ void stash_piece(float (*tile)[BT + 4], const float4& v, int tid) {
    if (K_FAST) {
        const int r = tid >> 1, k = 4 * (tid & 1);
        tile[k][r] = v.x; tile[k + 1][r] = v.y; tile[k + 2][r] = v.z; tile[k + 3][r] = v.w;
    } else {
        *reinterpret_cast<float4*>(&tile[tid >> 5][4 * (tid & 31)]) = v;
    }
}

// C[m][n] (+)= epi( sum_k A(m,k) B(k,n) ).  A_KFAST: A(m,k) = A[m * lda + k], else A[k * lda + m];
// B_KFAST: B(k,n) = B[n * ldb + k], else B[k * ldb + n].  blockIdx.z selects a k-range of k_chunk elements.
template <bool A_KFAST, bool B_KFAST, int EPI>
__global__ void __launch_bounds__(256, 2)
gemm128_kernel(int M, int N, int K, const float* __restrict__ A, int64_t lda, const float* __restrict__ Bm, int64_t ldb,
               float* __restrict__ C, int64_t ldc, const float* __restrict__ bias, const float* __restrict__ mask,
               int64_t ldm, int k_chunk) {
    wait_for_predecessor();
    __shared__ __align__(16) float As[2][BK][BT + 4];
    __shared__ __align__(16) float Bs[2][BK][BT + 4];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * BT, n0 = blockIdx.x * BT;
    const int k_begin = blockIdx.z * k_chunk, k_end = min(K, k_begin + k_chunk);
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = 0.f;

    float4 pa = fetch_piece<A_KFAST>(A, lda, m0, M, k_begin, k_end, tid);
    float4 pb = fetch_piece<B_KFAST>(Bm, ldb, n0, N, k_begin, k_end, tid);
    stash_piece<A_KFAST>(As[0], pa, tid);
    stash_piece<B_KFAST>(Bs[0], pb, tid);
    __syncthreads();
    int buf = 0;
    for (int k0 = k_begin; k0 < k_end; k0 += BK) {
        const bool more = k0 + BK < k_end;
        if (more) {                                               // the next tile travels while this one is used
            pa = fetch_piece<A_KFAST>(A, lda, m0, M, k0 + BK, k_end, tid);
            pb = fetch_piece<B_KFAST>(Bm, ldb, n0, N, k0 + BK, k_end, tid);
        }
#pragma unroll
        for (int k = 0; k < BK; ++k) {
            const float4 a0 = *reinterpret_cast<const float4*>(&As[buf][k][ty * 4]);
            const float4 a1 = *reinterpret_cast<const float4*>(&As[buf][k][64 + ty * 4]);
            const float4 b0 = *reinterpret_cast<const float4*>(&Bs[buf][k][tx * 4]);
            const float4 b1 = *reinterpret_cast<const float4*>(&Bs[buf][k][64 + tx * 4]);
            const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (more) {
            stash_piece<A_KFAST>(As[buf ^ 1], pa, tid);           // the other buffer: nobody reads it during this tile
            stash_piece<B_KFAST>(Bs[buf ^ 1], pb, tid);
            __syncthreads();
            buf ^= 1;
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int gm = m0 + (i < 4 ? ty * 4 + i : 64 + ty * 4 + i - 4);
        if (gm >= M) continue;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int gn = n0 + 64 * h + tx * 4;
            if (gn >= N) continue;                                // N is a multiple of 4 here: whole 4-wide strips
            float v[4] = {acc[i][4 * h], acc[i][4 * h + 1], acc[i][4 * h + 2], acc[i][4 * h + 3]};
            if (EPI == EPI_BIAS_RELU) {
                const float4 bb = __ldg(reinterpret_cast<const float4*>(bias + gn));
                v[0] = fmaxf(v[0] + bb.x, 0.f); v[1] = fmaxf(v[1] + bb.y, 0.f);
                v[2] = fmaxf(v[2] + bb.z, 0.f); v[3] = fmaxf(v[3] + bb.w, 0.f);
            }
            if (EPI == EPI_MASK) {
                const float4 mm = __ldg(reinterpret_cast<const float4*>(mask + (int64_t)gm * ldm + gn));
                v[0] = mm.x > 0.f ? v[0] : 0.f; v[1] = mm.y > 0.f ? v[1] : 0.f;
                v[2] = mm.z > 0.f ? v[2] : 0.f; v[3] = mm.w > 0.f ? v[3] : 0.f;
            }
            float* dst = C + (int64_t)gm * ldc + gn;
            if (EPI == EPI_ATOMIC) red_add_f4(dst, make_float4(v[0], v[1], v[2], v[3]));
            else st_f4(dst, make_float4(v[0], v[1], v[2], v[3]));
        }
    }
}

static bool ptr16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Tries the 128 x 128 kernel; false if the shapes, strides or alignments do not fit it.
template <int EPI>
static bool try_gemm128(int M, int N, int K, const float* A, int64_t sam, int64_t sak, const float* B, int64_t sbk,
                        int64_t sbn, float* C, int64_t ldc, const float* bias, const float* mask, int64_t ldm, int splits,
                        cudaStream_t st) {
    if (M < 96 || N < 96 || (N & 3) || (ldc & 3) || !ptr16(C) || !ptr16(A) || !ptr16(B)) return false;
    const bool a_kfast = sak == 1, b_kfast = sbk == 1;
    if (!a_kfast && sam != 1) return false;
    if (!b_kfast && sbn != 1) return false;
    const int64_t lda = a_kfast ? sam : sak, ldb = b_kfast ? sbn : sbk;
    if ((lda & 3) || (ldb & 3)) return false;
    if (EPI == EPI_BIAS_RELU && !ptr16(bias)) return false;
    if (EPI == EPI_MASK && ((ldm & 3) || !ptr16(mask))) return false;
    // as many slices of the reduction as fill the GPU twice over (two blocks per SM), each a multiple of the tile depth
    const int64_t tiles = ceil_div(M, BT) * ceil_div(N, BT);
    int64_t s = splits > 1 ? ceil_div(2 * sm_count(), tiles) : 1;
    const int64_t max_s = ceil_div(K, 256);
    if (s > max_s) s = max_s;
    if (s < 1) s = 1;
    const int k_chunk = (int)ceil_div(ceil_div(K, s), BK) * BK;
    const dim3 grid((unsigned)ceil_div(N, BT), (unsigned)ceil_div(M, BT), (unsigned)ceil_div(K, k_chunk));
#define GEAR_G128(AK, BKF) launch_dependent(gemm128_kernel<AK, BKF, EPI>, grid, dim3(256), 0, st, M, N, K, A, lda, B, ldb, C, ldc, bias, mask, ldm, k_chunk)
    if (a_kfast && !b_kfast) GEAR_G128(true, false);
    else if (!a_kfast && !b_kfast) GEAR_G128(false, false);
    else if (a_kfast && b_kfast) GEAR_G128(true, true);
    else GEAR_G128(false, true);
#undef GEAR_G128
    return true;
}

template <typename TA, typename TB, typename TC, typename TM, int EPI>
static void launch_gemm(int M, int N, int K, const TA* A, int64_t sam, int64_t sak, const TB* B, int64_t sbk,
                        int64_t sbn, TC* C, int64_t ldc, const float* bias, const TM* mask, int64_t ldm,
                        int splits, cudaStream_t st, Profiler* prof, const char* name) {
    if (M <= 0 || N <= 0 || K <= 0) return;
    KernelScope ks(prof, name, st);
    if constexpr (std::is_same<TA, float>::value && std::is_same<TB, float>::value && std::is_same<TC, float>::value &&
                  std::is_same<TM, float>::value) {
        if (try_gemm128<EPI>(M, N, K, A, sam, sak, B, sbk, sbn, C, ldc, bias, mask, ldm, splits, st)) return;
    }
    int k_chunk = (int)ceil_div(ceil_div(K, splits), GK) * GK;
    splits = (int)ceil_div(K, k_chunk);
    dim3 grid((unsigned)ceil_div(N, GT), (unsigned)ceil_div(M, GT), (unsigned)splits);
    launch_dependent(gemm_kernel<TA, TB, TC, TM, EPI>, grid, dim3(256), 0, st, M, N, K, A, sam, sak, B, sbk, sbn, C, ldc, bias, mask,
                                                          ldm, k_chunk);
}

// 8 consecutive activations as floats (one 16-byte load for bf16, two for fp32)
__device__ __forceinline__ void load8(const float* p, float* v) {
    const float4 a = ld_f4(p), b = ld_f4(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float* v) {
    const uint4 t = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) { v[2 * k] = __uint_as_float(w[k] << 16); v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
}
// stores 8 values in the head dtype and returns them as stored (rounded for bf16)
__device__ __forceinline__ void store8(float* p, float* v) {
    st_f4(p, make_float4(v[0], v[1], v[2], v[3]));
    st_f4(p + 4, make_float4(v[4], v[5], v[6], v[7]));
}
__device__ __forceinline__ void store8(__nv_bfloat16* p, float* v) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
        w[k] = *reinterpret_cast<uint32_t*>(&h2);
        v[2 * k] = __uint_as_float(w[k] << 16);
        v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

// Eight consecutive activations as they sit in memory (kept in registers between the two passes over a row).
template <typename TX> struct Raw8;
template <> struct Raw8<float> {
    float4 a, b;
    __device__ __forceinline__ void load(const float* p) { a = ld_f4(p); b = ld_f4(p + 4); }
    __device__ __forceinline__ void clear() { a = b = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ void unpack(float* v) const {
        v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
    }
};
template <> struct Raw8<__nv_bfloat16> {
    uint4 t;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { t = *reinterpret_cast<const uint4*>(p); }
    __device__ __forceinline__ void clear() { t = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ void unpack(float* v) const {
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) { v[2 * k] = __uint_as_float(w[k] << 16); v[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u); }
    }
};

// Output unit, loss and everything that hangs off the top hidden layer:
//   z = h . w_out + b_out;  p = sigmoid(z);  BCE in its overflow-safe form;  dz = (p - y) / B
//   dA_top[b][j] = dz * w_out[j] where h[b][j] > 0, else 0            (stored in the head dtype)
//   gw_out[j] += sum_b h[b][j] dz[b];  gb_top[j] += sum_b dA_top[b][j];  gb_out += sum_b dz[b]
// A warp takes ROWS views at a time; a lane owns NQ = ceil(H / 256) chunks of 8 columns (128-bit loads and stores)
// and keeps its part of the ROWS rows in registers, so the top activations are read once.  The ROWS dot products
// are reduced together (a shuffle transpose-reduction: lane l ends up with the sum of row l >> (5 - log2 ROWS)),
// and sigmoid, loss and dz of the ROWS views are then worked out side by side, one view per group of lanes.
template <typename TX, int NQ, int ROWS>
__global__ void __launch_bounds__(256, NQ == 4 ? 1 : 2)
head_out_kernel(int B, int H, const TX* __restrict__ h, const float* __restrict__ w_out,
                const float* __restrict__ b_out, const float* __restrict__ label, float* __restrict__ prob,
                float* __restrict__ dz, TX* __restrict__ dA, float* __restrict__ loss_part,
                float* __restrict__ gw_out, float* __restrict__ gb_top, float* __restrict__ gb_out,
                unsigned int* __restrict__ ticket, float* __restrict__ loss) {
    wait_for_predecessor();
    constexpr int LG = ROWS == 8 ? 3 : ROWS == 4 ? 2 : ROWS == 2 ? 1 : 0;
    static_assert((1 << LG) == ROWS, "ROWS is 1, 2, 4 or 8");
    __shared__ float part[8], gpart[8];
    __shared__ float s_gw[1024], s_gb[1024];
    const unsigned lane = lane_id(), warp = threadIdx.x >> 5;
    for (int j = threadIdx.x; j < H; j += 256) { s_gw[j] = 0.f; s_gb[j] = 0.f; }
    float w[NQ][8], gw[NQ][8], gb[NQ][8];
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const int c0 = (lane + 32 * q) * 8;
#pragma unroll
        for (int k = 0; k < 8; ++k) { w[q][k] = c0 < H ? w_out[c0 + k] : 0.f; gw[q][k] = 0.f; gb[q][k] = 0.f; }
    }
    float local = 0.f, gsum = 0.f;
    const float bias = b_out[0];
    const int my_row = (int)(lane >> (5 - LG));            // the row of a batch whose sum this lane ends up with
    const bool my_first = (lane & ((32u >> LG) - 1u)) == 0u;   // one lane per row records the row's scalars
    __syncthreads();
    for (int b0 = (blockIdx.x * 8 + warp) * ROWS; b0 < B; b0 += gridDim.x * 8 * ROWS) {
        Raw8<TX> raw[ROWS][NQ];
        // the label of this lane's view: asked for first, so that its latency passes while the rows are summed
        const float y = b0 + my_row < B ? __ldg(label + b0 + my_row) : 0.f;
#pragma unroll
        for (int j = 0; j < ROWS; ++j)
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int c0 = (lane + 32 * q) * 8;
                if (b0 + j < B && c0 < H) raw[j][q].load(h + (int64_t)(b0 + j) * H + c0);
                else raw[j][q].clear();
            }
        float z[ROWS];
#pragma unroll
        for (int j = 0; j < ROWS; ++j) {
            z[j] = 0.f;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                float v[8];
                raw[j][q].unpack(v);
#pragma unroll
                for (int k = 0; k < 8; ++k) z[j] = fmaf(v[k], w[q][k], z[j]);
            }
        }
        // rows still held: ROWS, ROWS / 2, ..., 1; each round hands half of them to the lane 16, 8, 4 away
#pragma unroll
        for (int r = 0; r < LG; ++r) {
            const int s = 16 >> r, half = ROWS >> (r + 1);
            const bool upper = (lane & s) != 0;
#pragma unroll
            for (int i = 0; i < half; ++i) {
                const float send = upper ? z[i] : z[i + half];
                const float keep = upper ? z[i + half] : z[i];
                z[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
            }
        }
        float zz = z[0];
#pragma unroll
        for (int s = 16 >> LG; s >= 1; s >>= 1) zz += __shfl_xor_sync(0xffffffffu, zz, s);
        zz += bias;
        const int b = b0 + my_row;
        const bool live = b < B;
        const float p = 1.0f / (1.0f + expf(-zz));
        const float g = live ? (p - y) / (float)B : 0.f;
        if (live && my_first) {
            local += fmaxf(zz, 0.f) - zz * y + log1pf(expf(-fabsf(zz)));
            gsum += g;
            if (prob) prob[b] = p;
            dz[b] = g;
        }
#pragma unroll
        for (int j = 0; j < ROWS; ++j) {
            const float gj = __shfl_sync(0xffffffffu, g, j << (5 - LG));
            if (b0 + j >= B) continue;                        // warp-uniform
            TX* drow = dA + (int64_t)(b0 + j) * H;
#pragma unroll
            for (int q = 0; q < NQ; ++q) {
                const int c0 = (lane + 32 * q) * 8;
                if (c0 >= H) continue;
                float v[8], d[8];
                raw[j][q].unpack(v);
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    gw[q][k] = fmaf(v[k], gj, gw[q][k]);
                    d[k] = v[k] > 0.f ? gj * w[q][k] : 0.f;
                }
                store8(drow + c0, d);
#pragma unroll
                for (int k = 0; k < 8; ++k) gb[q][k] += d[k];
            }
        }
    }
#pragma unroll
    for (int q = 0; q < NQ; ++q) {
        const int c0 = (lane + 32 * q) * 8;
        if (c0 >= H) continue;
#pragma unroll
        for (int k = 0; k < 8; ++k) { atomicAdd(&s_gw[c0 + k], gw[q][k]); atomicAdd(&s_gb[c0 + k], gb[q][k]); }
    }
    local = warp_sum(local);                 // one lane per row of a batch held that row's terms
    gsum = warp_sum(gsum);
    if (lane == 0) { part[warp] = local; gpart[warp] = gsum; }
    __syncthreads();
    for (int j = threadIdx.x; j < H; j += 256) { atomicAdd(gw_out + j, s_gw[j]); atomicAdd(gb_top + j, s_gb[j]); }
    if (threadIdx.x == 0) {
        float s = 0.f, t = 0.f;
        for (int k = 0; k < 8; ++k) { s += part[k]; t += gpart[k]; }
        loss_part[blockIdx.x] = s;
        atomicAdd(gb_out, t);
    }
    // The block that delivers its partial loss last adds them all up, always in block order (the ticket counts
    // arrivals and wraps back to zero by itself, ready for the next launch).
    __shared__ int is_last;
    if (threadIdx.x == 0) {
        __threadfence();
        is_last = atomicInc(ticket, gridDim.x - 1) == gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    float s = 0.f;
    for (int i = threadIdx.x; i < (int)gridDim.x; i += 256) s += __ldcg(loss_part + i);
    s = warp_sum(s);
    __syncthreads();
    if (lane == 0) part[warp] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int k = 0; k < 8; ++k) t += part[k];
        loss[0] = B > 0 ? t / (float)B : 0.f;
    }
}

// out[n] += sum_b A[b][n]: bias gradient of a lower hidden layer.  A block of 256 threads sums its own range of
// rows: thread t owns the 8 columns of chunk t % (N/8) (128-bit loads) and every (256 / (N/8))-th row, four loads
// in flight.  Each block adds its partial sums to the output with one atomic per column.
template <typename TA>
__global__ void __launch_bounds__(256)
colsum_kernel(int B, int N, const TA* __restrict__ A, float* __restrict__ out) {
    wait_for_predecessor();
    __shared__ float s[1024];
    const int tpr = N / 8, rpp = 256 / tpr;
    const int chunk = threadIdx.x % tpr, rsub = threadIdx.x / tpr;
    const int rows_per_block = (int)ceil_div(B, gridDim.x);
    const int b0 = blockIdx.x * rows_per_block, b1 = min(B, b0 + rows_per_block);
    for (int j = threadIdx.x; j < N; j += 256) s[j] = 0.f;
    __syncthreads();
    if (rsub < rpp) {
        float acc[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) acc[k] = 0.f;
        for (int b = b0 + rsub; b < b1; b += 4 * rpp) {
            float v[4][8];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                if (b + r * rpp < b1) load8(A + (int64_t)(b + r * rpp) * N + chunk * 8, v[r]);
                else {
#pragma unroll
                    for (int k = 0; k < 8; ++k) v[r][k] = 0.f;
                }
            }
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int k = 0; k < 8; ++k) acc[k] += v[r][k];
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) atomicAdd(&s[chunk * 8 + k], acc[k]);
    }
    __syncthreads();
    for (int j = threadIdx.x; j < N; j += 256) atomicAdd(out + j, s[j]);
}

// fp32 master weights -> bf16 in both orientations, all hidden layers in one launch (blockIdx.y = layer)
struct RoundArgs {
    int fan_in[MAX_LAYERS], fan_out[MAX_LAYERS];
    const float* W[MAX_LAYERS];
    __nv_bfloat16* wb[MAX_LAYERS];
    __nv_bfloat16* wbt[MAX_LAYERS];
};
// 32 x 32 tiles through shared memory, so that both copies are written with coalesced rows
__global__ void __launch_bounds__(256)
round_weights_kernel(const RoundArgs a) {
    wait_for_predecessor();
    __shared__ __nv_bfloat16 tile[32][33];
    const int l = blockIdx.z;
    const int fan_in = a.fan_in[l], fan_out = a.fan_out[l];
    const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    if (r0 >= fan_in || c0 >= fan_out) return;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int r = r0 + ty + 8 * k, c = c0 + tx;
        if (r < fan_in && c < fan_out) {
            const __nv_bfloat16 v = __float2bfloat16_rn(a.W[l][(int64_t)r * fan_out + c]);
            a.wb[l][(int64_t)r * fan_out + c] = v;
            tile[ty + 8 * k][tx] = v;
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int c = c0 + ty + 8 * k, r = r0 + tx;
        if (r < fan_in && c < fan_out) a.wbt[l][(int64_t)c * fan_in + r] = tile[tx][ty + 8 * k];
    }
}

struct HeadParams {
    const float* W[MAX_LAYERS]; const float* b[MAX_LAYERS];
    float* gW[MAX_LAYERS]; float* gb[MAX_LAYERS];
    const float* w_out; const float* b_out; float* gw_out; float* gb_out;
    int fan[MAX_LAYERS + 1];
};

static HeadParams split_params(const gear_ctx_impl& c, float* grad) {
    HeadParams p;
    const float* base = c.buf.head_params;
    int64_t pos = 0;
    p.fan[0] = c.d_in;
    for (int l = 0; l < c.cfg.n_hidden; ++l) {
        const int h = c.cfg.hidden[l];
        p.W[l] = base + pos; p.gW[l] = grad + pos; pos += (int64_t)p.fan[l] * h;
        p.b[l] = base + pos; p.gb[l] = grad + pos; pos += h;
        p.fan[l + 1] = h;
    }
    p.w_out = base + pos; p.gw_out = grad + pos; pos += p.fan[c.cfg.n_hidden];
    p.b_out = base + pos; p.gb_out = grad + pos;
    return p;
}

static int splits_for(int M, int N, int K) {
    const int64_t tiles = ceil_div(M, GT) * ceil_div(N, GT);
    int64_t s = ceil_div(148 * 4, tiles);
    const int64_t max_s = ceil_div(K, 256);
    if (s > max_s) s = max_s;
    return (int)(s < 1 ? 1 : s);
}

// bf16 copies of the hidden layers' weights in both orientations (what the tensor-core products read).  Depends on
// head_params only, so a step runs it ahead of the gather.
cudaError_t launch_round_weights(const gear_ctx_impl& c, cudaStream_t st) {
    if (c.cfg.head_dtype != GEAR_BF16) return cudaSuccess;
    const int L = c.cfg.n_hidden;
    RoundArgs ra;
    int max_in = 0, max_out = 0, fan = c.d_in;
    int64_t pos = 0;
    for (int l = 0; l < L; ++l) {
        const int h = c.cfg.hidden[l];
        ra.fan_in[l] = fan; ra.fan_out[l] = h; ra.W[l] = c.buf.head_params + pos;
        ra.wb[l] = c.at<__nv_bfloat16>(c.ws.wb[l]); ra.wbt[l] = c.at<__nv_bfloat16>(c.ws.wbt[l]);
        if (fan > max_in) max_in = fan;
        if (h > max_out) max_out = h;
        pos += (int64_t)fan * h + h;
        fan = h;
    }
    KernelScope ks(&c.prof, "round_weights", st);
    return launch_dependent(round_weights_kernel, dim3((unsigned)ceil_div(max_out, 32), (unsigned)ceil_div(max_in, 32), (unsigned)L),
                            dim3(256), 0, st, ra);
}

template <typename TX>
static cudaError_t run_head(const gear_ctx_impl& c, const gear_batch& bt, const gear_step_out& o, cudaStream_t st,
                            const HeadHooks& hooks) {
    constexpr bool BF = !std::is_same<TX, float>::value;
    const int L = c.cfg.n_hidden, B = bt.B;
    HeadParams p = split_params(c, o.head_grad);
    cudaError_t err = cudaMemsetAsync(o.head_grad, 0, sizeof(float) * c.n_params, st);
    if (err != cudaSuccess) return err;
    if (B <= 0) return cudaMemsetAsync(o.loss, 0, sizeof(float), st);

    TX* H[MAX_LAYERS + 1];
    TX* dA[MAX_LAYERS + 1];
    H[0] = c.at<TX>(c.ws.x);
    dA[0] = nullptr;
    for (int l = 0; l < L; ++l) { H[l + 1] = c.at<TX>(c.ws.h[l]); dA[l + 1] = c.at<TX>(c.ws.da[l]); }
    float* dz = c.at<float>(c.ws.dz);
    float* loss_part = c.at<float>(c.ws.loss_part);

    // weights as the products see them
    const void* Wop[MAX_LAYERS];
    if (BF) {
        for (int l = 0; l < L; ++l) Wop[l] = c.at<__nv_bfloat16>(c.ws.wb[l]);
        if (!hooks.weights_ready) {
            cudaError_t re = launch_round_weights(c, st);
            if (re != cudaSuccess) return re;
        }
    } else {
        for (int l = 0; l < L; ++l) Wop[l] = p.W[l];
    }
    int32_t* tc_err = &c.state()->tc_error;
    cudaError_t tce = cudaSuccess;
    // forward
    for (int l = 0; l < L; ++l) {
        const int K = p.fan[l], N = p.fan[l + 1];
        if constexpr (BF) {
            tce = tc_gemm_kmajor(&c.prof, "tc_gemm_fwd", B, N, K, H[l], K, c.at<__nv_bfloat16>(c.ws.wbt[l]), K, 0,
                                 H[l + 1], N, p.b[l], nullptr, 0, nullptr, tc_err, st);
            if (tce != cudaSuccess) return tce;
        } else
        launch_gemm<TX, TX, TX, TX, EPI_BIAS_RELU>(B, N, K, H[l], K, 1, static_cast<const TX*>(Wop[l]), N, 1,
                                                    H[l + 1], N, p.b[l], (const TX*)nullptr, 0, 1, st, &c.prof,
                                                    "simt_gemm_fwd");
    }
    const int HT = p.fan[L];
    {
        KernelScope ks(&c.prof, "head_out", st);
        const int nq = (int)ceil_div(HT, 256);
        // rows per warp and pass: as many as the registers hold (8 chunks of bf16, 4 of fp32)
        constexpr int RMAX = BF ? 8 : 4;
        const int rows = nq <= 1 ? RMAX : nq == 2 ? RMAX / 4 : 1;
        // every warp gets the same number of passes where the batch allows it
        const int64_t batches = ceil_div(B, rows);
        const int64_t passes = ceil_div(batches, (int64_t)c.ws.loss_blocks * 8);
        const int blocks = (int)ceil_div(batches, 8 * passes);
#define GEAR_HEAD_OUT(NQ, ROWS) launch_dependent(head_out_kernel<TX, NQ, ROWS>, dim3(blocks), dim3(256), 0, st, B, HT, H[L], p.w_out, p.b_out, bt.label, \
        o.prob, dz, dA[L], loss_part, p.gw_out, p.gb[L - 1], p.gb_out, &c.state()->colsum_ticket, o.loss)
        if (nq <= 1) GEAR_HEAD_OUT(1, RMAX);
        else if (nq == 2) GEAR_HEAD_OUT(2, RMAX / 4);
        else GEAR_HEAD_OUT(4, 1);
#undef GEAR_HEAD_OUT
    }
    // backward.  Per layer the gradient that the layers below wait for (dA_l, at the bottom dX) comes first, its weight
    // gradient after it: once dX exists the caller's hook may start the embedding scatter on another stream, beside the
    // last weight-gradient product.
    for (int l = L - 1; l >= 0; --l) {
        const int K = p.fan[l], N = p.fan[l + 1];
        // bias gradient of a lower layer (the top layer's came out of head_out_kernel); the tensor-core path
        // sums the columns of dA inside the epilogue of the product that makes dA
        if (!BF && l < L - 1) {
            KernelScope ks(&c.prof, "colsum", st);
            const int blocks = B < CS_BLOCKS * 8 ? (int)ceil_div(B, 8) : CS_BLOCKS;
            launch_dependent(colsum_kernel<TX>, dim3(blocks), dim3(256), 0, st, B, N, dA[l + 1], p.gb[l]);
        }
        if constexpr (BF) {
            const __nv_bfloat16* wb = c.at<__nv_bfloat16>(c.ws.wb[l]);
            if (l > 0) tce = tc_gemm_kmajor(&c.prof, "tc_gemm_dh", B, K, N, dA[l + 1], N, wb, N, 1, dA[l], K, nullptr,
                                            H[l], K, p.gb[l - 1], tc_err, st);
            else tce = tc_gemm_kmajor(&c.prof, "tc_gemm_dx", B, K, N, dA[l + 1], N, wb, N, 2, o.dX, K, nullptr, nullptr,
                                      0, nullptr, tc_err, st);
            if (tce != cudaSuccess) return tce;
        } else if (l > 0) {
            launch_gemm<TX, TX, TX, TX, EPI_MASK>(B, K, N, dA[l + 1], N, 1, static_cast<const TX*>(Wop[l]), 1, N,
                                                  dA[l], K, nullptr, H[l], K, 1, st, &c.prof, "simt_gemm_dh");
        } else {
            launch_gemm<TX, TX, float, TX, EPI_NONE>(B, K, N, dA[l + 1], N, 1, static_cast<const TX*>(Wop[l]), 1, N,
                                                     o.dX, K, nullptr, (const TX*)nullptr, 0, 1, st, &c.prof, "simt_gemm_dx");
        }
        if (l == 0 && hooks.after_dx) {
            cudaError_t he = hooks.after_dx(hooks.arg);
            if (he != cudaSuccess) return he;
        }
        // dW_l = H_l^T dA_{l+1}
        if constexpr (BF) {
            tce = tc_gemm_mnmajor(&c.prof, "tc_gemm_dw", K, N, B, H[l], K, dA[l + 1], N, p.gW[l], N, tc_err, st);
            if (tce != cudaSuccess) return tce;
        } else
        launch_gemm<TX, TX, float, TX, EPI_ATOMIC>(K, N, B, H[l], 1, K, dA[l + 1], N, 1, p.gW[l], N, nullptr,
                                                   (const TX*)nullptr, 0, splits_for(K, N, B), st, &c.prof, "simt_gemm_dw");
    }
    return cudaGetLastError();
}

cudaError_t launch_head_simt(const gear_ctx_impl& c, const gear_batch& b, const gear_step_out& o, cudaStream_t st,
                             const HeadHooks& hooks) {
    if (c.cfg.head_dtype == GEAR_BF16) return run_head<__nv_bfloat16>(c, b, o, st, hooks);
    return run_head<float>(c, b, o, st, hooks);
}

}  // namespace gear
