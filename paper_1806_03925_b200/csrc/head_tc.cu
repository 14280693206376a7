// bf16 matrix products of the head on the 5th-generation tensor cores (sm_100a):
// tcgen05.mma with fp32 accumulators in tensor memory, operands staged in shared memory by TMA.
//
// One persistent kernel, one CTA per SM, three roles:
//   warp 0     TMA producer: streams 128 x 64 (A) and BN x 64 (B) bf16 tiles through a ring of
//              shared-memory stages (128-byte swizzle), one mbarrier pair per stage;
//   warp 1     MMA issuer: one elected lane issues tcgen05.mma (M 128, N BN, K 16) into one of two
//              accumulator buffers in tensor memory and commits each stage back to the producer;
//   warps 2-9  epilogue: tcgen05.ld the finished accumulator (32 lanes x 32 columns per instruction),
//              apply bias+ReLU / ReLU mask / nothing, and store; meanwhile the MMA warp already fills
//              the other accumulator buffer with the next tile.  Two warps share each quarter of the
//              tensor-memory lanes and split the tile's columns; the read of the next 32 columns and
//              the loads of the bias are in flight while the current 32 columns are processed; the ReLU
//              mask of a 32 x 32 block arrives by TMA, requested two blocks ahead of its use.
//              The ReLU-mask epilogue also sums its output columns (the bias gradient of the layer
//              below): each lane adds up two columns of the block staged for the store; per-CTA partials
//              in shared memory.
// Two operand layouts:
//   K-major   C[M][N] = A[M][K] . W[N][K]^T     (activations x weights; K contiguous in both)
//   MN-major  C[M][N] += A[K][M]^T . B[K][N]    (weight gradients: the reduction runs over the batch,
//                                                split across CTAs; a CTA's partial tile leaves like any
//                                                fp32 output, in 32 x 32 blocks through shared memory, but
//                                                as a TMA reduction: the copy engine adds it to the matrix)
// No cluster launch and no multicast.  Every wait is bounded: on a timeout the kernel records an error
// code, leaves its loops, frees its tensor memory and returns.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "internal.h"

namespace gear {

constexpr int TC_BM = 128;
constexpr int TC_BK = 64;                 // 64 bf16 = 128 bytes = one swizzle row
// Epilogue warps per CTA (a multiple of four: each warp reaches one quarter of the tensor-memory lanes).
constexpr int tc_threads(int ew) { return 64 + 32 * ew; }
constexpr int TC_MAX_N = 1024;            // widest output the column-sum partials cover
constexpr int TC_MASK_BLOCK = 32 * 64;    // a warp's ReLU-mask block for 32 columns: 32 rows of 64 bytes (two per warp)
constexpr uint32_t TC_SPIN_LIMIT = 1u << 22;

enum { TC_EPI_BIAS_RELU = 0, TC_EPI_MASK = 1, TC_EPI_F32 = 2, TC_EPI_RED = 3 };

constexpr int TC_OUT_BLOCK = 32 * 128;   // a warp's output block on its way to a TMA store: 32 rows of 128 bytes

template <int BN, int EW, int EPI> struct TcCfg {
    static constexpr int A_BYTES = TC_BM * TC_BK * 2;            // 16 KB
    static constexpr int B_BYTES = BN * TC_BK * 2;               // 32 KB or 16 KB
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int OUT_BYTES = EW * TC_OUT_BLOCK;       // one output block per epilogue warp
    static constexpr int MASK_BYTES = EPI == TC_EPI_MASK ? EW * 2 * TC_MASK_BLOCK : 0;
    static constexpr int COLSUM_BYTES = EPI == TC_EPI_MASK ? TC_MAX_N * 4 : 0;     // per-CTA column sums of the masked product
    static constexpr int FIXED = 1024 /*alignment slack*/ + 512 /*barriers*/ + COLSUM_BYTES + OUT_BYTES + MASK_BYTES;
    static constexpr int ROOM = (227 * 1024 - FIXED) / STAGE_BYTES;
    static constexpr int STAGES = ROOM > (BN == 256 ? 4 : 6) ? (BN == 256 ? 4 : 6) : ROOM;
    static constexpr int SMEM = STAGES * STAGE_BYTES + FIXED;
    static constexpr int TMEM_COLS = BN == 192 ? 512 : 2 * BN;   // two accumulator buffers (a power of two is allocated)
    static_assert(STAGES >= 3, "operand ring too short");
    static_assert(SMEM > 116 * 1024, "one CTA per SM: two CTAs would both ask for tensor memory");
    static_assert(SMEM <= 227 * 1024, "shared memory budget");
};

struct TcArgs {
    int M, N, K;              // output rows, output columns, reduction length
    int m_tiles, n_tiles, k_splits, kb_per_split;   // kb = blocks of TC_BK along K
    void* out; int64_t ldo;
    const float* bias;
    const __nv_bfloat16* mask; int64_t ldm;
    float* colsum;            // ReLU-mask epilogue: colsum[n] += sum over rows of the stored output (may be null)
    int32_t* err;             // device word that receives a non-zero code on a timeout
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
// Arrival that orders nothing but the barrier itself: the epilogue hands its accumulator buffer back with this one,
// so that the hand-over does not wait for the tile's global stores to drain (tensor-memory reads are complete by
// then: tcgen05.wait::ld, then tcgen05.fence::before_thread_sync).
__device__ __forceinline__ void mbar_arrive_relaxed(uint32_t bar) {
    asm volatile("mbarrier.arrive.relaxed.cta.shared::cta.b64 _, [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and records `code`) if the phase never completed.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int32_t* err, int code) {
    for (uint32_t i = 0; i < TC_SPIN_LIMIT; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i > 64) __nanosleep(32);
        if ((i & 1023u) == 1023u && *reinterpret_cast<volatile int32_t*>(err) != 0) return false;
    }
    atomicCAS(err, 0, code);
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 :: "r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y) : "memory");
}

// Store of a shared-memory box (128-byte swizzle) into the output matrix; parts of the box past the matrix edge are
// dropped by the copy engine.  Bulk groups belong to the issuing thread: the same lane commits and waits.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
                 :: "l"(map), "r"(src), "r"(x), "r"(y) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// The same with an L2 eviction policy for the lines written.
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* map, uint32_t src, int x, int y, uint64_t policy) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;"
                 :: "l"(map), "r"(src), "r"(x), "r"(y), "l"(policy) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// The same box added to the matrix instead of stored (fp32 adds by the copy engine, whole rows of the box at a time).
__device__ __forceinline__ void tma_reduce_add_2d(const CUtensorMap* map, uint32_t src, int x, int y) {
    asm volatile("cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3}], [%1];"
                 :: "l"(map), "r"(src), "r"(x), "r"(y) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int PENDING>
__device__ __forceinline__ void tma_store_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" :: "n"(PENDING) : "memory");
}
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void sts_u4(uint32_t addr, const uint4& v) {
    asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" :: "r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\t"
                 "setp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(taddr) : "memory");
}
// Waits for the tensor-memory reads issued so far.  The registers are passed through so that no use of
// them can be scheduled ahead of the wait.
__device__ __forceinline__ void tc_wait_ld(uint32_t (&r)[32]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :: "memory");
}

__device__ __forceinline__ float4 ldg_f4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ uint4 ldg_u4(const void* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }

// Shared-memory matrix descriptor, 128-byte swizzle, sm_100 format (version 1).
//   K-major operand : rows of 128 bytes, 8-row groups 1024 bytes apart (SBO); LBO unused.
//   MN-major operand: 64-element (128-byte) slabs along M/N, `lbo` bytes apart; 8-deep K groups 1024 bytes apart.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3ffffu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
    d |= (uint64_t)1 << 46;            // descriptor version
    d |= (uint64_t)2 << 61;            // SWIZZLE_128B
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = BN.
__host__ __device__ constexpr uint32_t instr_desc(int bn, bool mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((mn_major ? 1u : 0u) << 15) | ((mn_major ? 1u : 0u) << 16) |
           ((uint32_t)(bn >> 3) << 17) | ((uint32_t)(TC_BM >> 4) << 24);
}

// Epilogue of one finished accumulator buffer `a`, as run by one of the epilogue warps: warp w reads
// tensor-memory lanes 32 * (w % 4) .. + 31 (its rows of the tile); the EW / 4 warps of a lane quarter split the
// tile's columns evenly (warps 2..5 take the first share, 6..9 the second, ...).
//
// Output leaves through the copy engine: a lane owns a row of the accumulator, so it writes its row's 128 bytes
// (64 bf16 or 32 fp32 columns) into a 32-row block in shared memory, 16-byte pieces XOR-swizzled by the row number
// (conflict-free 128-bit writes, and the layout a 128-byte-swizzle tensor map expects); one lane then hands the
// block to a TMA store, which writes whole rows of it, drops what lies past the matrix edge and needs no register
// or issue slot of the warp while it runs.  `out_buf` is the shared-memory address of this warp's block(s).
// The ReLU mask of a warp's 32 x 32 blocks travels by TMA, two blocks ahead of their use: block c goes to the warp's
// half-buffer c % 2 (32 rows of 64 bytes, 64-byte swizzle) and reports to that half's mbarrier; as soon as the lanes
// have read a half, the block two further on (of this tile or the next) is requested into it.
struct MaskPipe {
    const CUtensorMap* map;
    uint32_t buf, bar;         // shared-memory addresses of the warp's two half-buffers / two mbarriers
    uint32_t parity;           // bit h: phase the next wait on half h looks for
    uint32_t pending;          // bit h: a copy into half h has been issued and not yet waited for
    int next_m0, next_col0;    // first row / column of this warp's part of the CTA's next tile (-1: there is none)
};
__device__ __forceinline__ void mask_request(MaskPipe& mp, int h, int x, int y, int lane) {
    __syncwarp();                                             // every lane has read the half's previous contents
    if (lane == 0) {
        fence_async_smem();
        const uint32_t bar = mp.bar + 8u * h;
        mbar_expect_tx(bar, TC_MASK_BLOCK);
        tma_load_2d(mp.buf + (uint32_t)h * TC_MASK_BLOCK, mp.map, bar, x, y);
    }
    mp.pending |= 1u << h;
}

template <int BN, int EPI, int EW>
__device__ __forceinline__ void epilogue_tile(const TcArgs& g, const CUtensorMap* map_out, uint32_t tmem_base, int a, int mt,
                                              int nt, int warp, int lane, float* s_colsum, MaskPipe& mp, uint32_t out_buf,
                                              uint64_t keep_policy) {
    const int quarter = warp & 3;
    const int part = (warp - 2) >> 2;
    constexpr int COLS = BN / (EW / 4);                   // columns per warp and tile
    constexpr int CHUNKS = COLS / 32;                     // 32-column chunks per warp and tile
    static_assert(EPI == TC_EPI_F32 || EPI == TC_EPI_RED || CHUNKS % 2 == 0, "bf16 output leaves in blocks of 64 columns");
    const int m0 = mt * TC_BM + quarter * 32;         // first row of this warp's block
    const int m = m0 + lane;
    const int rows = min(32, max(0, g.M - m0));
    const int col0 = nt * BN + part * COLS;
    const uint32_t t_row = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(a * BN + part * COLS);
    const uint32_t swz = (uint32_t)(lane & 7);
    uint32_t r[2][32];
    tc_ld32(t_row, r[0]);
#pragma unroll
    for (int c = 0; c < CHUNKS; ++c) {
        const int n0 = col0 + c * 32;
        const bool chunk_ok = n0 < g.N;               // warp-uniform; N is a multiple of 8
        // what this chunk's epilogue reads from memory, requested while the tensor-memory read is in flight
        float4 bias4[EPI == TC_EPI_BIAS_RELU ? 8 : 1];
        uint4 mask4[EPI == TC_EPI_MASK ? 4 : 1];
        if (EPI == TC_EPI_BIAS_RELU) {
#pragma unroll
            for (int j = 0; j < 8; ++j)
                bias4[j] = (n0 + 4 * j < g.N) ? ldg_f4(g.bias + n0 + 4 * j) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        tc_wait_ld(r[c & 1]);
        if (c + 1 < CHUNKS) tc_ld32(t_row + (uint32_t)((c + 1) * 32), r[(c + 1) & 1]);
        if (EPI == TC_EPI_MASK) {
            // this block's mask has been on its way since two blocks ago; a lane reads its own row (rows and columns past
            // the matrix edge arrive as zeros), then the half is free for the block two further on
            const int h = c & 1;
            mbar_wait(mp.bar + 8u * h, (mp.parity >> h) & 1u, g.err, 6);
            mp.parity ^= 1u << h;
            mp.pending &= ~(1u << h);
            const uint32_t row_addr = mp.buf + (uint32_t)h * TC_MASK_BLOCK + (uint32_t)lane * 64u;
            const uint32_t sw = ((uint32_t)lane >> 1) & 3u;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(mask4[j].x), "=r"(mask4[j].y), "=r"(mask4[j].z), "=r"(mask4[j].w)
                             : "r"(row_addr + ((((uint32_t)j) ^ sw) << 4)) : "memory");
            if (c + 2 < CHUNKS) mask_request(mp, h, n0 + 64, m0, lane);
            else if (mp.next_m0 >= 0) mask_request(mp, h, mp.next_col0 + (c + 2 - CHUNKS) * 32, mp.next_m0, lane);
        }
        if (!chunk_ok || rows == 0) continue;
        uint32_t (&acc)[32] = r[c & 1];
        if (EPI == TC_EPI_BIAS_RELU || EPI == TC_EPI_MASK) {
            uint32_t pk[16];
            if (EPI == TC_EPI_BIAS_RELU) {
                float v[32];
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(acc[i]);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    v[4 * j + 0] = fmaxf(v[4 * j + 0] + bias4[j].x, 0.f);
                    v[4 * j + 1] = fmaxf(v[4 * j + 1] + bias4[j].y, 0.f);
                    v[4 * j + 2] = fmaxf(v[4 * j + 2] + bias4[j].z, 0.f);
                    v[4 * j + 3] = fmaxf(v[4 * j + 3] + bias4[j].w, 0.f);
                }
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * q], v[2 * q + 1]);
                    pk[q] = *reinterpret_cast<uint32_t*>(&h2);
                }
            } else {
                // two columns at a time: round the pair, then clear the halves whose activation was not positive (a
                // packed compare of the two activations against zero gives all-ones per passing half)
                const __nv_bfloat162 zero2 = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t w[4] = {mask4[j].x, mask4[j].y, mask4[j].z, mask4[j].w};
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        __nv_bfloat162 h2 = __floats2bfloat162_rn(__uint_as_float(acc[8 * j + 2 * q]), __uint_as_float(acc[8 * j + 2 * q + 1]));
                        const unsigned int keep = __hgt2_mask(*reinterpret_cast<const __nv_bfloat162*>(&w[q]), zero2);
                        pk[4 * j + q] = *reinterpret_cast<uint32_t*>(&h2) & keep;
                    }
                }
            }
            {
                // chunks 2k and 2k+1 fill the left and right half of one 64-column block
                const int half = c & 1;
                const uint32_t row_addr = out_buf + (uint32_t)lane * 128u;
                if (half == 0) {
                    if (lane == 0) tma_store_wait_read<0>();          // the block's previous contents have been read
                    __syncwarp();
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    sts_u4(row_addr + ((((uint32_t)(4 * half + j)) ^ swz) << 4),
                           make_uint4(pk[4 * j], pk[4 * j + 1], pk[4 * j + 2], pk[4 * j + 3]));
                if (half == 1 || n0 + 32 >= g.N) {
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) tma_store_2d(map_out, out_buf, n0 - 32 * half, m0);
                    if (EPI == TC_EPI_MASK && g.colsum != nullptr) {
                        // column sums of what was stored (the rounded values), read back from the block: lane l owns
                        // columns 2l and 2l + 1 of the 64, one word per row (rows past M hold zeros: their operand rows
                        // and mask were read as zeros)
                        const int nb = n0 - 32 * half + 2 * lane;
                        float s_lo = 0.f, s_hi = 0.f;
#pragma unroll
                        for (int rr = 0; rr < 32; ++rr) {
                            uint32_t wv;
                            const uint32_t addr = out_buf + (uint32_t)rr * 128u + ((((uint32_t)lane >> 2) ^ (uint32_t)(rr & 7)) << 4) +
                                                  (((uint32_t)lane & 3u) << 2);
                            asm volatile("ld.shared.b32 %0, [%1];" : "=r"(wv) : "r"(addr) : "memory");
                            s_lo += __uint_as_float(wv << 16);
                            s_hi += __uint_as_float(wv & 0xffff0000u);
                        }
                        if (nb < g.N) { atomicAdd(&s_colsum[nb], s_lo); atomicAdd(&s_colsum[nb + 1], s_hi); }
                    }
                }
            }
        } else {
            // fp32 output (dX): one block per 32 columns; it is read again right
            // after (embedding and DFV gradients): ask the L2 to keep it
            const uint32_t buf = out_buf;
            if (lane == 0) tma_store_wait_read<0>();                  // the block's previous contents have been read
            __syncwarp();
            const uint32_t row_addr = buf + (uint32_t)lane * 128u;
#pragma unroll
            for (int j = 0; j < 8; ++j)
                sts_u4(row_addr + (((uint32_t)j ^ swz) << 4), make_uint4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]));
            fence_async_smem();
            __syncwarp();
            if (lane == 0) {
                // a slice's partial tile of a weight gradient is added to the matrix by the copy engine
                if (EPI == TC_EPI_RED) tma_reduce_add_2d(map_out, buf, n0, m0);
                else tma_store_2d_hint(map_out, buf, n0, m0, keep_policy);
            }
        }
    }
}

// ---------------------------------------------------------------- the kernel
template <int BN, bool MN_MAJOR, int EPI, int EW>
__device__ __forceinline__ void tc_gemm_body(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_out,
                                             const CUtensorMap& map_mask, const TcArgs& g) {
    using Cfg = TcCfg<BN, EW, EPI>;
    constexpr int STAGES = Cfg::STAGES;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;                  // operand stages, 1024-byte aligned
    const uint32_t out_blocks = tiles + STAGES * Cfg::STAGE_BYTES;  // output blocks of the epilogue warps, 1024-byte aligned
    const uint32_t mask_blocks = out_blocks + Cfg::OUT_BYTES;       // ReLU-mask blocks of the epilogue warps, 1024-byte aligned
    const uint32_t bars = mask_blocks + Cfg::MASK_BYTES;            // mbarriers, then the tmem address word
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
    auto acc_full = [&](int a) { return bars + 8u * (2 * STAGES + a); };
    auto acc_empty = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
    const uint32_t tmem_word = bars + 8u * (2 * STAGES + 4);
    volatile uint32_t* tmem_word_ptr =
        reinterpret_cast<volatile uint32_t*>(smem_raw + (tmem_word - raw));
    auto mask_bar = [&](int w, int h) { return bars + 8u * (24 + 2 * w + h); };     // two per epilogue warp
    float* s_colsum = reinterpret_cast<float*>(smem_raw + (bars + 512u - raw));     // [TC_MAX_N] per-CTA column sums

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total_tiles = g.m_tiles * g.n_tiles * g.k_splits;
    const int total_kb = (g.K + TC_BK - 1) / TC_BK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(acc_full(a), 1); mbar_init(acc_empty(a), 32 * EW); }
        if (EPI == TC_EPI_MASK)
            for (int w = 0; w < EW; ++w) { mbar_init(mask_bar(w, 0), 1); mbar_init(mask_bar(w, 1), 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" :: "l"(&map_a) : "memory");
        asm volatile("prefetch.tensormap [%0];" :: "l"(&map_b) : "memory");
        asm volatile("prefetch.tensormap [%0];" :: "l"(&map_out) : "memory");
        if (EPI == TC_EPI_MASK) asm volatile("prefetch.tensormap [%0];" :: "l"(&map_mask) : "memory");
    }
    if (EPI == TC_EPI_MASK && g.colsum != nullptr)
        for (int n = threadIdx.x; n < TC_MAX_N; n += tc_threads(EW)) s_colsum[n] = 0.f;
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(tmem_word), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_word_ptr;
    wait_for_predecessor();      // barriers, tensor memory and descriptors are set up while the previous kernel drains

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                // column tiles of one row tile are neighbours in the order: CTAs that run side by side read the same rows of A,
                // which then come from memory once
                const int nt = t % g.n_tiles, mt = (t / g.n_tiles) % g.m_tiles, ks = t / (g.m_tiles * g.n_tiles);
                const int kb0 = ks * g.kb_per_split, kb1 = min(total_kb, kb0 + g.kb_per_split);
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!(ok = mbar_wait(empty_bar(s), ((it / STAGES) & 1u) ^ 1u, g.err, 1))) break;
                    const uint32_t a_dst = tiles + s * Cfg::STAGE_BYTES, b_dst = a_dst + Cfg::A_BYTES;
                    mbar_expect_tx(full_bar(s), Cfg::STAGE_BYTES);
                    if (!MN_MAJOR) {
                        tma_load_2d(a_dst, &map_a, full_bar(s), kb * TC_BK, mt * TC_BM);     // 128 rows x 64 k
                        tma_load_2d(b_dst, &map_b, full_bar(s), kb * TC_BK, nt * BN);        // BN rows x 64 k
                    } else {
                        // 64 k-rows x 64 columns per box; the slabs of one operand sit 8 KB apart
#pragma unroll
                        for (int j = 0; j < TC_BM / 64; ++j)
                            tma_load_2d(a_dst + j * 8192, &map_a, full_bar(s), mt * TC_BM + j * 64, kb * TC_BK);
#pragma unroll
                        for (int j = 0; j < BN / 64; ++j)
                            tma_load_2d(b_dst + j * 8192, &map_b, full_bar(s), nt * BN + j * 64, kb * TC_BK);
                    }
                }
            }
            if (*reinterpret_cast<volatile int32_t*>(g.err) != 0) {
                // leaving early: let the copies already issued land before the CTA gives its shared memory back
                const uint32_t first = it > (uint32_t)STAGES ? it - STAGES : 0u;
                for (uint32_t j = first; j < it; ++j)
                    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try(full_bar(j % STAGES), (j / STAGES) & 1u); ++spin)
                        __nanosleep(64);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(BN, MN_MAJOR);
            uint32_t it = 0, tile_it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tile_it) {
                const int ks = t / (g.m_tiles * g.n_tiles);
                const int kb0 = ks * g.kb_per_split, kb1 = min(total_kb, kb0 + g.kb_per_split);
                const int a = tile_it & 1;
                if (!(ok = mbar_wait(acc_empty(a), ((tile_it >> 1) & 1u) ^ 1u, g.err, 2))) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * BN);
                for (int kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = it % STAGES;
                    if (!(ok = mbar_wait(full_bar(s), (it / STAGES) & 1u, g.err, 3))) break;
                    tc_fence_after();
                    const uint32_t a_src = tiles + s * Cfg::STAGE_BYTES, b_src = a_src + Cfg::A_BYTES;
#pragma unroll
                    for (int k = 0; k < TC_BK / 16; ++k) {
                        uint64_t da, db;
                        if (!MN_MAJOR) {
                            da = smem_desc(a_src + k * 32, 16, 1024);
                            db = smem_desc(b_src + k * 32, 16, 1024);
                        } else {
                            da = smem_desc(a_src + k * 2048, 8192, 1024);
                            db = smem_desc(b_src + k * 2048, 8192, 1024);
                        }
                        tc_mma(d_tmem, da, db, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                    }
                    tc_commit(empty_bar(s));            // the stage may be refilled once these MMAs have read it
                }
                if (ok) tc_commit(acc_full(a));          // accumulator complete
            }
        }
    } else {
        // ---------------- epilogue warps
        const uint32_t out_buf = out_blocks + (uint32_t)((warp - 2) * TC_OUT_BLOCK);
        const uint64_t keep_policy = l2_policy_evict_last();
        uint32_t tile_it = 0;
        bool ok = true;
        constexpr int COLS = BN / (EW / 4);
        // where this warp's part of tile t starts
        auto part_m0 = [&](int t) { return ((t / g.n_tiles) % g.m_tiles) * TC_BM + (warp & 3) * 32; };
        auto part_col0 = [&](int t) { return (t % g.n_tiles) * BN + ((warp - 2) >> 2) * COLS; };
        MaskPipe mp{&map_mask, mask_blocks + (uint32_t)((warp - 2) * 2 * TC_MASK_BLOCK), mask_bar(warp - 2, 0), 0u, 0u, -1, -1};
        if (EPI == TC_EPI_MASK && (int)blockIdx.x < total_tiles) {
            // the masks of the first tile's first two blocks (after the wait for the previous kernel, which wrote them)
            mask_request(mp, 0, part_col0(blockIdx.x), part_m0(blockIdx.x), lane);
            mask_request(mp, 1, part_col0(blockIdx.x) + 32, part_m0(blockIdx.x), lane);
        }
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++tile_it) {
            const int nt = t % g.n_tiles, mt = (t / g.n_tiles) % g.m_tiles;
            const int a = tile_it & 1;
            if (EPI == TC_EPI_MASK) {
                const int tn = t + (int)gridDim.x;
                mp.next_m0 = tn < total_tiles ? part_m0(tn) : -1;
                mp.next_col0 = tn < total_tiles ? part_col0(tn) : -1;
            }
            if (!(ok = mbar_wait(acc_full(a), (tile_it >> 1) & 1u, g.err, 4))) break;
            tc_fence_after();
            epilogue_tile<BN, EPI, EW>(g, &map_out, tmem_base, a, mt, nt, warp, lane, s_colsum, mp, out_buf, keep_policy);
            tc_fence_before();
            mbar_arrive_relaxed(acc_empty(a));                   // all epilogue threads arrive: the buffer returns to the MMA warp
        }
        if (lane == 0) tma_store_wait_all();   // this warp's stores have left shared memory and landed
        if (EPI == TC_EPI_MASK && mp.pending) {
            // leaving early: let the mask copies already issued land before the CTA gives its shared memory back
            for (int h = 0; h < 2; ++h)
                if (mp.pending & (1u << h))
                    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_try(mp.bar + 8u * h, (mp.parity >> h) & 1u); ++spin)
                        __nanosleep(64);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (EPI == TC_EPI_MASK && g.colsum != nullptr)
        for (int n = threadIdx.x; n < g.N && n < TC_MAX_N; n += tc_threads(EW)) {
            const float v = s_colsum[n];
            if (v != 0.f) atomicAdd(g.colsum + n, v);
        }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;"
                     :: "r"(tmem_base), "r"((uint32_t)Cfg::TMEM_COLS) : "memory");
    }
}

// Eight epilogue warps, at most 128 registers per thread: a CTA (320 threads) then fits on an SM beside a block of
// the ID sort.  One CTA per SM follows from the shared-memory footprint.
template <int BN, bool MN_MAJOR, int EPI>
__global__ void __maxnreg__(128)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_out, const __grid_constant__ CUtensorMap map_mask, const TcArgs g) {
    tc_gemm_body<BN, MN_MAJOR, EPI, 8>(map_a, map_b, map_out, map_mask, g);
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// A step encodes the same eighteen maps every time (operands and outputs live at fixed places in the workspace): a
// small table of the most recent encodings saves the driver calls.  A map depends on the key alone.
struct MapKey { const void* ptr; int64_t rows, cols, ld; int box_rows, f32; };
struct MapCache {
    static constexpr int N = 64;
    std::mutex mu;
    MapKey key[N];
    CUtensorMap map[N];
    int used = 0, next = 0;
    bool find(const MapKey& k, CUtensorMap* out) {
        std::lock_guard<std::mutex> lock(mu);
        for (int i = 0; i < used; ++i)
            if (key[i].ptr == k.ptr && key[i].rows == k.rows && key[i].cols == k.cols && key[i].ld == k.ld &&
                key[i].box_rows == k.box_rows && key[i].f32 == k.f32) { *out = map[i]; return true; }
        return false;
    }
    void put(const MapKey& k, const CUtensorMap& m) {
        std::lock_guard<std::mutex> lock(mu);
        const int i = used < N ? used++ : (next = (next + 1) % N);
        key[i] = k; map[i] = m;
    }
};
static MapCache g_maps;

static bool make_map_f32(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows);
static bool encode_bf16(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows);

// bf16 matrix [rows][cols] with leading dimension ld (elements); box = box_rows x 64 columns, 128-byte swizzle.
// Out-of-range parts of a box read as zero.
static bool make_map(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    const MapKey k{ptr, rows, cols, ld, box_rows, 0};
    if (g_maps.find(k, m)) return true;
    if (!encode_bf16(m, ptr, rows, cols, ld, box_rows)) return false;
    g_maps.put(k, *m);
    return true;
}
static bool encode_bf16(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 matrix [rows][cols] with leading dimension ld (elements); box = box_rows x 32 columns, 128-byte swizzle.
static bool make_map_f32(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    const MapKey k{ptr, rows, cols, ld, box_rows, 1};
    if (g_maps.find(k, m)) return true;
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 4};
    cuuint32_t box[2] = {32, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    if (fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return false;
    g_maps.put(k, *m);
    return true;
}

// bf16 matrix [rows][cols] read in boxes of 32 rows x 32 columns (64 bytes a row), 64-byte swizzle: the ReLU mask.
static bool make_map_mask(CUtensorMap* m, const void* ptr, int64_t rows, int64_t cols, int64_t ld) {
    const MapKey k{ptr, rows, cols, ld, 32, 2};
    if (g_maps.find(k, m)) return true;
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    if (fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) return false;
    g_maps.put(k, *m);
    return true;
}

template <int BN, bool MN, int EPI, int EW>
static cudaError_t launch_variant(const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mo, const CUtensorMap& mm,
                                  const TcArgs& g, cudaStream_t st) {
    using Cfg = TcCfg<BN, EW, EPI>;
    static_assert(EW == 8, "one kernel entry point: eight epilogue warps");
    auto kernel = tc_gemm_kernel<BN, MN, EPI>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::SMEM);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const int tiles = g.m_tiles * g.n_tiles * g.k_splits;
    const int grid = tiles < sm_count() ? tiles : sm_count();
    return launch_dependent(kernel, dim3(grid), dim3(tc_threads(EW)), (size_t)Cfg::SMEM, st, ma, mb, mo, mm, g);
}

template <bool MN, int EPI, int EW = 8>
static cudaError_t launch_bn(int bn, const CUtensorMap& ma, const CUtensorMap& mb, const CUtensorMap& mo, const CUtensorMap& mm,
                             const TcArgs& g, cudaStream_t st) {
    return bn == 256 ? launch_variant<256, MN, EPI, EW>(ma, mb, mo, mm, g, st)
                     : launch_variant<128, MN, EPI, EW>(ma, mb, mo, mm, g, st);
}

cudaError_t tc_gemm_kmajor(Profiler* prof, const char* name, int M, int N, int K, const __nv_bfloat16* A, int64_t lda,
                           const __nv_bfloat16* W, int64_t ldw, int epi, void* out, int64_t ldo, const float* bias,
                           const __nv_bfloat16* mask, int64_t ldm, float* colsum, int32_t* err, cudaStream_t st) {
    if (M <= 0 || N <= 0 || K <= 0) return cudaSuccess;
    // column tiles of 256 or 128; the fp32 output (dX) also has 192, which fits a width like 384 without a half-empty tile
    int bn = N > 128 ? 256 : 128;
    if (epi == TC_EPI_F32 && N > 128 && ceil_div(N, 192) * 192 < ceil_div(N, 256) * 256) bn = 192;
    CUtensorMap ma, mb, mo;
    if (!make_map(&ma, A, M, K, lda, TC_BM) || !make_map(&mb, W, N, K, ldw, bn)) return cudaErrorInvalidValue;
    // the output leaves in boxes of 32 rows x 128 bytes
    if (!(epi == TC_EPI_F32 ? make_map_f32(&mo, out, M, N, ldo, 32) : make_map(&mo, out, M, N, ldo, 32))) return cudaErrorInvalidValue;
    TcArgs g;
    g.M = M; g.N = N; g.K = K;
    g.m_tiles = (int)ceil_div(M, TC_BM); g.n_tiles = (int)ceil_div(N, bn); g.k_splits = 1;
    g.kb_per_split = (int)ceil_div(K, TC_BK);
    g.out = out; g.ldo = ldo; g.bias = bias; g.mask = mask; g.ldm = ldm; g.err = err;
    g.colsum = (epi == TC_EPI_MASK && N <= TC_MAX_N) ? colsum : nullptr;
    if (epi == TC_EPI_MASK && colsum != nullptr && g.colsum == nullptr) return cudaErrorInvalidValue;
    KernelScope ks(prof, name, st);
    switch (epi) {
    case TC_EPI_BIAS_RELU: return launch_bn<false, TC_EPI_BIAS_RELU>(bn, ma, mb, mo, ma /*unused*/, g, st);
    case TC_EPI_MASK: {
        CUtensorMap mm;
        if (!mask || !make_map_mask(&mm, mask, M, N, ldm)) return cudaErrorInvalidValue;
        return launch_bn<false, TC_EPI_MASK>(bn, ma, mb, mo, mm, g, st);
    }
    default:
        if (bn == 192) return launch_variant<192, false, TC_EPI_F32, 8>(ma, mb, mo, ma /*unused*/, g, st);
        return launch_bn<false, TC_EPI_F32>(bn, ma, mb, mo, ma /*unused*/, g, st);
    }
}

cudaError_t tc_gemm_mnmajor(Profiler* prof, const char* name, int M, int N, int K, const __nv_bfloat16* A, int64_t lda,
                            const __nv_bfloat16* Bm, int64_t ldb, float* out, int64_t ldo, int32_t* err,
                            cudaStream_t st) {
    if (M <= 0 || N <= 0 || K <= 0) return cudaSuccess;
    const int bn = N > 128 ? 256 : 128;
    CUtensorMap ma, mb, mo;
    if (!make_map(&ma, A, K, M, lda, 64) || !make_map(&mb, Bm, K, N, ldb, 64) || !make_map_f32(&mo, out, M, N, ldo, 32))
        return cudaErrorInvalidValue;
    TcArgs g;
    g.M = M; g.N = N; g.K = K;
    g.m_tiles = (int)ceil_div(M, TC_BM); g.n_tiles = (int)ceil_div(N, bn);
    const int total_kb = (int)ceil_div(K, TC_BK);
    // as many slices of the reduction as fit in one wave of CTAs (one more would leave a second, nearly empty wave)
    int splits = sm_count() / (g.m_tiles * g.n_tiles);
    if (splits > total_kb) splits = total_kb;
    if (splits < 1) splits = 1;
    g.kb_per_split = (int)ceil_div(total_kb, splits);
    g.k_splits = (int)ceil_div(total_kb, g.kb_per_split);
    g.out = out; g.ldo = ldo; g.bias = nullptr; g.mask = nullptr; g.ldm = 0; g.colsum = nullptr; g.err = err;
    KernelScope ks(prof, name, st);
    return launch_bn<true, TC_EPI_RED>(bn, ma, mb, mo, ma /*unused*/, g, st);
}

}  // namespace gear
