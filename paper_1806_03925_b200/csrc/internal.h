// Host-side internals of libgear: the ctx, the workspace plan and the launch functions each .cu exports.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/gear.h"
#include "common.cuh"

namespace gear {

constexpr int EXP_TILE = 8192;     // entries of the timestamp table per block of the expiry scan's write pass
constexpr int EXP_MARK_TILE = 2048; // ... and per block (and per count) of its mark pass
constexpr int MAX_LAYERS = 2;
constexpr int CS_BLOCKS = 296;      // blocks of the column-sum kernel (two per SM)

// Byte offsets into the caller's workspace.  Everything is 256-byte aligned.
struct WsPlan {
    size_t state;                       // DevState
    size_t x;                           // [max_batch][d_in]      head dtype: head input
    size_t h[MAX_LAYERS];               // [max_batch][hidden[l]] head dtype: post-ReLU activations
    size_t da[MAX_LAYERS];              // [max_batch][hidden[l]] head dtype: gradient at the pre-activation
    size_t dz;                          // [max_batch] fp32
    size_t loss_part;                   // [loss_blocks] fp32 per-block partial losses
    size_t colsum_part;                 // [CS_BLOCKS][1024] fp32 per-block partial column sums
    size_t wb[MAX_LAYERS];              // bf16 head: W_l as [in][out]
    size_t wbt[MAX_LAYERS];             // bf16 head: W_l as [out][in]
    // four sets of sort buffers: user IDs, URL IDs (max_batch each), image IDs (max_nnz), ready queue (ready_cap)
    size_t sort_keys[4][2], sort_vals[4][2];
    size_t sort_hist[4], sort_tot[4];
    int64_t sort_n[4];
    size_t tile_cnt;                    // [sort tiles + 1] uint2 per-tile (groups, complete) counts
    size_t grp_rec;                     // [max_nnz] uint4 group records (start | first flag, image ID, queue slot, held rows)
    size_t blk_first;                   // [ceil(max_nnz / 16) + 2] uint32: first group that starts in each span of sorted positions
    size_t run_end;                     // [max_nnz] uint32: at the first position of an image's run, one past its last
    size_t pmeta;                       // [max_nnz] int2: source row and scale (fp32 bits) of every sorted position
    size_t q_id;                        // [ready_cap] int32
    size_t q_avg;                       // [ready_cap][dfv_dim] fp32
    size_t emb_gsum[2];                 // [max_batch][emb_dim] fp32 per table: summed gradient of every distinct ID of the
                                        // batch, in the row of the sorted position where the ID's run starts (Adam only)
    size_t exp_bits;                    // [ceil(img_vocab / 32)] uint32 expired bitmap
    size_t exp_cnt;                     // [expiry mark tiles + 1] uint2
    size_t total;
    int64_t ready_cap;
    int loss_blocks;
};

int plan_workspace(const gear_config& c, WsPlan* p);

struct gear_ctx_impl {
    gear_config cfg;
    gear_buffers buf;
    WsPlan ws;
    int d_in;
    int64_t n_params;
    cudaStream_t last_stream;
    // streams the calls were enqueued on (the expiry scan and the refresh may sit on streams of their own); the
    // calls that wait for the ctx's work wait for all of them
    static constexpr int MAX_STREAMS = 4;
    cudaStream_t seen_stream[MAX_STREAMS] = {};
    int n_seen = 0;
    void note_stream(cudaStream_t st) {
        for (int i = 0; i < n_seen; ++i) if (seen_stream[i] == st) return;
        if (n_seen < MAX_STREAMS) seen_stream[n_seen++] = st;
        else { cudaStreamSynchronize(seen_stream[0]); seen_stream[0] = st; }     // a fifth stream: retire the oldest
    }
    bool alive;
    void* tc_state;     // tensor-core head state (tensor maps), owned by head_tc.cu; may be null
    cudaStream_t side_stream;          // runs the ID sort of a step beside the gather and the head
    cudaEvent_t ev_fork, ev_join;
    mutable Profiler prof;
    mutable GridBarrierState gbs;
    // image IDs of the last gear_forward_backward batch, already sorted (reused by gear_accumulate_dfv_grad)
    const int32_t* last_img_id;         // img_id array of that batch (the atomic mode reads it unsorted)
    bool img_sorted;
    int64_t img_sorted_n;
    mutable int img_sorted_buf;
    mutable bool img_sort_valid;        // the sort buffers still hold that batch's order (an accumulate call with
                                        // explicit IDs sorts into the same buffers)
    // accumulate plan made ahead by gear_forward_backward (valid for exactly these arguments)
    mutable bool plan_ready;
    mutable int64_t plan_n;
    mutable const int32_t* plan_src_row;
    mutable const float* plan_scale;
    cudaEvent_t ev_gather;              // the gather's outputs (row_view, inv_n) exist
    cudaEvent_t ev_dx;                  // dX exists: the embedding scatter may start on the side stream
    mutable int acc_calls_pending;      // accumulate calls enqueued since a collect that was sure to drain the queue

    template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(static_cast<char*>(buf.workspace) + off); }
    DevState* state() const { return at<DevState>(ws.state); }
    enum { SORT_USER = 0, SORT_URL = 1, SORT_IMG = 2, SORT_READY = 3 };
    // a job over buffer set `which`; the caller fills ids / n / bits
    SortJob sort_job(int which) const {
        SortJob j{};
        j.keys[0] = at<uint32_t>(ws.sort_keys[which][0]); j.keys[1] = at<uint32_t>(ws.sort_keys[which][1]);
        j.vals[0] = at<uint32_t>(ws.sort_vals[which][0]); j.vals[1] = at<uint32_t>(ws.sort_vals[which][1]);
        j.hist = at<uint32_t>(ws.sort_hist[which]); j.tot = at<uint32_t>(ws.sort_tot[which]);
        j.sentinel = 0xffffffffu;
        j.status = &state()->status;
        j.identity_vals = 1;
        return j;
    }
    SortBatch sort_batch() const {
        SortBatch b{};
        b.err = &state()->tc_error;
        return b;
    }
};

// fill.cu
cudaError_t launch_fill_uniform(void* dst, int dtype, int64_t n_elems, uint64_t seed, uint64_t tag, double amp,
                                cudaStream_t st);
cudaError_t launch_fill_ts(int64_t* ts, int64_t n, uint64_t seed, int64_t expire, int64_t now, cudaStream_t st);

// gather.cu
cudaError_t launch_gather(const gear_ctx_impl& c, const gear_batch& b, int32_t* row_view, float* inv_n,
                          void* x_debug, cudaStream_t st);

// head_simt.cu: forward + backward of the head (fp32 FMA products, or the tensor-core products of head_tc.cu).
// weights_ready: the bf16 copies of the weights have been made already (launch_round_weights earlier on the same stream).  after_dx(arg) is called once dX has been enqueued, before the last weight-gradient product.
struct HeadHooks { bool weights_ready; cudaError_t (*after_dx)(void*); void* arg; };
cudaError_t launch_head_simt(const gear_ctx_impl& c, const gear_batch& b, const gear_step_out& o, cudaStream_t st,
                             const HeadHooks& hooks);
cudaError_t launch_round_weights(const gear_ctx_impl& c, cudaStream_t st);

// head_tc.cu: bf16 products on tcgen05 tensor cores.  epi: 0 bias+ReLU -> bf16, 1 ReLU mask -> bf16, 2 plain fp32.
// colsum (epi 1 only, may be null): colsum[n] += sum over the rows of the stored (rounded) output.
cudaError_t tc_gemm_kmajor(Profiler* prof, const char* name, int M, int N, int K, const __nv_bfloat16* A, int64_t lda,
                           const __nv_bfloat16* W, int64_t ldw, int epi, void* out, int64_t ldo, const float* bias,
                           const __nv_bfloat16* mask, int64_t ldm, float* colsum, int32_t* err, cudaStream_t st);
// out[M][N] (fp32) += A[K][M]^T . Bm[K][N]
cudaError_t tc_gemm_mnmajor(Profiler* prof, const char* name, int M, int N, int K, const __nv_bfloat16* A, int64_t lda,
                            const __nv_bfloat16* Bm, int64_t ldb, float* out, int64_t ldo, int32_t* err,
                            cudaStream_t st);

// emb_scatter.cu
// table[id] += alpha * (sum of the dX rows of the views with that id) for the user and the URL-hash table, given the
// sorted (id, view) pairs of buffer sets SORT_USER / SORT_URL
cudaError_t launch_emb_reduce(const gear_ctx_impl& c, int buf, int32_t B, float* user_table, float* url_table,
                              const float* dX, int ldx, float alpha, cudaStream_t st);

// dense.cu: a linear Dense Part (DFV = raw row . Wd) and Adam
struct EmbAdamTable { const uint32_t* ks; uint32_t vocab; float* table; float* m; float* v; const float* gsum; };
cudaError_t launch_dense_forward(const gear_ctx_impl& c, const float* raw, int R, const float* Wd, const int32_t* ids,
                                 int64_t n, const int64_t* d_n, float* rows, int64_t ld, cudaStream_t st);
cudaError_t launch_dense_backward(const gear_ctx_impl& c, const float* raw, int R, const int32_t* ids, const float* avg,
                                  int64_t ld_avg, int64_t n, const int64_t* d_n, float* G, cudaStream_t st);
cudaError_t launch_adam_dense(Profiler* prof, float* p, const float* g, float* m, float* v, int64_t n, int64_t t,
                              const gear_adam& cfg, cudaStream_t st);
cudaError_t launch_emb_adam_rows(const gear_ctx_impl& c, const EmbAdamTable& t0, const EmbAdamTable& t1, int32_t B,
                                 int64_t t, const gear_adam& cfg, cudaStream_t st);
// emb_scatter.cu: Adam on the embedding rows the batch touched (per-ID sums into compact buffers, then the row steps)
cudaError_t launch_emb_adam(const gear_ctx_impl& c, int buf, int32_t B, const float* dX, int ldx, const gear_adam& cfg,
                            int64_t t, float* user_m, float* user_v, float* url_m, float* url_v, cudaStream_t st);

// shard.cu: row fetch for a table shard's owner; event 5's gradient rows in materialised form
cudaError_t launch_fetch_rows(const gear_ctx_impl& c, int which, const int32_t* ids, int64_t n, void* out, cudaStream_t st);
cudaError_t launch_dfv_grad_rows(const gear_ctx_impl& c, const float* dX, const int32_t* row_view, const float* inv_n,
                                 int64_t nnz, float* out, cudaStream_t st);
// emb_scatter.cu: table[id] += alpha * (sum of the rows with that id), ids given explicitly (sorted here)
cudaError_t launch_apply_emb_grad(const gear_ctx_impl& c, int which, const int32_t* ids, const float* rows, int64_t ld,
                                  int64_t n, float alpha, cudaStream_t st);

// accumulate.cu
// img_id == nullptr: use the image IDs sorted by the last gear_forward_backward (buffer set SORT_IMG)
cudaError_t launch_accumulate(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                              const int32_t* src_row, const float* scale, int64_t n, cudaStream_t st);
// GEAR_ACC_ATOMIC: reductions on the accumulator rows, then one settle pass over the touched images
cudaError_t launch_accumulate_atomic(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                                     const int32_t* src_row, const float* scale, int64_t n, cudaStream_t st);
// steps 2-4 of the sorted accumulate for the batch just sorted by gear_forward_backward, ahead of the accumulate call
cudaError_t launch_accumulate_plan_ahead(const gear_ctx_impl& c, int64_t n, const int32_t* src_row, const float* scale,
                                         cudaStream_t st);
cudaError_t launch_collect_ready(const gear_ctx_impl& c, int32_t* ids, int32_t* seq, float* avg, int64_t cap,
                                 int64_t* d_n, cudaStream_t st);
// accumulate followed by the hand-over; averages bypass the queue when the host knows it to be empty and cap >= n
cudaError_t launch_accumulate_collect(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                                      const int32_t* src_row, const float* scale, int64_t n, int32_t* ids, int32_t* seq,
                                      float* avg, int64_t cap, int64_t* d_n, cudaStream_t st);

// expiry.cu
cudaError_t launch_refresh_dfv(const gear_ctx_impl& c, const int32_t* ids, const float* rows, int64_t ld, int64_t n,
                               const int64_t* d_n, int64_t now, cudaStream_t st);
cudaError_t launch_collect_expired(const gear_ctx_impl& c, int64_t now, int restamp, int32_t* ids, int64_t cap,
                                   int64_t* d_n, cudaStream_t st);

}  // namespace gear
