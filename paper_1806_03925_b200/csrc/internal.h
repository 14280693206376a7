// Host-side internals of libgear: the ctx, the workspace plan and the launch functions each .cu exports.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/gear.h"
#include "common.cuh"

namespace gear {

constexpr int EXP_TILE = 8192;     // entries of the timestamp table per block of the expiry scan
constexpr int MAX_LAYERS = 2;

// Byte offsets into the caller's workspace.  Everything is 256-byte aligned.
struct WsPlan {
    size_t state;                       // DevState
    size_t x;                           // [max_batch][d_in]      head dtype: head input
    size_t h[MAX_LAYERS];               // [max_batch][hidden[l]] head dtype: post-ReLU activations
    size_t da[MAX_LAYERS];              // [max_batch][hidden[l]] head dtype: gradient at the pre-activation
    size_t dz;                          // [max_batch] fp32
    size_t loss_part;                   // [loss_blocks] fp32 per-block partial losses
    size_t wb[MAX_LAYERS];              // bf16 head: W_l as [in][out]
    size_t wbt[MAX_LAYERS];             // bf16 head: W_l as [out][in]
    size_t sort_keys[2], sort_vals[2];  // [sort_cap] uint32
    size_t sort_hist, sort_tot;
    size_t tile_cnt;                    // [sort tiles + 1] uint2 per-tile (groups, complete) counts
    size_t grp_start;                   // [max_nnz] uint32 (top bit: first group of its image in this call)
    size_t grp_slot;                    // [max_nnz] int32 ready-queue slot or -1
    size_t q_id;                        // [ready_cap] int32
    size_t q_avg;                       // [ready_cap][dfv_dim] fp32
    size_t exp_bits;                    // [ceil(img_vocab / 32)] uint32 expired bitmap
    size_t exp_cnt;                     // [expiry tiles + 1] uint2
    size_t total;
    int64_t sort_cap;
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
    bool alive;
    void* tc_state;     // tensor-core head state (tensor maps), owned by head_tc.cu; may be null
    mutable Profiler prof;

    template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(static_cast<char*>(buf.workspace) + off); }
    DevState* state() const { return at<DevState>(ws.state); }
    SortBufs sort_bufs() const {
        SortBufs b;
        b.keys[0] = at<uint32_t>(ws.sort_keys[0]); b.keys[1] = at<uint32_t>(ws.sort_keys[1]);
        b.vals[0] = at<uint32_t>(ws.sort_vals[0]); b.vals[1] = at<uint32_t>(ws.sort_vals[1]);
        b.hist = at<uint32_t>(ws.sort_hist); b.tot = at<uint32_t>(ws.sort_tot);
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

// head_simt.cu: forward + backward of the head with fp32 FMA products (operands fp32 or bf16)
cudaError_t launch_head_simt(const gear_ctx_impl& c, const gear_batch& b, const gear_step_out& o, cudaStream_t st);

// emb_scatter.cu
cudaError_t launch_emb_scatter(const gear_ctx_impl& c, const int32_t* ids, int32_t B, int64_t vocab, float* table,
                               const float* dX, int ldx, int col0, float alpha, cudaStream_t st);

// accumulate.cu
cudaError_t launch_accumulate(const gear_ctx_impl& c, const int32_t* img_id, const float* grads, int64_t ld,
                              const int32_t* src_row, const float* scale, int64_t n, cudaStream_t st);
cudaError_t launch_collect_ready(const gear_ctx_impl& c, int32_t* ids, int32_t* seq, float* avg, int64_t cap,
                                 int64_t* d_n, cudaStream_t st);

// expiry.cu
cudaError_t launch_collect_expired(const gear_ctx_impl& c, int64_t now, int restamp, int32_t* ids, int64_t cap,
                                   int64_t* d_n, cudaStream_t st);

}  // namespace gear
