// The C ABI of libgear (see include/gear.h): argument validation, workspace planning and the
// order in which the kernels of each call are enqueued.  No device memory is allocated here.
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"
#include "internal.h"

namespace gear {

static thread_local char g_last_error[256] = "";

static int cuda_fail(cudaError_t e, const char* where) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %s", where, cudaGetErrorString(e));
    return GEAR_ERR_CUDA;
}
static int arg_fail(const char* what) {
    snprintf(g_last_error, sizeof(g_last_error), "bad argument: %s", what);
    return GEAR_ERR_ARG;
}

static int validate_config(const gear_config& c) {
    const int64_t vmax = 2147483646ll;
    if (c.user_vocab < 1 || c.user_vocab > vmax || c.url_vocab < 1 || c.url_vocab > vmax || c.img_vocab < 1 ||
        c.img_vocab > vmax)
        return arg_fail("vocabulary sizes must be in [1, 2^31 - 2]");
    if (c.emb_dim < 4 || c.emb_dim % 4 || c.emb_dim > 1024) return arg_fail("emb_dim: multiple of 4 in [4, 1024]");
    if (c.dfv_dim < 8 || c.dfv_dim % 8 || c.dfv_dim > 1024) return arg_fail("dfv_dim: multiple of 8 in [8, 1024]");
    if (c.dfv_dtype != GEAR_F32 && c.dfv_dtype != GEAR_BF16) return arg_fail("dfv_dtype");
    if (c.head_dtype != GEAR_F32 && c.head_dtype != GEAR_BF16) return arg_fail("head_dtype");
    if (c.n_hidden < 1 || c.n_hidden > MAX_LAYERS) return arg_fail("n_hidden must be 1 or 2");
    for (int l = 0; l < c.n_hidden; ++l) {
        const int mult = c.head_dtype == GEAR_BF16 ? 64 : 8;
        if (c.hidden[l] < mult || c.hidden[l] % mult || c.hidden[l] > 1024)
            return arg_fail("hidden widths: multiples of 8 (fp32 head) or 64 (bf16 head), at most 1024");
    }
    if (c.M < 1) return arg_fail("M >= 1");
    if (c.expire < 0) return arg_fail("expire >= 0");
    if (c.max_batch < 1 || c.max_batch > (1 << 30) - 1) return arg_fail("max_batch in [1, 2^30 - 1]");
    const int64_t nmax = (1ll << 30) - 1;         // element counts of the key sort fit 30 bits
    if (c.max_nnz < 1 || c.max_nnz > nmax) return arg_fail("max_nnz in [1, 2^30 - 1]");
    if (c.ready_cap < 0 || c.ready_cap > nmax) return arg_fail("ready_cap in [0, 2^30 - 1]");
    if (c.accum_mode != GEAR_ACC_SORT && c.accum_mode != GEAR_ACC_ATOMIC) return arg_fail("accum_mode");
    if (c.accum_mode == GEAR_ACC_ATOMIC && c.M >= (1 << 29)) return arg_fail("GEAR_ACC_ATOMIC needs M < 2^29");
    if (c.fast_dim < 0 || c.fast_dim % 8 || c.fast_dim > 4096) return arg_fail("fast_dim: multiple of 8 in [0, 4096]");
    return GEAR_OK;
}

int plan_workspace(const gear_config& c, WsPlan* p) {
    memset(p, 0, sizeof(*p));
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    const size_t hsz = c.head_dtype == GEAR_BF16 ? 2 : 4;
    const int d_in = 2 * c.emb_dim + c.dfv_dim + c.fast_dim;
    const size_t B = (size_t)c.max_batch;
    p->ready_cap = c.ready_cap > 0 ? c.ready_cap : c.max_nnz;
    p->loss_blocks = (int)ceil_div(c.max_batch, 8);
    if (p->loss_blocks > 2 * sm_count()) p->loss_blocks = 2 * sm_count();   // two resident blocks of the output-unit kernel per SM

    p->state = take(sizeof(DevState));
    p->x = take(B * d_in * hsz);
    int fan = d_in;
    for (int l = 0; l < c.n_hidden; ++l) {
        p->h[l] = take(B * c.hidden[l] * hsz);
        p->da[l] = take(B * c.hidden[l] * hsz);
        p->wb[l] = take((size_t)fan * c.hidden[l] * 2);
        p->wbt[l] = take((size_t)fan * c.hidden[l] * 2);
        fan = c.hidden[l];
    }
    p->dz = take(B * 4);
    p->loss_part = take((size_t)p->loss_blocks * 4);
    p->colsum_part = take((size_t)CS_BLOCKS * 1024 * 4);
    p->sort_n[0] = p->sort_n[1] = c.max_batch;
    p->sort_n[2] = c.max_nnz;
    p->sort_n[3] = p->ready_cap;
    for (int s = 0; s < 4; ++s) {
        for (int i = 0; i < 2; ++i) {
            p->sort_keys[s][i] = take((size_t)p->sort_n[s] * 4);
            p->sort_vals[s][i] = take((size_t)p->sort_n[s] * 4);
        }
        p->sort_hist[s] = take((size_t)RS_MAX_PASSES * RS_BUCKETS * sort_tiles(p->sort_n[s]) * 4);
        p->sort_tot[s] = take((size_t)RS_MAX_PASSES * RS_BUCKETS * 4);
    }
    p->tile_cnt = take((size_t)(ceil_div(c.max_nnz, 1024) + 1) * sizeof(uint2));
    p->grp_rec = take((size_t)c.max_nnz * 16);
    p->pmeta = take((size_t)c.max_nnz * 8);
    p->blk_first = take((size_t)(ceil_div(c.max_nnz, ACC_SPAN) + 2) * 4);
    p->run_end = take((size_t)c.max_nnz * 4);
    p->q_id = take((size_t)p->ready_cap * 4);
    p->q_avg = take((size_t)p->ready_cap * c.dfv_dim * 4);
    p->emb_gsum[0] = take(B * c.emb_dim * 4);
    p->emb_gsum[1] = take(B * c.emb_dim * 4);
    p->exp_bits = take((size_t)ceil_div(c.img_vocab, 32) * 4);
    p->exp_cnt = take((size_t)(ceil_div(c.img_vocab, EXP_MARK_TILE) + 1) * sizeof(uint2));
    p->total = off;
    return GEAR_OK;
}

static int64_t param_count(const gear_config& c) {
    int64_t n = 0, fan = 2 * c.emb_dim + c.dfv_dim + c.fast_dim;
    for (int l = 0; l < c.n_hidden; ++l) { n += fan * c.hidden[l] + c.hidden[l]; fan = c.hidden[l]; }
    return n + fan + 1;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// the ctx's side stream and fork/join events (host-side driver objects, no device memory)
static void release_host_objects(gear_ctx_impl& c) {
    if (c.ev_fork) cudaEventDestroy(c.ev_fork);
    if (c.ev_join) cudaEventDestroy(c.ev_join);
    if (c.ev_gather) cudaEventDestroy(c.ev_gather);
    if (c.ev_dx) cudaEventDestroy(c.ev_dx);
    c.ev_dx = nullptr;
    if (c.side_stream) cudaStreamDestroy(c.side_stream);
    c.ev_fork = c.ev_join = c.ev_gather = nullptr;
    c.side_stream = nullptr;
}

}  // namespace gear

using namespace gear;

struct gear_ctx { gear_ctx_impl impl; };

extern "C" {

const char* gear_last_error(void) { return g_last_error; }

int gear_workspace_bytes(const gear_config* cfg, size_t* out_bytes) {
    if (!cfg || !out_bytes) return arg_fail("NULL pointer");
    int rc = validate_config(*cfg);
    if (rc != GEAR_OK) return rc;
    WsPlan p;
    plan_workspace(*cfg, &p);
    *out_bytes = p.total;
    return GEAR_OK;
}

int gear_fill_uniform(void* dst, int32_t dtype, int64_t n_rows, int32_t dim, uint64_t seed, uint64_t tag, double amp,
                      void* stream) {
    if (!dst || n_rows < 0 || dim < 1 || !aligned16(dst)) return arg_fail("gear_fill_uniform");
    if (dtype != GEAR_F32 && dtype != GEAR_BF16) return arg_fail("dtype");
    cudaError_t e = launch_fill_uniform(dst, dtype, n_rows * dim, seed, tag, amp, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GEAR_OK : cuda_fail(e, "gear_fill_uniform");
}

int gear_init_tables(gear_ctx** out_ctx, const gear_config* cfg, const gear_buffers* buf, uint64_t seed, int fill,
                     int64_t now, void* stream) {
    if (!out_ctx || !cfg || !buf) return arg_fail("NULL pointer");
    *out_ctx = nullptr;
    int rc = validate_config(*cfg);
    if (rc != GEAR_OK) return rc;
    if (!buf->user_emb || !buf->url_emb || !buf->dfv || !buf->dfv_gsum || !buf->dfv_gcnt || !buf->dfv_ts ||
        !buf->head_params || !buf->workspace)
        return arg_fail("NULL buffer");
    if (!aligned16(buf->user_emb) || !aligned16(buf->url_emb) || !aligned16(buf->dfv) || !aligned16(buf->dfv_gsum) ||
        (reinterpret_cast<uintptr_t>(buf->workspace) & 255u))
        return arg_fail("tables must be 16-byte aligned, the workspace 256-byte aligned");
    gear_ctx* ctx = new (std::nothrow) gear_ctx;
    if (!ctx) return arg_fail("out of host memory");
    gear_ctx_impl& c = ctx->impl;
    c.cfg = *cfg;
    c.buf = *buf;
    plan_workspace(*cfg, &c.ws);
    if (buf->workspace_bytes < c.ws.total) { delete ctx; return arg_fail("workspace too small"); }
    c.d_in = 2 * cfg->emb_dim + cfg->dfv_dim + cfg->fast_dim;
    c.n_params = param_count(*cfg);
    c.alive = true;
    c.tc_state = nullptr;
    c.gbs.device_counter = &c.state()->grid_barrier;
    c.gbs.host_base = 0;
    c.img_sorted = false;
    c.img_sort_valid = false;
    c.img_sorted_n = 0;
    c.img_sorted_buf = 0;
    c.last_img_id = nullptr;
    c.acc_calls_pending = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.last_stream = st;
    c.side_stream = nullptr;
    c.ev_fork = c.ev_join = c.ev_gather = c.ev_dx = nullptr;
    c.plan_ready = false; c.plan_n = 0; c.plan_src_row = nullptr; c.plan_scale = nullptr;

    cudaError_t e = cudaStreamCreateWithFlags(&c.side_stream, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c.ev_gather, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c.ev_fork, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c.ev_join, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c.ev_dx, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaMemsetAsync(c.state(), 0, sizeof(DevState), st);
    if (e == cudaSuccess && fill) {
        const double amp = 0.17320508075688773;   // uniform half-width for standard deviation 0.1
        e = launch_fill_uniform(buf->user_emb, GEAR_F32, cfg->user_vocab * cfg->emb_dim, seed, GEAR_TAG_USER, amp, st);
        if (e == cudaSuccess)
            e = launch_fill_uniform(buf->url_emb, GEAR_F32, cfg->url_vocab * cfg->emb_dim, seed, GEAR_TAG_URL, amp, st);
        if (e == cudaSuccess)
            e = launch_fill_uniform(buf->dfv, cfg->dfv_dtype, cfg->img_vocab * cfg->dfv_dim, seed, GEAR_TAG_DFV, amp, st);
        if (e == cudaSuccess)
            e = cudaMemsetAsync(buf->dfv_gsum, 0, sizeof(float) * (size_t)cfg->img_vocab * cfg->dfv_dim, st);
        if (e == cudaSuccess) e = cudaMemsetAsync(buf->dfv_gcnt, 0, sizeof(int32_t) * (size_t)cfg->img_vocab, st);
        if (e == cudaSuccess) e = launch_fill_ts(buf->dfv_ts, cfg->img_vocab, seed, cfg->expire, now, st);
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { release_host_objects(c); delete ctx; return cuda_fail(e, "gear_init_tables"); }
    *out_ctx = ctx;
    return GEAR_OK;
}

int gear_forward_backward(gear_ctx* ctx, const gear_batch* batch, float lr, const gear_step_out* out, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    if (!batch || !out) return arg_fail("NULL pointer");
    gear_ctx_impl& c = ctx->impl;
    const gear_batch& b = *batch;
    const gear_step_out& o = *out;
    if (b.B < 0 || b.B > c.cfg.max_batch) return arg_fail("B outside [0, max_batch]");
    if (b.nnz < 0 || b.nnz > c.cfg.max_nnz) return arg_fail("nnz outside [0, max_nnz]");
    if (b.B > 0 && (!b.user_id || !b.url_id || !b.img_off || !b.label)) return arg_fail("NULL batch array");
    if (b.nnz > 0 && !b.img_id) return arg_fail("NULL img_id");
    if (b.B > 0 && c.cfg.fast_dim > 0 && (!b.fast || !aligned16(b.fast))) return arg_fail("fast: needed (16-byte aligned) when fast_dim > 0");
    if (!o.loss || !o.head_grad || !o.dX) return arg_fail("loss, head_grad and dX are required outputs");
    if ((o.user_grad == nullptr) != (o.url_grad == nullptr)) return arg_fail("user_grad and url_grad: both or neither");
    gear_adam adam_cfg = {0.f, 0.f, 0.f, 0.f};
    if (o.adam) {
        adam_cfg = *o.adam;
        if (o.user_grad) return arg_fail("adam and user_grad / url_grad exclude each other");
        if (!o.user_m || !o.user_v || !o.url_m || !o.url_v) return arg_fail("adam needs the four moment tables");
        if (!aligned16(o.user_m) || !aligned16(o.user_v) || !aligned16(o.url_m) || !aligned16(o.url_v))
            return arg_fail("moment tables must be 16-byte aligned");
        if (o.adam_step < 1) return arg_fail("adam_step >= 1");
        if (!(adam_cfg.beta1 >= 0.f && adam_cfg.beta1 < 1.f && adam_cfg.beta2 >= 0.f && adam_cfg.beta2 < 1.f && adam_cfg.eps >= 0.f))
            return arg_fail("adam: beta1, beta2 in [0, 1), eps >= 0");
    }
    if (c.cfg.head_dtype == GEAR_BF16 && (!aligned16(o.head_grad) || !aligned16(c.buf.head_params)))
        return arg_fail("bf16 head: head_params and head_grad must be 16-byte aligned");
    if (o.dfv_grad && (!o.row_view || !o.inv_n || !aligned16(o.dfv_grad)))
        return arg_fail("dfv_grad needs row_view and inv_n and 16-byte alignment");
    if (!aligned16(o.dX) || (o.x_debug && !aligned16(o.x_debug)) || (o.user_grad && !aligned16(o.user_grad)) ||
        (o.url_grad && !aligned16(o.url_grad)))
        return arg_fail("dX, x_debug, user_grad, url_grad must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.last_stream = st;

    // What depends on the batch's ID arrays and on head_params alone runs on the ctx's side stream, beside the gather
    // and the head: the bf16 copies of the weights, the key sort of the three ID arrays (the user and URL orders drive
    // the embedding scatter, the image order is kept for gear_accumulate_dfv_grad with img_id == NULL) and, once the
    // gather has written row_view / inv_n, the plan of that accumulate call.  The embedding scatter itself joins them
    // there as soon as dX exists, beside the last weight-gradient product; the caller's stream waits for the side
    // stream before the call returns.  With per-kernel timing on, everything stays on the caller's stream so that each
    // kernel is timed alone.
    c.img_sorted = false;
    c.img_sort_valid = false;
    c.plan_ready = false;
    const bool forked = (!c.prof.on || c.prof.keep_streams) && b.B > 0;
    bool join_pending = false;          // the side stream holds work the caller's stream has not waited for
    cudaStream_t side = forked ? c.side_stream : st;
    // A failure between the fork and the join must not leave the side stream unjoined or the sorted order marked as
    // usable: the caller's stream waits for whatever the side stream was given, and the ctx forgets the batch.
    auto abandon = [&](cudaError_t err, const char* where) {
        if (join_pending) {
            if (cudaEventRecord(c.ev_join, c.side_stream) != cudaSuccess || cudaStreamWaitEvent(st, c.ev_join, 0) != cudaSuccess)
                cudaStreamSynchronize(c.side_stream);
        }
        c.img_sorted = false; c.img_sort_valid = false; c.plan_ready = false;
        return cuda_fail(err, where);
    };
    cudaError_t e = cudaSuccess;
    if (forked) {
        e = cudaEventRecord(c.ev_fork, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(c.side_stream, c.ev_fork, 0);
        if (e != cudaSuccess) return cuda_fail(e, "fork");
        join_pending = true;
    }
    // bf16 copies of the head's weights: first on the caller's stream, ahead of the gather.  The gather keeps every SM
    // busy for its whole duration, so a small kernel on another stream would get its blocks placed only when the gather
    // ends, and the first product of the head would wait for it.
    const bool weights_early = b.B > 0 && c.cfg.head_dtype == GEAR_BF16;
    if (weights_early) {
        e = launch_round_weights(c, st);
        if (e != cudaSuccess) return abandon(e, "weight copies");
    }
    int sorted_buf = 0;
    if (b.B > 0) {
        SortBatch batch = c.sort_batch();
        batch.job[0] = c.sort_job(gear_ctx_impl::SORT_USER);
        batch.job[0].ids = b.user_id; batch.job[0].sentinel = (uint32_t)c.cfg.user_vocab;
        batch.job[0].n_max = b.B; batch.job[0].bits = bits_for(c.cfg.user_vocab);
        batch.job[1] = c.sort_job(gear_ctx_impl::SORT_URL);
        batch.job[1].ids = b.url_id; batch.job[1].sentinel = (uint32_t)c.cfg.url_vocab;
        batch.job[1].n_max = b.B; batch.job[1].bits = bits_for(c.cfg.url_vocab);
        batch.n_jobs = 2;
        if (b.nnz > 0 && c.cfg.accum_mode == GEAR_ACC_SORT) {      // the atomic mode takes the image IDs as they come
            batch.job[2] = c.sort_job(gear_ctx_impl::SORT_IMG);
            batch.job[2].ids = b.img_id; batch.job[2].sentinel = (uint32_t)c.cfg.img_vocab;
            batch.job[2].n_max = b.nnz; batch.job[2].bits = bits_for(c.cfg.img_vocab);
            batch.n_jobs = 3;
        }
        cudaError_t se = cudaSuccess;
        batch.name = "sort_ids";
        sorted_buf = sort_jobs(batch, &c.gbs, side, &c.prof, &se);
        if (se != cudaSuccess) return abandon(se, "id sort");
        if (b.nnz > 0) {
            c.img_sorted = true; c.img_sorted_n = b.nnz; c.img_sorted_buf = sorted_buf; c.last_img_id = b.img_id;
            c.img_sort_valid = c.cfg.accum_mode == GEAR_ACC_SORT;
        }
    }
    e = launch_gather(c, b, o.row_view, o.inv_n, o.x_debug, st);
    if (e != cudaSuccess) return abandon(e, "gather");
    if (forked && b.nnz > 0 && o.row_view && o.inv_n && c.cfg.accum_mode == GEAR_ACC_SORT) {
        // behind the sort: the plan of the accumulate call that usually follows (which rows form which group, where every
        // group's rows and queue slot are).  It needs the gather's row_view / inv_n.
        e = cudaEventRecord(c.ev_gather, st);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(c.side_stream, c.ev_gather, 0);
        if (e == cudaSuccess) e = launch_accumulate_plan_ahead(c, b.nnz, o.row_view, o.inv_n, c.side_stream);
        if (e != cudaSuccess) return abandon(e, "accumulate plan");
    }
    // the embedding scatter: enqueued by the head as soon as dX is on its way
    struct Scatter {
        gear_ctx_impl* c; const gear_step_out* o; int sorted_buf; int32_t B; float lr; cudaStream_t st; bool forked;
        const gear_adam* adam;
    } sc{&c, &o, sorted_buf, b.B, lr, st, forked, o.adam ? &adam_cfg : nullptr};
    auto scatter = [](void* arg) -> cudaError_t {
        Scatter& k = *static_cast<Scatter*>(arg);
        gear_ctx_impl& c = *k.c;
        float* ut = k.o->user_grad ? k.o->user_grad : c.buf.user_emb;
        float* ht = k.o->url_grad ? k.o->url_grad : c.buf.url_emb;
        const float alpha = k.o->user_grad ? 1.0f : -k.lr;
        cudaStream_t where = k.st;
        if (k.forked) {
            cudaError_t e = cudaEventRecord(c.ev_dx, k.st);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(c.side_stream, c.ev_dx, 0);
            if (e != cudaSuccess) return e;
            where = c.side_stream;
        }
        if (k.adam)
            return launch_emb_adam(c, k.sorted_buf, k.B, k.o->dX, c.d_in, *k.adam, k.o->adam_step, k.o->user_m, k.o->user_v,
                                   k.o->url_m, k.o->url_v, where);
        return launch_emb_reduce(c, k.sorted_buf, k.B, ut, ht, k.o->dX, c.d_in, alpha, where);
    };
    const HeadHooks hooks{weights_early, scatter, &sc};
    e = launch_head_simt(c, b, o, st, hooks);
    if (e != cudaSuccess) return abandon(e, "head");
    if (o.dfv_grad && b.B > 0) {
        e = launch_dfv_grad_rows(c, o.dX, o.row_view, o.inv_n, b.nnz, o.dfv_grad, st);
        if (e != cudaSuccess) return abandon(e, "gradient rows");
    }
    if (forked) {
        e = cudaEventRecord(c.ev_join, c.side_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(st, c.ev_join, 0);
        if (e != cudaSuccess) return abandon(e, "join");
        join_pending = false;
    }
    return GEAR_OK;
}

int gear_accumulate_dfv_grad(gear_ctx* ctx, const int32_t* img_id, const float* grads, int64_t ld,
                             const int32_t* src_row, const float* scale, int64_t n, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (n < 0 || n > c.cfg.max_nnz) return arg_fail("n outside [0, max_nnz]");
    if (n == 0) return GEAR_OK;
    if (!grads) return arg_fail("NULL pointer");
    if (!img_id && (!c.img_sorted || c.img_sorted_n != n)) {
        snprintf(g_last_error, sizeof(g_last_error),
                 "img_id == NULL needs a preceding gear_forward_backward whose nnz equals n");
        return GEAR_ERR_STATE;
    }
    if (ld < c.cfg.dfv_dim || ld % 4 || !aligned16(grads)) return arg_fail("grads rows must be 16-byte aligned, ld >= dfv_dim");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.last_stream = st;
    cudaError_t e = c.cfg.accum_mode == GEAR_ACC_ATOMIC
                        ? launch_accumulate_atomic(c, img_id ? img_id : c.last_img_id, grads, ld, src_row, scale, n, st)
                        : launch_accumulate(c, img_id, grads, ld, src_row, scale, n, st);
    return e == cudaSuccess ? GEAR_OK : cuda_fail(e, "accumulate");
}

static int finish_count(gear_ctx_impl& c, const int64_t* d_src, int64_t cap, int64_t* h_n, cudaStream_t st);

int gear_accumulate_collect(gear_ctx* ctx, const int32_t* img_id, const float* grads, int64_t ld, const int32_t* src_row,
                            const float* scale, int64_t n, int32_t* ids, int32_t* seq, float* avg, int64_t cap,
                            int64_t* d_n, int64_t* h_n, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (n < 0 || n > c.cfg.max_nnz) return arg_fail("n outside [0, max_nnz]");
    if (n > 0 && !grads) return arg_fail("NULL pointer");
    if (n > 0 && !img_id && (!c.img_sorted || c.img_sorted_n != n)) {
        snprintf(g_last_error, sizeof(g_last_error),
                 "img_id == NULL needs a preceding gear_forward_backward whose nnz equals n");
        return GEAR_ERR_STATE;
    }
    if (n > 0 && (ld < c.cfg.dfv_dim || ld % 4 || !aligned16(grads)))
        return arg_fail("grads rows must be 16-byte aligned, ld >= dfv_dim");
    if (cap < 0 || (cap > 0 && (!ids || !seq || !avg))) return arg_fail("NULL output with cap > 0");
    if (avg && !aligned16(avg)) return arg_fail("avg must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.last_stream = st;
    int64_t* d_cnt = d_n ? d_n : &c.state()->pad[0];
    cudaError_t e = launch_accumulate_collect(c, img_id, grads, ld, src_row, scale, n, ids, seq, avg, cap, d_cnt, st);
    if (e != cudaSuccess) return cuda_fail(e, "accumulate_collect");
    return finish_count(c, d_cnt, cap, h_n, st);
}

// Waits for everything the ctx has enqueued: the stream of the training calls and, if the expiry scan went to a
// stream of its own, that one too.
static cudaError_t sync_streams(const gear_ctx_impl& c) {
    cudaError_t e = cudaStreamSynchronize(c.last_stream);
    for (int i = 0; i < c.n_seen && e == cudaSuccess; ++i)
        if (c.seen_stream[i] != c.last_stream) e = cudaStreamSynchronize(c.seen_stream[i]);
    return e;
}

static int finish_count(gear_ctx_impl& c, const int64_t* d_src, int64_t cap, int64_t* h_n, cudaStream_t st) {
    if (!h_n) return GEAR_OK;
    cudaError_t e = cudaMemcpyAsync(h_n, d_src, sizeof(int64_t), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return cuda_fail(e, "read count");
    if (*h_n > cap) {
        snprintf(g_last_error, sizeof(g_last_error), "capacity %lld too small, %lld entries waiting", (long long)cap,
                 (long long)*h_n);
        return GEAR_ERR_CAPACITY;
    }
    return GEAR_OK;
}

int gear_collect_ready(gear_ctx* ctx, int32_t* ids, int32_t* seq, float* avg, int64_t cap, int64_t* d_n, int64_t* h_n,
                       void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (cap < 0 || (cap > 0 && (!ids || !seq || !avg))) return arg_fail("NULL output with cap > 0");
    if (avg && !aligned16(avg)) return arg_fail("avg must be 16-byte aligned");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.last_stream = st;
    // the count is staged in the device state so that h_n can be served even when d_n is NULL
    int64_t* d_cnt = d_n ? d_n : &c.state()->pad[0];
    cudaError_t e = launch_collect_ready(c, ids, seq, avg, cap, d_cnt, st);
    if (e != cudaSuccess) return cuda_fail(e, "collect_ready");
    return finish_count(c, d_cnt, cap, h_n, st);
}

int gear_collect_expired(gear_ctx* ctx, int64_t now, int restamp, int32_t* ids, int64_t cap, int64_t* d_n,
                         int64_t* h_n, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (cap < 0 || (cap > 0 && !ids)) return arg_fail("NULL output with cap > 0");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.note_stream(st);             // may differ from the stream of the training calls: the scan shares nothing with them
    int64_t* d_cnt = d_n ? d_n : &c.state()->pad[1];
    cudaError_t e = launch_collect_expired(c, now, restamp, ids, cap, d_cnt, st);
    if (e != cudaSuccess) return cuda_fail(e, "collect_expired");
    return finish_count(c, d_cnt, cap, h_n, st);
}

int gear_refresh_dfv(gear_ctx* ctx, const int32_t* ids, const float* rows, int64_t ld, int64_t n, const int64_t* d_n,
                     int64_t now, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (n < 0) return arg_fail("n < 0");
    if (n == 0) return GEAR_OK;
    if (!ids || !rows) return arg_fail("NULL pointer");
    if (ld < c.cfg.dfv_dim || (ld & 3) || !aligned16(rows)) return arg_fail("rows must be 16-byte aligned, ld >= dfv_dim and a multiple of 4");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.note_stream(st);
    cudaError_t e = launch_refresh_dfv(c, ids, rows, ld, n, d_n, now, st);
    if (e != cudaSuccess) return cuda_fail(e, "refresh_dfv");
    return GEAR_OK;
}

int gear_fetch_rows(gear_ctx* ctx, int32_t which, const int32_t* ids, int64_t n, void* out, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (which != GEAR_TABLE_USER && which != GEAR_TABLE_URL && which != GEAR_TABLE_DFV) return arg_fail("which");
    if (n < 0) return arg_fail("n < 0");
    if (n == 0) return GEAR_OK;
    if (!ids || !out || !aligned16(out)) return arg_fail("NULL or misaligned pointer");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.note_stream(st);
    cudaError_t e = launch_fetch_rows(c, which, ids, n, out, st);
    return e == cudaSuccess ? GEAR_OK : cuda_fail(e, "fetch_rows");
}

int gear_apply_emb_grad(gear_ctx* ctx, int32_t which, const int32_t* ids, const float* rows, int64_t ld, int64_t n, float lr,
                        void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (which != GEAR_TABLE_USER && which != GEAR_TABLE_URL) return arg_fail("which: GEAR_TABLE_USER or GEAR_TABLE_URL");
    if (n < 0 || n > c.cfg.max_batch) return arg_fail("n outside [0, max_batch]");
    if (n == 0) return GEAR_OK;
    if (!ids || !rows || !aligned16(rows) || ld < c.cfg.emb_dim || (ld & 3)) return arg_fail("rows: 16-byte aligned, ld >= emb_dim, multiple of 4");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.last_stream = st;
    cudaError_t e = launch_apply_emb_grad(c, which, ids, rows, ld, n, -lr, st);
    return e == cudaSuccess ? GEAR_OK : cuda_fail(e, "apply_emb_grad");
}

int gear_dense_forward(gear_ctx* ctx, const float* raw, int32_t raw_dim, const float* Wd, const int32_t* ids, int64_t n,
                       const int64_t* d_n, float* rows, int64_t ld, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (n < 0 || raw_dim < 1) return arg_fail("n >= 0, raw_dim >= 1");
    if (n == 0) return GEAR_OK;
    if (!raw || !Wd || !ids || !rows || ld < c.cfg.dfv_dim) return arg_fail("NULL pointer or ld < dfv_dim");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.note_stream(st);
    cudaError_t e = launch_dense_forward(c, raw, raw_dim, Wd, ids, n, d_n, rows, ld, st);
    return e == cudaSuccess ? GEAR_OK : cuda_fail(e, "dense_forward");
}

int gear_dense_backward(gear_ctx* ctx, const float* raw, int32_t raw_dim, const int32_t* ids, const float* avg, int64_t n,
                        const int64_t* d_n, float* Wd_grad, void* stream) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    if (n < 0 || raw_dim < 1) return arg_fail("n >= 0, raw_dim >= 1");
    if (n == 0) return GEAR_OK;
    if (!raw || !ids || !avg || !Wd_grad) return arg_fail("NULL pointer");
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    c.note_stream(st);
    cudaError_t e = launch_dense_backward(c, raw, raw_dim, ids, avg, c.cfg.dfv_dim, n, d_n, Wd_grad, st);
    return e == cudaSuccess ? GEAR_OK : cuda_fail(e, "dense_backward");
}

int gear_adam_dense(float* param, const float* grad, float* m, float* v, int64_t n, int64_t t, const gear_adam* cfg,
                    void* stream) {
    if (n < 0 || t < 1 || !cfg) return arg_fail("n >= 0, t >= 1, cfg");
    if (n == 0) return GEAR_OK;
    if (!param || !grad || !m || !v) return arg_fail("NULL pointer");
    if (!(cfg->beta1 >= 0.f && cfg->beta1 < 1.f && cfg->beta2 >= 0.f && cfg->beta2 < 1.f && cfg->eps >= 0.f))
        return arg_fail("adam: beta1, beta2 in [0, 1), eps >= 0");
    cudaError_t e = launch_adam_dense(nullptr, param, grad, m, v, n, t, *cfg, static_cast<cudaStream_t>(stream));
    return e == cudaSuccess ? GEAR_OK : cuda_fail(e, "adam_dense");
}

int gear_status(gear_ctx* ctx, int32_t* device_status, int64_t* pending_ready) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    gear_ctx_impl& c = ctx->impl;
    DevState h;
    memset(&h, 0, sizeof(h));
    cudaError_t e = sync_streams(c);
    if (e == cudaSuccess) e = cudaMemcpy(&h, c.state(), sizeof(DevState), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "gear_status");      // h holds nothing to look at
    if (h.tc_error != 0) h.status |= GEAR_DEV_TIMEOUT;
    if (e == cudaSuccess && h.status != 0) e = cudaMemset(c.state(), 0, 2 * sizeof(int32_t));   // status, tc_error
    if (e == cudaSuccess && h.tc_error != 0) {
        // an abandoned grid barrier leaves its arrival counter short: start the count again
        e = cudaMemset(&c.state()->grid_barrier, 0, sizeof(unsigned long long));
        c.gbs.host_base = 0;
    }
    if (e != cudaSuccess) return cuda_fail(e, "gear_status");
    if (device_status) *device_status = h.status;
    if (pending_ready) *pending_ready = h.q_count;
    if (h.status & GEAR_DEV_TIMEOUT) {
        snprintf(g_last_error, sizeof(g_last_error), "a bounded device wait gave up (code %d)", h.tc_error);
        return GEAR_ERR_CUDA;
    }
    if (h.status & GEAR_DEV_BAD_ID) return GEAR_ERR_BAD_ID;
    if (h.status & (GEAR_DEV_READY_OVERFLOW | GEAR_DEV_OUT_CAPACITY)) return GEAR_ERR_CAPACITY;
    if (h.status & GEAR_DEV_BAD_CSR) return GEAR_ERR_ARG;
    return GEAR_OK;
}

int gear_profile_enable(gear_ctx* ctx, int on) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    sync_streams(ctx->impl);
    ctx->impl.prof.clear();
    ctx->impl.prof.on = on != 0;
    ctx->impl.prof.keep_streams = on == 2;
    return GEAR_OK;
}

int gear_profile_timeline(gear_ctx* ctx, char* names, float* start_ms, float* stop_ms, int32_t cap, int32_t* n_out) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    if (!n_out || cap < 0 || (cap > 0 && (!names || !start_ms || !stop_ms))) return arg_fail("gear_profile_timeline");
    gear_ctx_impl& c = ctx->impl;
    cudaError_t e = sync_streams(c);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c.side_stream);
    if (e != cudaSuccess) return cuda_fail(e, "gear_profile_timeline");
    int n = 0;
    for (const auto& r : c.prof.recs) {
        if (n >= cap) break;
        float a = 0.f, b = 0.f;
        e = cudaEventElapsedTime(&a, c.prof.recs[0].start, r.start);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&b, c.prof.recs[0].start, r.stop);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventElapsedTime");
        strncpy(names + 64 * n, r.name, 63);
        names[64 * n + 63] = 0;
        start_ms[n] = a; stop_ms[n] = b;
        ++n;
    }
    *n_out = n;
    c.prof.clear();
    return GEAR_OK;
}

int gear_profile_read(gear_ctx* ctx, char* names, float* total_ms, int32_t* launches, int32_t cap, int32_t* n_out) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    if (!n_out || cap < 0 || (cap > 0 && (!names || !total_ms || !launches))) return arg_fail("gear_profile_read");
    gear_ctx_impl& c = ctx->impl;
    cudaError_t e = sync_streams(c);
    if (e != cudaSuccess) return cuda_fail(e, "gear_profile_read");
    int n = 0;
    for (const auto& r : c.prof.recs) {
        float ms = 0.f;
        e = cudaEventElapsedTime(&ms, r.start, r.stop);
        if (e != cudaSuccess) return cuda_fail(e, "cudaEventElapsedTime");
        int k = 0;
        while (k < n && strncmp(names + 64 * k, r.name, 63) != 0) ++k;
        if (k == n) {
            if (n >= cap) continue;
            strncpy(names + 64 * k, r.name, 63);
            names[64 * k + 63] = 0;
            total_ms[k] = 0.f;
            launches[k] = 0;
            ++n;
        }
        total_ms[k] += ms;
        launches[k] += 1;
    }
    *n_out = n;
    c.prof.clear();
    return GEAR_OK;
}

int gear_launch_count(gear_ctx* ctx, int64_t* n_launches) {
    if (!ctx || !ctx->impl.alive) return GEAR_ERR_STATE;
    if (!n_launches) return arg_fail("NULL pointer");
    *n_launches = ctx->impl.prof.launches;
    return GEAR_OK;
}

int gear_destroy(gear_ctx* ctx) {
    if (!ctx) return GEAR_OK;
    if (!ctx->impl.alive) return GEAR_ERR_STATE;     // a ctx that failed half-way through its set-up; a destroyed
                                                     // ctx is freed memory and must not be passed in again
    sync_streams(ctx->impl);
    cudaStreamSynchronize(ctx->impl.side_stream);
    release_host_objects(ctx->impl);
    ctx->impl.alive = false;
    delete ctx;
    return GEAR_OK;
}

}  // extern "C"
