/*
 * gear.h -- C ABI of libgear: the sparse-part training step of Gear Training
 * (arXiv 1806.03925) on one NVIDIA B200 (sm_100a), with the Dense Part replaced
 * by a table of cached Dense Feature Vectors (DFVs).
 *
 * The calls follow the paper's Section 3 event list (events 1-6) and the two
 * cache rules of Section 1 ("inference expired time", "accumulated to M"):
 *
 *   gear_init_tables          cluster start-up: the DFV cache, the gradient
 *                             store and the embedding tables exist and are warm.
 *   gear_forward_backward     events 1, 3, 4: fetch DFVs by Image ID, Sparse
 *                             Part forward to the loss, backward through the
 *                             Sparse Part only, stopping at dLoss/dDFV (Eq. 1,
 *                             left factor); apply the embedding gradients.
 *   gear_accumulate_dfv_grad  event 5 and the first half of event 6: (Image
 *                             ID, gradient) pairs arrive and are summed per
 *                             image; every M-th arrival completes a group.
 *   gear_collect_ready        event 6: hand over the averaged gradient of
 *                             every completed group.
 *   gear_accumulate_collect   events 5 and 6 as one call.
 *   gear_refresh_dfv          Section 1 / Section 3: recomputed DFVs replace
 *                             expired ones and restart their clocks.
 *   gear_dense_forward /      events 2-3 and the second half of event 6 for a
 *   gear_dense_backward       linear Dense Part; gear_adam_dense and the adam
 *                             fields of gear_step_out: Section 4's optimiser.
 *   gear_collect_expired      Section 1 / Section 3: cached inference results
 *                             older than the inference-expired time.
 *
 * General rules
 *   - Every function returns GEAR_OK (0) or a negative GEAR_ERR_* code.  None
 *     throws, exits or traps the device.
 *   - All device work is enqueued on the caller's stream (`stream` is a
 *     cudaStream_t passed as void*; NULL is the default stream).  A call
 *     blocks the host only when a host out-pointer (h_n) is non-NULL, in
 *     gear_status, and in gear_init_tables / gear_destroy.
 *   - Ownership: every table, every input and output array and the workspace
 *     are DEVICE memory allocated and owned by the caller.  The library
 *     allocates no device memory.  The gear_ctx is host memory owned by the
 *     library and released by gear_destroy.  Structs passed by pointer are
 *     HOST memory and are copied during the call.
 *   - Layout: all matrices are row-major and dense unless a leading dimension
 *     is given.  IDs are int32; an ID outside [0, vocab) is ignored (its row
 *     counts as zeros / its gradient is dropped) and raises the sticky
 *     GEAR_DEV_BAD_ID bit of the device status word.
 *   - Calls on one ctx must be issued from one host thread at a time and on
 *     one stream (or on streams the caller orders with events).
 */
#ifndef GEAR_H
#define GEAR_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    GEAR_OK = 0,
    GEAR_ERR_ARG = -1,       /* NULL pointer, bad dimension, misaligned buffer, batch larger than configured */
    GEAR_ERR_CAPACITY = -2,  /* an output list or the ready queue is too small; nothing was consumed */
    GEAR_ERR_BAD_ID = -3,    /* an out-of-range ID was met (reported by gear_status; the row was skipped) */
    GEAR_ERR_CUDA = -4,      /* a CUDA runtime or driver call failed */
    GEAR_ERR_STATE = -5      /* call order violated (e.g. img_id == NULL without a preceding gear_forward_backward) */
};

/* element types of tables and of the head's matrix-product operands */
enum { GEAR_F32 = 0, GEAR_BF16 = 1 };

/* how gear_accumulate_dfv_grad combines rows that share an Image ID */
enum {
    GEAR_ACC_SORT = 0,       /* stable key sort + segmented reduction: groups split exactly at every
                                M-th arrival in row order; deterministic */
    GEAR_ACC_ATOMIC = 1      /* fp32 reductions on the accumulator rows in whatever order the hardware takes
                                them: which arrivals share a group is not defined.  Counts and the number of
                                emissions per image equal the sorted path's; after the rows of a call have been
                                added, an image holding k >= M gradients emits floor(k / M) averages, each the mean
                                of all k pooled gradients, and keeps (k mod M) / k of the pooled sum, so that
                                M * (emitted averages) + kept sum = pooled sum.  A call is refused whole
                                (GEAR_DEV_READY_OVERFLOW) unless the queue has room for n more entries.
                                Needs M < 2^29.  Not bit-reproducible from run to run */
};

/* bits of the device status word (sticky until gear_status clears them) */
enum {
    GEAR_DEV_BAD_ID = 1,         /* an ID outside [0, vocab) was skipped */
    GEAR_DEV_READY_OVERFLOW = 2, /* an accumulate call would have overflowed the ready queue and was dropped whole */
    GEAR_DEV_OUT_CAPACITY = 4,   /* a collect call found cap too small and left everything in place */
    GEAR_DEV_BAD_CSR = 8,        /* img_off not non-decreasing / not ending at nnz */
    GEAR_DEV_TIMEOUT = 16        /* a bounded wait inside a kernel gave up; the step's results are invalid */
};

/* the three tables a request for rows can name (gear_fetch_rows, gear_apply_emb_grad) */
enum { GEAR_TABLE_USER = 0, GEAR_TABLE_URL = 1, GEAR_TABLE_DFV = 2 };

/* tags of the procedural table fill (SplitMix64 streams, see gear_fill_uniform) */
enum { GEAR_TAG_USER = 1, GEAR_TAG_URL = 2, GEAR_TAG_DFV = 3, GEAR_TAG_TS = 4, GEAR_TAG_GRAD = 5 };

typedef struct gear_ctx gear_ctx;

/* Static description of one model + store.  Validated by gear_init_tables. */
typedef struct {
    int64_t user_vocab, url_vocab, img_vocab; /* each in [1, 2^31 - 2] */
    int32_t emb_dim;       /* columns of the user and URL-hash tables (fp32); multiple of 4, <= 1024 */
    int32_t dfv_dim;       /* columns of the DFV table; multiple of 8, <= 1024 */
    int32_t dfv_dtype;     /* GEAR_F32 | GEAR_BF16: storage type of the DFV table */
    int32_t head_dtype;    /* GEAR_F32: fp32 FMA head.  GEAR_BF16: operands of the head's matrix products
                              (head input, weights, hidden activations, activation gradients) are rounded
                              to bfloat16 (nearest-even); products accumulate in fp32 */
    int32_t n_hidden;      /* 1 or 2 hidden ReLU layers; the output layer is one logistic unit */
    int32_t hidden[2];     /* widths; multiples of 8 (GEAR_F32) or 64 (GEAR_BF16), <= 1024 */
    int32_t M;             /* gradients per image per emitted average, >= 1 */
    int64_t expire;        /* inference-expired time, >= 0, in the caller's time unit */
    int32_t max_batch;     /* largest B of any gear_forward_backward call, < 2^30 */
    int64_t max_nnz;       /* largest number of rows of any forward_backward / accumulate call, < 2^30 */
    int64_t ready_cap;     /* rows of the ready queue (averages waiting for gear_collect_ready);
                              0 = max_nnz, which can never overflow if every accumulate call is
                              followed by a collect */
    int32_t accum_mode;    /* GEAR_ACC_SORT | GEAR_ACC_ATOMIC */
    int32_t fast_dim;      /* columns of dense input the Fastgear side brings along per view (Section 4: the part of the
                              image that is fed to the Fastgear Worker directly), appended to the head input after the
                              pooled DFV; 0 = none; multiple of 8, <= 4096 */
} gear_config;

/* Caller-owned device buffers that persist across calls. */
typedef struct {
    float*    user_emb;     /* [user_vocab][emb_dim] fp32 */
    float*    url_emb;      /* [url_vocab][emb_dim]  fp32 */
    void*     dfv;          /* [img_vocab][dfv_dim]  dfv_dtype; rows 16-byte aligned */
    float*    dfv_gsum;     /* [img_vocab][dfv_dim]  fp32 running sum of the open group of each image */
    int32_t*  dfv_gcnt;     /* [img_vocab]           arrivals in the open group, always in [0, M) */
    int64_t*  dfv_ts;       /* [img_vocab]           time the cached DFV was computed */
    float*    head_params;  /* packed fp32: per hidden layer W[in][out] then b[out]; then w_out[in], b_out.
                               Read at every gear_forward_backward; never written by the library */
    void*     workspace;    /* scratch, 256-byte aligned, >= gear_workspace_bytes; contents belong to the ctx */
    size_t    workspace_bytes;
} gear_buffers;

/* Adam (Kingma and Ba 2015, Algorithm 1), the optimiser of the paper's experiments (Section 4: learning rate 1e-4):
 *   m = beta1 m + (1 - beta1) g;  v = beta2 v + (1 - beta2) g^2;
 *   p -= lr * (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps),   t = 1, 2, ... */
typedef struct { float lr, beta1, beta2, eps; } gear_adam;

/* One batch of page views (Table 1 of the paper) in CSR form; device pointers. */
typedef struct {
    int32_t B;                 /* views, 0 <= B <= max_batch */
    int64_t nnz;               /* image occurrences, = img_off[B], <= max_nnz */
    const int32_t* user_id;    /* [B] */
    const int32_t* url_id;     /* [B]  URL already hashed to a bucket */
    const int32_t* img_off;    /* [B+1] img_off[0] = 0, non-decreasing, img_off[B] = nnz */
    const int32_t* img_id;     /* [nnz] view-major, slot-minor */
    const float*   label;      /* [B]  0 or 1 */
    const float*   fast;       /* [B][fast_dim] fp32, 16-byte aligned: the views' own dense input; NULL when fast_dim = 0 */
} gear_batch;

/* Outputs of one step; device pointers.  "optional" ones may be NULL. */
typedef struct {
    float* loss;        /* [1]  mean binary cross-entropy over the batch */
    float* prob;        /* [B]  sigmoid of the logit; optional */
    float* head_grad;   /* packed like head_params: dLoss/dparams (not applied by the library) */
    float* dX;          /* [B][d_in] dLoss/d(head input), d_in = 2*emb_dim + dfv_dim + fast_dim.  Columns
                           [2*emb_dim, 2*emb_dim + dfv_dim) are dLoss/d(pooled DFV) of each view: pass dX + 2*emb_dim
                           with ld = d_in to gear_accumulate_dfv_grad */
    int32_t* row_view;  /* [nnz] view index of every image occurrence (the src_row of accumulate); optional */
    float*   inv_n;     /* [B]   1/n_b, the mean-pool weight (the scale of accumulate); optional */
    void*  x_debug;     /* [B][d_in] copy of the head input in head_dtype; optional */
    float* dfv_grad;    /* [nnz][dfv_dim] optional: event 5 in its materialised form, one gradient row per image
                           occurrence (view-major, slot-minor): dX[view][2*emb_dim ..] * 1/n_view.  Needs row_view and
                           inv_n.  These are the rows a worker sends to the owners of the images */
    float* user_grad;   /* [user_vocab][emb_dim] optional: the summed embedding gradient is ADDED here and the */
    float* url_grad;    /* [url_vocab][emb_dim]  table is left untouched (both or neither) */
    /* Optional: Section 4's optimiser for the embedding tables in place of the plain scaled scatter (adam != NULL; not
     * together with user_grad / url_grad).  Every row that received a gradient in this step takes one Adam step with
     * the step count adam_step (>= 1) and its own rows of the moment tables; rows without a gradient, and their
     * moments, stay as they are.  lr of gear_forward_backward is ignored.  The struct is host memory. */
    const gear_adam* adam;
    int64_t adam_step;
    float *user_m, *user_v;   /* [user_vocab][emb_dim] first and second moments, zero before the first step */
    float *url_m, *url_v;     /* [url_vocab][emb_dim] */
} gear_step_out;

/* Bytes of workspace a ctx with this configuration needs.  Host-only. */
int gear_workspace_bytes(const gear_config* cfg, size_t* out_bytes);

/*
 * Create a ctx.  fill = 0: keep the caller's table contents (dfv_gcnt must be
 * in [0, M)).  fill = 1: user/url/DFV tables get the procedural uniform fill
 * with standard deviation 0.1 (the paper's initial value for all variables),
 * tags GEAR_TAG_USER/URL/DFV; dfv_gsum and dfv_gcnt are zeroed; dfv_ts[id] =
 * now - (draw(seed, GEAR_TAG_TS, id) mod max(expire, 1)).  The workspace is
 * initialised in both cases.  Synchronises the stream before returning.
 */
int gear_init_tables(gear_ctx** out_ctx, const gear_config* cfg, const gear_buffers* buf,
                     uint64_t seed, int fill, int64_t now, void* stream);

/*
 * Events 1, 3, 4.  X[b] = [user_emb[user_id[b]] | url_emb[url_id[b]] | mean_j DFV[img_id[j]] | fast[b]] (fp32 sum
 * in slot order, divided by n_b; zeros for n_b = 0; the last part only when fast_dim > 0); hidden layers h = ReLU(h W + b); z = h . w_out + b_out;
 * p = sigmoid(z); loss = mean_b BCE(p_b, label_b).  Backward yields head_grad and dX.  Then, per
 * embedding table, rows of views sharing an ID are summed and table[id] -= lr * sum (or the sums are
 * added to user_grad / url_grad when those are given).
 */
int gear_forward_backward(gear_ctx* ctx, const gear_batch* batch, float lr, const gear_step_out* out,
                          void* stream);

/*
 * Event 5 + 6a.  Row r (0 <= r < n) carries Image ID img_id[r] and the gradient
 *     g_r[c] = grads[s * ld + c] * (scale ? scale[s] : 1),  s = src_row ? src_row[r] : r,  c < dfv_dim.
 * Rows are taken to arrive in index order.  Per image: dfv_gsum += g_r, dfv_gcnt += 1; when the count
 * reaches M the group's average (sum / M, fp32) joins the ready queue and sum and count restart at 0;
 * a call may complete several groups of one image.  grads rows must be 16-byte aligned (ld multiple of 4).
 * If the queue cannot take every group the call completes, the whole call is dropped and
 * GEAR_DEV_READY_OVERFLOW is raised.
 * img_id == NULL means "the image occurrences of the batch of the most recent gear_forward_backward on
 * this ctx" (n must equal that batch's nnz; the batch's img_id array must not have changed): their IDs
 * were already key-sorted during that call, so the sort is not repeated.  GEAR_ERR_STATE if there is no
 * such batch.
 */
int gear_accumulate_dfv_grad(gear_ctx* ctx, const int32_t* img_id, const float* grads, int64_t ld,
                             const int32_t* src_row, const float* scale, int64_t n, void* stream);

/*
 * Event 6b.  Moves the ready queue to (ids[k], seq[k], avg[k][dfv_dim]), k < n, sorted by (id, seq);
 * seq numbers the emissions of one image since the previous collect, in arrival order.  The count is
 * written to *d_n (device, optional) and *h_n (host, optional: the call then synchronises).  If the queue
 * holds more than cap entries nothing is moved, the required count is reported, GEAR_DEV_OUT_CAPACITY is
 * raised and (when h_n is given) GEAR_ERR_CAPACITY is returned.
 */
int gear_collect_ready(gear_ctx* ctx, int32_t* ids, int32_t* seq, float* avg, int64_t cap,
                       int64_t* d_n, int64_t* h_n, void* stream);

/*
 * Events 5 and 6 in one call (Section 3: the gradients arrive and, as soon as M of an image are there, their average
 * goes on to the Dense Part): the same results as gear_accumulate_dfv_grad followed by gear_collect_ready with the
 * same arguments.  When no average was waiting in the ready queue before the call and cap >= n, the averages of
 * the groups this call completes are written straight into ids / seq / avg without passing through the queue;
 * in every other case the library does the two steps one after the other.  Capacity behaviour as in
 * gear_collect_ready (too small: the completed groups stay in the queue, nothing is handed over).
 */
int gear_accumulate_collect(gear_ctx* ctx, const int32_t* img_id, const float* grads, int64_t ld,
                            const int32_t* src_row, const float* scale, int64_t n,
                            int32_t* ids, int32_t* seq, float* avg, int64_t cap,
                            int64_t* d_n, int64_t* h_n, void* stream);

/*
 * Expiry scan.  Lists, in ascending order, every image with now - dfv_ts[id] >= expire; with
 * restamp != 0 the listed entries get dfv_ts[id] = now (a refresh has been requested).  Count and
 * capacity behaviour as in gear_collect_ready (too small: nothing listed, nothing restamped).
 * The scan reads and writes nothing the other calls use (only dfv_ts, its own part of the workspace and the
 * device status word), so it may be enqueued on a stream of its own and run beside a training step on the
 * same ctx; the caller orders it against its own readers and writers of dfv_ts, ids and d_n.  gear_status,
 * gear_profile_* and gear_destroy wait for that stream as well.
 */
int gear_collect_expired(gear_ctx* ctx, int64_t now, int restamp, int32_t* ids, int64_t cap,
                         int64_t* d_n, int64_t* h_n, void* stream);

/*
 * Refresh of cached inference results (Section 1, second point; Section 3: a Dense Feature Vector whose cached
 * copy has expired is computed again by the Dense Part).  For k < n:
 *     dfv[ids[k]][c] = rows[k * ld + c] rounded to dfv_dtype (bf16: nearest even), c < dfv_dim;  dfv_ts[ids[k]] = now.
 * The gradient store is not touched: gradients taken against the old vector keep accumulating.
 * ids: device, distinct -- the list gear_collect_expired returns qualifies; if an ID repeats, one of its rows is
 * stored, unspecified which.  rows: device fp32, 16-byte aligned, ld a multiple of 4.  An ID outside
 * [0, img_vocab) is skipped and raises GEAR_DEV_BAD_ID.  d_n (device, optional): the call processes
 * min(n, *d_n) entries, *d_n read on the device when the kernel runs, so that the count an expiry scan has just
 * written can be used without a trip to the host (n is then the capacity of ids / rows).
 * The call writes dfv and dfv_ts: the caller orders it after the training calls that should still see the old
 * vectors and before the next expiry scan (same stream, or events between streams).
 */
int gear_refresh_dfv(gear_ctx* ctx, const int32_t* ids, const float* rows, int64_t ld, int64_t n,
                     const int64_t* d_n, int64_t now, void* stream);

/*
 * Tables partitioned by ID across devices (Section 3: the Slowgear Workers serve the Fastgear Workers' requests "by
 * partition of Image ID"; Section 4 runs N of each).  The exchange itself is the caller's (any all-to-all); these two
 * calls are what the owner of a table shard does with what arrives.
 *
 * gear_fetch_rows      event 3, the owner's answer to a request: out[k] = row ids[k] of table `which`
 *                      (GEAR_TABLE_USER / URL: emb_dim fp32; GEAR_TABLE_DFV: dfv_dim values in dfv_dtype), k < n, dense,
 *                      bit-exact copies; an ID outside the table gives a zero row and raises GEAR_DEV_BAD_ID.
 *                      out: device, 16-byte aligned.
 * gear_apply_emb_grad  event 4's push, at the owner: table[id] -= lr * (sum of the rows[k], k < n, with ids[k] == id) for
 *                      `which` = GEAR_TABLE_USER or GEAR_TABLE_URL; rows fp32 [n][ld >= emb_dim], 16-byte aligned, ld a
 *                      multiple of 4; n <= max_batch.  What gear_forward_backward does with its own batch's rows.
 * Gradient rows for the image store arrive the same way and go to gear_accumulate_dfv_grad / gear_accumulate_collect
 * with explicit img_id (rows are taken to arrive in index order: sender by sender, each in its own row order).
 */
int gear_fetch_rows(gear_ctx* ctx, int32_t which, const int32_t* ids, int64_t n, void* out, void* stream);
int gear_apply_emb_grad(gear_ctx* ctx, int32_t which, const int32_t* ids, const float* rows, int64_t ld, int64_t n,
                        float lr, void* stream);

/*
 * The smallest Dense Part there is, for closing the loop on one device: DFV[id] = raw[id] . Wd, with raw
 * [img_vocab][raw_dim] the images' raw feature rows and Wd [raw_dim][dfv_dim] the Dense Part's weights (fp32, device,
 * row-major).
 *
 * gear_dense_forward   Section 3, events 2 and 3 (Dense Part inference): rows[k][c] = sum_r raw[ids[k]][r] Wd[r][c] for
 *                      k < n (and k < *d_n when d_n, a device count such as the one an expiry scan wrote, is given);
 *                      rows fp32 with leading dimension ld >= dfv_dim: the input gear_refresh_dfv takes.
 * gear_dense_backward  Section 3, event 6, second half; Eq. 1, right factor: Wd_grad[r][c] += sum over the emissions
 *                      e < n (e < *d_n) of raw[ids[e]][r] * avg[e][c]; ids / avg are the lists gear_collect_ready or
 *                      gear_accumulate_collect returned (avg rows dfv_dim apart).  Wd_grad is added to: the caller
 *                      zeroes it.  Sums are fp32 in an order the hardware picks.
 * An ID outside [0, img_vocab) contributes a zero row / nothing and raises GEAR_DEV_BAD_ID.
 */
int gear_dense_forward(gear_ctx* ctx, const float* raw, int32_t raw_dim, const float* Wd, const int32_t* ids, int64_t n,
                       const int64_t* d_n, float* rows, int64_t ld, void* stream);
int gear_dense_backward(gear_ctx* ctx, const float* raw, int32_t raw_dim, const int32_t* ids, const float* avg,
                        int64_t n, const int64_t* d_n, float* Wd_grad, void* stream);

/*
 * One Adam step (Section 4) on n parameters that all have a gradient: the head's parameters with the head_grad of a
 * step, the Dense Part's weights with the Wd_grad of gear_dense_backward.  param, grad, m, v: device fp32 [n]; m and
 * v zero before the first step; t >= 1 counts the steps.  cfg is host memory.
 */
int gear_adam_dense(float* param, const float* grad, float* m, float* v, int64_t n, int64_t t, const gear_adam* cfg,
                    void* stream);

/*
 * Synchronises the stream last used; returns the device status word (GEAR_DEV_* bits, then cleared) and
 * the number of averages waiting in the ready queue.  Either out-pointer may be NULL.  Returns
 * GEAR_ERR_BAD_ID if GEAR_DEV_BAD_ID was set, GEAR_ERR_CAPACITY for the two capacity bits, else GEAR_OK.
 */
int gear_status(gear_ctx* ctx, int32_t* device_status, int64_t* pending_ready);

/* Releases the ctx (host memory only).  Synchronises the stream last used.  The pointer is dangling afterwards:
 * passing it to any call again, gear_destroy included, is undefined. */
int gear_destroy(gear_ctx* ctx);

/*
 * Procedural fill used by gear_init_tables, exposed for building synthetic inputs on the device.
 * Element (r, c) of a [n_rows][dim] array is  float(k - 2^23) * float(amp / 2^23)  with
 * k = top 24 bits of draw(seed, tag, r * dim + c), draw(seed, tag, i) = mix(mix(seed + G*(tag+1)) + G*(i+1)),
 * mix = the SplitMix64 finaliser and G = 0x9e3779b97f4a7c15 (Steele, Lea, Flood 2014); bf16 output is
 * the nearest-even rounding of that float.  Not part of the paper.  dst: device, 16-byte aligned.
 */
int gear_fill_uniform(void* dst, int32_t dtype, int64_t n_rows, int32_t dim, uint64_t seed, uint64_t tag,
                      double amp, void* stream);

/*
 * The expiry scan for callers that cannot allocate device memory.  (The paper has no counterpart: it is
 * gear_collect_expired without a ctx.)
 *
 * Who needs it: code that runs where cudaMalloc is not available to it -- a serving process whose device
 * memory was partitioned at start-up, a plug-in that receives buffers but no allocator, a path on which an
 * allocation's implicit device synchronisation is not acceptable.  Such a caller cannot supply the
 * workspace a gear_ctx requires, so this call takes the timestamp table directly and keeps its scratch in
 * a fixed array inside the library image.
 *
 *   - Same semantics as gear_collect_expired: lists, ascending, every id < img_vocab with
 *     now - dfv_ts[id] >= expire; restamp != 0 sets dfv_ts[id] = now for the listed ones; count to *d_n
 *     (device, optional) and *h_n (host, optional: then the call synchronises the stream); cap too small:
 *     nothing is listed or restamped, the required count is reported and, with h_n, GEAR_ERR_CAPACITY returned.
 *   - img_vocab may be at most GEAR_STATIC_EXPIRY_MAX_VOCAB; larger tables are refused with
 *     GEAR_ERR_CAPACITY before anything is enqueued.
 *   - Cost: every GPU on which the library is loaded holds GEAR_STATIC_EXPIRY_SCRATCH_BYTES (about 2.2 MB)
 *     of device memory for this array until the process exits, whether or not the call is ever made.
 *   - The first call on a device looks up the array's device address (once per device, with that device
 *     current); make that first call before starting any stream capture.
 *   - The call allocates nothing, on the device or through any library.
 *   - All calls on one device share the array.  Calls whose kernels may overlap on the GPU (different
 *     streams without ordering between them) race on it: order them.  Nothing in the array carries over
 *     from one call to the next.
 * dfv_ts and ids are device pointers; dfv_ts is written only when restamp != 0.
 */
#define GEAR_STATIC_EXPIRY_MAX_VOCAB 16777216
#define GEAR_STATIC_EXPIRY_SCRATCH_BYTES (256 + GEAR_STATIC_EXPIRY_MAX_VOCAB / 8 + 65792)
int gear_collect_expired_static(int64_t* dfv_ts, int64_t img_vocab, int64_t expire, int64_t now, int restamp,
                                int32_t* ids, int64_t cap, int64_t* d_n, int64_t* h_n, void* stream);

/*
 * Per-kernel timing (not part of the paper).  While enabled, every kernel the library launches for this
 * ctx is bracketed by a pair of CUDA events on the caller's stream.  gear_profile_read synchronises,
 * sums the elapsed time and the launch count per kernel name since the last read or enable, writes up to
 * cap entries (names: cap rows of 64 chars, NUL-terminated; total_ms, launches: cap entries) and clears
 * the records.  Event records cost a few microseconds each, and while profiling is on the library keeps all
 * its work on the caller's stream (no side stream), so that every kernel is timed alone: do not time
 * throughput with profiling on.
 * gear_launch_count returns the number of kernels this ctx has launched since it was created.
 * on = 2 is the timeline mode: the events are recorded, but the library keeps its side stream, so that
 * gear_profile_timeline can show what ran beside what: start and stop of every launch since the mode was switched on,
 * in milliseconds after the first launch's start, in launch order (cap entries at most; names as in gear_profile_read).
 * A kernel's start event completes when the stream reaches it, which may be well before the kernel's blocks get an SM.
 */
int gear_profile_enable(gear_ctx* ctx, int on);
int gear_profile_timeline(gear_ctx* ctx, char* names, float* start_ms, float* stop_ms, int32_t cap, int32_t* n_out);
int gear_profile_read(gear_ctx* ctx, char* names, float* total_ms, int32_t* launches, int32_t cap, int32_t* n_out);
int gear_launch_count(gear_ctx* ctx, int64_t* n_launches);

/* Last CUDA error string seen by the library on this thread ("" if none).  Host-only. */
const char* gear_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* GEAR_H */
