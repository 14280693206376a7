/*
 * gear_oracle.c -- CPU oracle for the Gear Training sparse-part step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the parity authority for the CUDA
 * library: a plain, slow, single-threaded restatement of what the step
 * computes, written from the paper (arXiv 1806.03925).  It shares no code
 * with the CUDA path and must never be linked, imported or called by it.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * All arithmetic is IEEE double.  Tables are read in their storage type
 * (double, float or bfloat16 bit patterns) through load_elem().
 *
 * What each function follows:
 *   orc_forward_backward  Section 3, events 1, 3 and 4: fetch the cached Dense
 *                         Feature Vectors (DFVs) by Image ID, run the Sparse
 *                         Part forward to the loss, back-propagate through the
 *                         Sparse Part only, and stop at dLoss/dDFV (left
 *                         factor of Eq. 1).
 *   orc_emb_apply         event 4, "push gradients of Sparse Part".
 *   orc_dfv_grad_rows     event 5: one (Image ID, gradient) pair per image
 *                         occurrence.
 *   orc_accumulate        Section 1 (third point) and event 6: keep the
 *                         gradients of an image until M have arrived, then
 *                         emit their average.
 *   orc_accumulate_pooled the same store when arrival order is not recorded
 *                         (asynchronous workers): emissions carry the mean of
 *                         the pooled gradients.
 *   orc_collect_expired   Section 1 (second point) and Section 3: cached
 *                         inference results older than the inference-expired
 *                         time are dropped / refreshed.
 *   orc_refresh_dfv       Section 1 (second point) and Section 3: a refreshed
 *                         Dense Feature Vector replaces the expired cached one
 *                         and restarts its clock.
 *   orc_dense_forward     Section 3, events 2 and 3, for a linear Dense Part
 *                         (DFV = raw image row times a weight matrix).
 *   orc_dense_backward    event 6, second half; right factor of Eq. 1: the
 *                         averaged gradients go back through the Dense Part.
 *   orc_adam_step         Section 4: the optimiser of the paper's experiments
 *   orc_emb_adam          (Adam), dense and for the rows of an embedding
 *                         table that received a gradient.
 *   orc_fill_*            not in the paper: counter-based table
 *                         initialisation (SplitMix64, Steele, Lea and Flood
 *                         2014) so that tables too large to ship can be
 *                         regenerated row by row.
 *
 * Parity pins (tests/test_oracle_pins.py): finite differences and a
 * reverse-mode autodiff library for the head and the pooling; closed forms;
 * a literal keep-every-gradient-in-a-list store for the accumulate rule;
 * Eq. 1 with a linear dense part at M = 1 and zero expiry; count
 * conservation; expiry special cases; the Dense Part's gradient by finite
 * differences of the loss; Adam against an optimiser library in double
 * precision and the closed form of its first step.
 * Parity unpinned: the training-trajectory effects the paper reports
 * (convergence against expiry time and M) -- figures and datasets are not
 * available, nothing here claims them.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_F64 = 0, ORC_F32 = 1, ORC_BF16 = 2 };

typedef struct {
    int64_t user_vocab, url_vocab, img_vocab;
    int32_t emb_dim, dfv_dim;
    int32_t n_hidden;      /* 1 or 2 hidden ReLU layers, then one logistic unit */
    int32_t hidden[2];
    int32_t round_bf16;    /* 1: operands of the head's matrix products are rounded to bfloat16 */
    int32_t fast_dim;      /* dense input columns the Fastgear side brings along per view (Section 4: the part of
                              the image fed to the Fastgear Worker directly); appended to the head input */
} orc_model;

/* ---------------------------------------------------------------- storage */

static float bf16_bits_to_float(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* round-to-nearest-even float -> bfloat16 bit pattern */
static uint16_t float_to_bf16_bits(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40); /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

static double load_elem(const void* p, int dtype, int64_t i) {
    switch (dtype) {
    case ORC_F64: return ((const double*)p)[i];
    case ORC_F32: return (double)((const float*)p)[i];
    default:      return (double)bf16_bits_to_float(((const uint16_t*)p)[i]);
    }
}

static void store_elem(void* p, int dtype, int64_t i, double v) {
    switch (dtype) {
    case ORC_F64: ((double*)p)[i] = v; break;
    case ORC_F32: ((float*)p)[i] = (float)v; break;
    default:      ((uint16_t*)p)[i] = float_to_bf16_bits((float)v); break;
    }
}

/* value -> nearest bfloat16 (via float, as the device rounds an fp32 accumulator) */
static double round_bf16(double v) {
    return (double)bf16_bits_to_float(float_to_bf16_bits((float)v));
}

double orc_round_bf16(double v) { return round_bf16(v); }

/* ------------------------------------------------- procedural table fill */

static const uint64_t GAMMA = 0x9e3779b97f4a7c15ull;

static uint64_t mix64(uint64_t z) {
    z ^= z >> 30; z *= 0xbf58476d1ce4e5b9ull;
    z ^= z >> 27; z *= 0x94d049bb133111ebull;
    z ^= z >> 31;
    return z;
}

uint64_t orc_mix64(uint64_t z) { return mix64(z); }

/* The idx-th output (0-based) of the SplitMix64 stream whose seed is derived
 * from (seed, tag). */
uint64_t orc_draw(uint64_t seed, uint64_t tag, uint64_t idx) {
    uint64_t key = mix64(seed + GAMMA * (tag + 1));
    return mix64(key + GAMMA * (idx + 1));
}

/* Uniform value on a 2^24-point grid in [-amp, amp): one int->float
 * conversion (exact) and one float multiply, so any IEEE machine agrees. */
static float fill_value(uint64_t seed, uint64_t tag, uint64_t idx, double amp) {
    float step = (float)(amp / 8388608.0);
    int32_t k = (int32_t)(orc_draw(seed, tag, idx) >> 40) - 8388608;
    return (float)k * step;
}

/* out[i, :] = row rows[i] (or row i when rows == NULL) of the procedural
 * table (seed, tag) with `dim` columns; element (r, c) uses counter r*dim+c. */
int orc_fill_rows(uint64_t seed, uint64_t tag, int32_t dim, double amp,
                  const int64_t* rows, int64_t n_rows, int out_dtype, void* out) {
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t r = rows ? rows[i] : i;
        for (int32_t c = 0; c < dim; ++c) {
            float v = fill_value(seed, tag, (uint64_t)r * (uint64_t)dim + (uint64_t)c, amp);
            store_elem(out, out_dtype, i * dim + c, (double)v);
        }
    }
    return 0;
}

/* Procedural timestamps: ts[id] = now - (draw mod span), span = max(expire, 1). */
int orc_fill_ts(uint64_t seed, uint64_t tag, int64_t expire, int64_t now,
                const int64_t* rows, int64_t n_rows, int64_t* out) {
    uint64_t span = expire > 1 ? (uint64_t)expire : 1u;
    for (int64_t i = 0; i < n_rows; ++i) {
        int64_t r = rows ? rows[i] : i;
        out[i] = now - (int64_t)(orc_draw(seed, tag, (uint64_t)r) % span);
    }
    return 0;
}

/* ----------------------------------------------------------------- head */

static int64_t head_param_count(const orc_model* m) {
    int64_t n = 0, fan = 2 * m->emb_dim + m->dfv_dim + m->fast_dim;
    for (int l = 0; l < m->n_hidden; ++l) { n += fan * m->hidden[l] + m->hidden[l]; fan = m->hidden[l]; }
    return n + fan + 1;
}

int64_t orc_head_param_count(const orc_model* m) { return head_param_count(m); }

/*
 * One forward + backward pass of the Sparse Part over a batch of page views.
 *
 * Inputs : the three tables (storage type given per table), packed head
 *          parameters (doubles: per hidden layer W[in][out] then b[out]; then
 *          w_out[in], b_out), and the batch in CSR form.
 *          fast[B][fast_dim] (fast_dim > 0): dense input the view brings itself.
 * Outputs: X[B][Din]   head input = [user row | url row | mean of the view's DFVs | fast row]
 *          prob[B]     sigmoid(z)
 *          *loss       mean binary cross-entropy
 *          head_grad   dLoss/dparams, packed like params
 *          dX[B][Din]  dLoss/dX; its last dfv_dim columns are dLoss/d(pooled DFV)
 * Any output pointer except X and loss may be NULL (forward only).
 *
 * The derivative of ReLU is decided by the sign of a floating-point number.  A
 * pre-activation within rounding distance of zero may fall on the other side
 * on a machine that sums in another order or precision, and either decision is
 * then a correct evaluation of the method.  So that a comparison can accept
 * both decisions there and nowhere else, the units (layer l, view b, column j)
 * with |pre-activation| <= relu_margin + relu_margin_rel * max_i|in_i| *
 * max|W_l| (in: the unit's input row, W_l: the layer's weights as the product
 * sees them) are listed in near_units (coded (l * B + b) * 1024 + j; *n_near
 * receives their number, near_cap bounds the list; near_units may be NULL;
 * near_abs, optional, receives |pre-activation| of every listed unit), and the
 * units named in flip_units take the other branch in the backward pass (their
 * forward value is left as computed).  The list reports; it changes no result.
 *
 * Returns the number of out-of-range IDs met (their rows count as zeros).
 */
int64_t orc_forward_backward(const orc_model* m,
                             const void* user_emb, int user_dt,
                             const void* url_emb, int url_dt,
                             const void* dfv, int dfv_dt,
                             const double* params,
                             int32_t B, const int32_t* user_id, const int32_t* url_id,
                             const int32_t* img_off, const int32_t* img_id, const double* label,
                             const double* fast,
                             double* X, double* prob, double* loss,
                             double* head_grad, double* dX,
                             double relu_margin, double relu_margin_rel, int64_t* near_units, double* near_abs,
                             int64_t near_cap, int64_t* n_near,
                             const int64_t* flip_units, int64_t n_flip) {
    const int E = m->emb_dim, D = m->dfv_dim, F = m->fast_dim, Din = 2 * E + D + F;
    const int L = m->n_hidden;
    const int rb = m->round_bf16;
    int64_t bad = 0;
    if (n_near) *n_near = 0;

    /* parameter views */
    const double* W[2] = {0, 0}; const double* bias[2] = {0, 0};
    int fan[3]; fan[0] = Din;
    int64_t pos = 0;
    for (int l = 0; l < L; ++l) {
        W[l] = params + pos; pos += (int64_t)fan[l] * m->hidden[l];
        bias[l] = params + pos; pos += m->hidden[l];
        fan[l + 1] = m->hidden[l];
    }
    const double* w_out = params + pos; pos += fan[L];
    const double b_out = params[pos];
    const int64_t n_par = pos + 1;

    /* rounded copies of the matrix-product operands (identity when rb == 0) */
    double* Wr[2] = {0, 0};
    double w_amax[2] = {0.0, 0.0};
    for (int l = 0; l < L; ++l) {
        int64_t n = (int64_t)fan[l] * m->hidden[l];
        Wr[l] = (double*)malloc(sizeof(double) * n);
        for (int64_t i = 0; i < n; ++i) {
            Wr[l][i] = rb ? round_bf16(W[l][i]) : W[l][i];
            if (fabs(Wr[l][i]) > w_amax[l]) w_amax[l] = fabs(Wr[l][i]);
        }
    }

    /* events 1-3: gather the embeddings, fetch and mean-pool the DFVs */
    for (int32_t b = 0; b < B; ++b) {
        double* x = X + (int64_t)b * Din;
        int32_t u = user_id[b], h = url_id[b];
        if (u < 0 || u >= m->user_vocab) { ++bad; for (int c = 0; c < E; ++c) x[c] = 0.0; }
        else for (int c = 0; c < E; ++c) x[c] = load_elem(user_emb, user_dt, (int64_t)u * E + c);
        if (h < 0 || h >= m->url_vocab) { ++bad; for (int c = 0; c < E; ++c) x[E + c] = 0.0; }
        else for (int c = 0; c < E; ++c) x[E + c] = load_elem(url_emb, url_dt, (int64_t)h * E + c);
        double* pool = x + 2 * E;
        for (int c = 0; c < D; ++c) pool[c] = 0.0;
        int32_t n_b = img_off[b + 1] - img_off[b];
        for (int32_t j = img_off[b]; j < img_off[b + 1]; ++j) {
            int32_t id = img_id[j];
            if (id < 0 || id >= m->img_vocab) { ++bad; continue; }
            for (int c = 0; c < D; ++c) pool[c] += load_elem(dfv, dfv_dt, (int64_t)id * D + c);
        }
        if (n_b > 0) for (int c = 0; c < D; ++c) pool[c] /= (double)n_b;
        for (int c = 0; c < F; ++c) x[2 * E + D + c] = fast[(int64_t)b * F + c];     /* the view's own dense input */
        if (rb) for (int c = 0; c < Din; ++c) x[c] = round_bf16(x[c]);
    }

    /* event 4, forward: hidden ReLU layers, logistic output, mean BCE */
    double* H[3]; H[0] = X;
    for (int l = 0; l < L; ++l) H[l + 1] = (double*)malloc(sizeof(double) * (size_t)B * m->hidden[l]);
    double* dz = (double*)malloc(sizeof(double) * (size_t)(B > 0 ? B : 1));
    double total = 0.0;
    for (int32_t b = 0; b < B; ++b) {
        for (int l = 0; l < L; ++l) {
            const int K = fan[l], N = m->hidden[l];
            const double* in = H[l] + (int64_t)b * K;
            double* out = H[l + 1] + (int64_t)b * N;
            for (int j = 0; j < N; ++j) out[j] = 0.0;
            double in_amax = 0.0;
            for (int i = 0; i < K; ++i) {
                const double xi = in[i];
                const double* wrow = Wr[l] + (int64_t)i * N;
                for (int j = 0; j < N; ++j) out[j] += xi * wrow[j];
                if (fabs(xi) > in_amax) in_amax = fabs(xi);
            }
            const double near = relu_margin + relu_margin_rel * in_amax * w_amax[l];
            for (int j = 0; j < N; ++j) {
                double a = out[j] + bias[l][j];
                if (near_units && fabs(a) <= near) {
                    if (*n_near < near_cap) {
                        near_units[*n_near] = ((int64_t)l * B + b) * 1024 + j;
                        if (near_abs) near_abs[*n_near] = fabs(a);
                    }
                    ++*n_near;
                }
                a = a > 0.0 ? a : 0.0;
                out[j] = rb ? round_bf16(a) : a;
            }
        }
        const double* top = H[L] + (int64_t)b * fan[L];
        double z = b_out;
        for (int i = 0; i < fan[L]; ++i) z += top[i] * w_out[i];
        const double y = label[b];
        const double p = 1.0 / (1.0 + exp(-z));
        /* -[y log p + (1-y) log(1-p)] in its overflow-safe form */
        total += (z > 0.0 ? z : 0.0) - z * y + log1p(exp(-fabs(z)));
        if (prob) prob[b] = p;
        dz[b] = (p - y) / (double)B;
    }
    *loss = B > 0 ? total / (double)B : 0.0;

    /* event 4, backward through the Sparse Part, down to dLoss/dX */
    if (head_grad && dX) {
        for (int64_t i = 0; i < n_par; ++i) head_grad[i] = 0.0;
        double* gW[2]; double* gb[2];
        pos = 0;
        for (int l = 0; l < L; ++l) {
            gW[l] = head_grad + pos; pos += (int64_t)fan[l] * m->hidden[l];
            gb[l] = head_grad + pos; pos += m->hidden[l];
        }
        double* gw_out = head_grad + pos; pos += fan[L];
        double* gb_out = head_grad + pos;
        int maxw = Din;
        for (int l = 0; l < L; ++l) if (m->hidden[l] > maxw) maxw = m->hidden[l];
        double* d_hi = (double*)malloc(sizeof(double) * maxw);
        double* d_lo = (double*)malloc(sizeof(double) * maxw);
        for (int32_t b = 0; b < B; ++b) {
            const double* top = H[L] + (int64_t)b * fan[L];
            *gb_out += dz[b];
            for (int i = 0; i < fan[L]; ++i) {
                gw_out[i] += top[i] * dz[b];
                d_hi[i] = dz[b] * w_out[i];            /* dLoss/d(top activation) */
            }
            for (int l = L - 1; l >= 0; --l) {
                const int K = fan[l], N = m->hidden[l];
                const double* in = H[l] + (int64_t)b * K;
                const double* out = H[l + 1] + (int64_t)b * N;
                /* through the ReLU (derivative 0 at 0); operand rounding for bf16 heads */
                for (int j = 0; j < N; ++j) {
                    int active = out[j] > 0.0;
                    for (int64_t q = 0; q < n_flip; ++q)
                        if (flip_units[q] == ((int64_t)l * B + b) * 1024 + j) active = !active;
                    double g = active ? d_hi[j] : 0.0;
                    d_hi[j] = rb ? round_bf16(g) : g;
                    gb[l][j] += d_hi[j];
                }
                for (int i = 0; i < K; ++i) {
                    const double xi = in[i];
                    const double* wrow = Wr[l] + (int64_t)i * N;
                    double* gwrow = gW[l] + (int64_t)i * N;
                    double acc = 0.0;
                    for (int j = 0; j < N; ++j) {
                        gwrow[j] += xi * d_hi[j];
                        acc += wrow[j] * d_hi[j];
                    }
                    d_lo[i] = acc;
                }
                double* t = d_hi; d_hi = d_lo; d_lo = t;
            }
            for (int c = 0; c < Din; ++c) dX[(int64_t)b * Din + c] = d_hi[c];
        }
        free(d_hi); free(d_lo);
    }
    for (int l = 0; l < L; ++l) { free(H[l + 1]); free(Wr[l]); }
    free(dz);
    return bad;
}

/*
 * Event 4, second half: apply the embedding gradients of one ID column.
 * G[id] = sum over the views b (ascending) with ids[b] == id of
 * dX[b][col0 .. col0+E); then table[id] += alpha * G[id], once per distinct id.
 * If G_out != NULL (dense double [vocab][E], caller-zeroed) the summed
 * gradient is added there and the table is left untouched.
 */
int64_t orc_emb_apply(void* table, int dt, int64_t vocab, int32_t E,
                      const int32_t* ids, int32_t B, const double* dX, int32_t ldx, int32_t col0,
                      double alpha, double* G_out) {
    int64_t bad = 0;
    double* G = G_out ? G_out : (double*)calloc((size_t)vocab * E, sizeof(double));
    uint8_t* seen = (uint8_t*)calloc((size_t)vocab, 1);
    for (int32_t b = 0; b < B; ++b) {
        int32_t id = ids[b];
        if (id < 0 || id >= vocab) { ++bad; continue; }
        seen[id] = 1;
        for (int c = 0; c < E; ++c) G[(int64_t)id * E + c] += dX[(int64_t)b * ldx + col0 + c];
    }
    if (!G_out) {
        for (int64_t id = 0; id < vocab; ++id) {
            if (!seen[id]) continue;
            for (int c = 0; c < E; ++c) {
                int64_t i = id * E + c;
                store_elem(table, dt, i, load_elem(table, dt, i) + alpha * G[i]);
            }
        }
        free(G);
    }
    free(seen);
    return bad;
}

/*
 * Event 5: the (Image ID, dLoss/dDFV) pairs of a batch, view-major and
 * slot-minor.  The pooled feature is the mean of the view's n_b DFVs, so each
 * occurrence receives dLoss/dpooled[b] * (1/n_b)  (Eq. 1, left factor).
 * rows[r][D] is written for r in [0, nnz).
 */
void orc_dfv_grad_rows(int32_t B, int32_t D, const int32_t* img_off,
                       const double* dX, int32_t ldx, int32_t col0, double* rows) {
    for (int32_t b = 0; b < B; ++b) {
        int32_t n_b = img_off[b + 1] - img_off[b];
        if (n_b <= 0) continue;
        double s = 1.0 / (double)n_b;
        for (int32_t j = img_off[b]; j < img_off[b + 1]; ++j)
            for (int c = 0; c < D; ++c)
                rows[(int64_t)j * D + c] = dX[(int64_t)b * ldx + col0 + c] * s;
    }
}

/*
 * Event 6 (first half): gradients arrive one at a time, in row order.
 *   sum[id] += g;  cnt[id] += 1;
 *   if cnt[id] == M: emit (id, seq[id], sum[id] / M); seq[id] += 1; sum[id] = 0; cnt[id] = 0.
 * seq[id] counts the emissions of id since the emit list was last collected.
 * Emissions are appended to (emit_id, emit_seq, emit_avg) starting at *n_emit,
 * up to emit_cap entries.  member_of (optional, [n]) receives for every
 * arrival the index of the emission it ended up in, or -1 while its group is
 * still open at the end of the call (arrivals of earlier calls that sit in
 * sum[] are not tracked).  Returns the number of out-of-range IDs (ignored
 * rows), or -1 if the emit list overflowed.
 */
int64_t orc_accumulate(double* sum, int32_t* cnt, int32_t* seq, int64_t vocab, int32_t D, int32_t M,
                       const int32_t* ids, const double* grads, int64_t n,
                       int32_t* emit_id, int32_t* emit_seq, double* emit_avg,
                       int64_t emit_cap, int64_t* n_emit, int64_t* member_of) {
    int64_t bad = 0;
    int64_t* open_head = NULL;   /* per id: first arrival of the open group, chained through next_in_group */
    int64_t* next_in_group = NULL;
    if (member_of) {
        open_head = (int64_t*)malloc(sizeof(int64_t) * (size_t)vocab);
        next_in_group = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n > 0 ? n : 1));
        for (int64_t i = 0; i < vocab; ++i) open_head[i] = -1;
        for (int64_t r = 0; r < n; ++r) member_of[r] = -1;
    }
    for (int64_t r = 0; r < n; ++r) {
        int32_t id = ids[r];
        if (id < 0 || id >= vocab) { ++bad; continue; }
        double* s = sum + (int64_t)id * D;
        const double* g = grads + r * D;
        for (int c = 0; c < D; ++c) s[c] += g[c];
        cnt[id] += 1;
        if (member_of) { next_in_group[r] = open_head[id]; open_head[id] = r; }
        if (cnt[id] == M) {
            if (*n_emit >= emit_cap) { free(open_head); free(next_in_group); return -1; }
            int64_t e = (*n_emit)++;
            emit_id[e] = id;
            emit_seq[e] = seq[id]++;
            for (int c = 0; c < D; ++c) { emit_avg[e * D + c] = s[c] / (double)M; s[c] = 0.0; }
            cnt[id] = 0;
            if (member_of) {
                for (int64_t q = open_head[id]; q >= 0; q = next_in_group[q]) member_of[q] = e;
                open_head[id] = -1;
            }
        }
    }
    free(open_head); free(next_in_group);
    return bad;
}

/*
 * The same store when the order of arrival is not recorded (the paper's
 * workers push gradients asynchronously, Section 3 events 5 and 6, so the
 * store may only know how many gradients an image holds and their sum).
 * All arrivals of the call are added first; then every image holding
 * k >= M gradients emits floor(k / M) averages, each the mean of all k pooled
 * gradients, and keeps k mod M gradients' worth of that mean:
 *     avg = sum / k;   emit floor(k / M) times;   sum = avg * (k mod M);   cnt = k mod M.
 * M * (sum of the emitted averages) + the kept sum equals the pooled sum, and
 * counts and emission counts are those of orc_accumulate.  Emissions are
 * listed image by image in order of first arrival.  Returns the number of
 * out-of-range IDs, or -1 if the emit list overflowed.
 */
int64_t orc_accumulate_pooled(double* sum, int32_t* cnt, int32_t* seq, int64_t vocab, int32_t D, int32_t M,
                              const int32_t* ids, const double* grads, int64_t n,
                              int32_t* emit_id, int32_t* emit_seq, double* emit_avg,
                              int64_t emit_cap, int64_t* n_emit) {
    int64_t bad = 0;
    for (int64_t r = 0; r < n; ++r) {
        int32_t id = ids[r];
        if (id < 0 || id >= vocab) { ++bad; continue; }
        double* s = sum + (int64_t)id * D;
        const double* g = grads + r * D;
        for (int c = 0; c < D; ++c) s[c] += g[c];
        cnt[id] += 1;
    }
    for (int64_t r = 0; r < n; ++r) {
        int32_t id = ids[r];
        if (id < 0 || id >= vocab) continue;
        const int32_t k = cnt[id];
        if (k < M) continue;                       /* also true once the image has been settled */
        double* s = sum + (int64_t)id * D;
        const int32_t e_count = k / M, rest = k % M;
        for (int32_t j = 0; j < e_count; ++j) {
            if (*n_emit >= emit_cap) return -1;
            int64_t e = (*n_emit)++;
            emit_id[e] = id;
            emit_seq[e] = seq[id]++;
            for (int c = 0; c < D; ++c) emit_avg[e * D + c] = s[c] / (double)k;
        }
        for (int c = 0; c < D; ++c) s[c] = s[c] / (double)k * (double)rest;
        cnt[id] = rest;
    }
    return bad;
}

/* The emit list has been handed over: emission numbering restarts. */
void orc_collect_ready(int32_t* seq, const int32_t* emit_id, int64_t n_emit) {
    for (int64_t e = 0; e < n_emit; ++e) seq[emit_id[e]] = 0;
}

/*
 * Inference-expired time: image id is expired when now - ts[id] >= expire.
 * IDs are listed in ascending order; with restamp != 0 a listed entry gets
 * ts[id] = now (a refresh has been issued for it).  Returns the count.
 */
int64_t orc_collect_expired(int64_t* ts, int64_t vocab, int64_t now, int64_t expire,
                            int restamp, int32_t* out_ids) {
    int64_t n = 0;
    for (int64_t id = 0; id < vocab; ++id) {
        if (now - ts[id] >= expire) {
            out_ids[n++] = (int32_t)id;
            if (restamp) ts[id] = now;
        }
    }
    return n;
}

/*
 * Refresh of cached inference results (Section 1, second point; Section 3: the
 * Slowgear side recomputes a Dense Feature Vector once its cached copy has
 * expired): row k of `rows` (fp32, leading dimension ld) replaces the cached
 * DFV of image ids[k], rounded to the table's storage type, and that image's
 * timestamp becomes now.  ts_ids[k] is the image's index into ts (a test that
 * keeps only some rows of a large table passes compact row numbers in ids and
 * the real IDs in ts_ids; NULL means ts_ids = ids).  Entries are taken in
 * index order.  An ID outside [0, vocab) is skipped; the return value counts
 * those.  The gradient store (sum, count) is not touched.
 */
int64_t orc_refresh_dfv(void* dfv, int dt, int64_t vocab, int32_t D, int64_t* ts, int64_t ts_len,
                        const int32_t* ids, const int32_t* ts_ids, const float* rows, int64_t ld,
                        int64_t n, int64_t now) {
    int64_t bad = 0;
    for (int64_t k = 0; k < n; ++k) {
        const int64_t id = ids[k];
        const int64_t t = ts_ids ? ts_ids[k] : id;
        if (id < 0 || id >= vocab || t < 0 || t >= ts_len) { ++bad; continue; }
        for (int32_t c = 0; c < D; ++c) store_elem(dfv, dt, id * (int64_t)D + c, (double)rows[k * ld + c]);
        ts[t] = now;
    }
    return bad;
}


/* --------------------------------------------------- a linear Dense Part */

/*
 * Dense Part inference (Section 3, events 2 and 3) for the smallest Dense Part
 * there is: a linear map of the image's raw feature row,
 *     DFV[id] = raw[id] . Wd        raw [vocab][R] (storage type given), Wd [R][D].
 * rows[k][D] receives the DFV of image ids[k]; an ID outside [0, vocab) gives a
 * zero row and is counted in the return value.
 */
int64_t orc_dense_forward(const void* raw, int raw_dt, int64_t vocab, int32_t R, const double* Wd, int32_t D,
                          const int32_t* ids, int64_t n, double* rows) {
    int64_t bad = 0;
    for (int64_t k = 0; k < n; ++k) {
        double* out = rows + k * D;
        for (int c = 0; c < D; ++c) out[c] = 0.0;
        const int64_t id = ids[k];
        if (id < 0 || id >= vocab) { ++bad; continue; }
        for (int r = 0; r < R; ++r) {
            const double x = load_elem(raw, raw_dt, id * (int64_t)R + r);
            for (int c = 0; c < D; ++c) out[c] += x * Wd[(int64_t)r * D + c];
        }
    }
    return bad;
}

/*
 * Event 6, second half, and the right factor of Eq. 1: the averaged gradient
 * of every completed group is back-propagated through the Dense Part.  For the
 * linear Dense Part dDFV[id][c] / dWd[r][c] = raw[id][r], so
 *     G[r][c] += sum over emissions e of raw[id_e][r] * avg_e[c].
 * G [R][D] is accumulated into (the caller zeroes it).  Returns the number of
 * out-of-range IDs (skipped).
 */
int64_t orc_dense_backward(const void* raw, int raw_dt, int64_t vocab, int32_t R, int32_t D,
                           const int32_t* ids, const double* avg, int64_t n, double* G) {
    int64_t bad = 0;
    for (int64_t e = 0; e < n; ++e) {
        const int64_t id = ids[e];
        if (id < 0 || id >= vocab) { ++bad; continue; }
        for (int r = 0; r < R; ++r) {
            const double x = load_elem(raw, raw_dt, id * (int64_t)R + r);
            for (int c = 0; c < D; ++c) G[(int64_t)r * D + c] += x * avg[e * D + c];
        }
    }
    return bad;
}

/* ------------------------------------------------------------ optimiser */

/*
 * One step of Adam (Kingma and Ba 2015, Algorithm 1), the optimiser of the
 * paper's Section 4 (learning rate 1e-4 there), on n parameters:
 *     m = b1 m + (1 - b1) g;   v = b2 v + (1 - b2) g^2;
 *     p -= lr * (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps),      t = 1, 2, ...
 */
void orc_adam_step(double* p, const double* g, double* m, double* v, int64_t n, int64_t t,
                   double lr, double b1, double b2, double eps) {
    const double c1 = 1.0 - pow(b1, (double)t), c2 = 1.0 - pow(b2, (double)t);
    for (int64_t i = 0; i < n; ++i) {
        m[i] = b1 * m[i] + (1.0 - b1) * g[i];
        v[i] = b2 * v[i] + (1.0 - b2) * g[i] * g[i];
        p[i] -= lr * (m[i] / c1) / (sqrt(v[i] / c2) + eps);
    }
}

/*
 * The same optimiser for an embedding table whose gradient is sparse (event 4,
 * "push gradients of Sparse Part"): G[id] = sum over the views b (ascending)
 * with ids[b] == id of dX[b][col0 .. col0+E); every row that received a
 * gradient takes one Adam step with its own moment rows m[id], v[id] and the
 * global step count t; rows without a gradient, and their moments, stay as they
 * are.  table in its storage type; m, v doubles [vocab][E].  Returns the
 * number of out-of-range IDs (skipped).
 */
int64_t orc_emb_adam(void* table, int dt, double* m, double* v, int64_t vocab, int32_t E,
                     const int32_t* ids, int32_t B, const double* dX, int32_t ldx, int32_t col0,
                     int64_t t, double lr, double b1, double b2, double eps) {
    int64_t bad = 0;
    double* G = (double*)calloc((size_t)vocab * E, sizeof(double));
    uint8_t* seen = (uint8_t*)calloc((size_t)vocab, 1);
    for (int32_t b = 0; b < B; ++b) {
        int32_t id = ids[b];
        if (id < 0 || id >= vocab) { ++bad; continue; }
        seen[id] = 1;
        for (int c = 0; c < E; ++c) G[(int64_t)id * E + c] += dX[(int64_t)b * ldx + col0 + c];
    }
    double* row = (double*)malloc(sizeof(double) * E);
    for (int64_t id = 0; id < vocab; ++id) {
        if (!seen[id]) continue;
        for (int c = 0; c < E; ++c) row[c] = load_elem(table, dt, id * E + c);
        orc_adam_step(row, G + id * E, m + id * E, v + id * E, E, t, lr, b1, b2, eps);
        for (int c = 0; c < E; ++c) store_elem(table, dt, id * E + c, row[c]);
    }
    free(row); free(G); free(seen);
    return bad;
}
