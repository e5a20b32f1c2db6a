/*
 * CPU oracle for the speculative-decoding verify path.  TEST INFRASTRUCTURE ONLY:
 * the product never calls this file; it shares no source with the CUDA path.
 *
 * It is a plain fp32 decoder-only transformer forward (pre-norm RMSNorm, rotary
 * position embedding in the rotate-half pairing, grouped-query attention, SwiGLU
 * feed-forward) plus the integer steps of retrieval-based greedy speculative
 * decoding: the n-gram suffix drafter over the request context and the strict
 * longest-matching-prefix acceptance.
 *
 * What it follows in the paper:
 *   - Draft-then-verify with strict acceptance (Sec. 3.2, "Breakdown of SD
 *     inefficiency" and Sec. 4.4 "Empirical analysis of reuse opportunities"):
 *     the target model runs once over [T, x_1..x_n] and yields y_1..y_{n+1};
 *     drafts are kept up to the first x_e != y_e; the emitted tokens are
 *     x_1..x_{e-1}, y_e.
 *   - Drafting from the request context by suffix matching (Sec. 3.2 and
 *     Sec. 5.5: the PLD drafter uses the current context only).
 *   - Chunked prefill with fixed-size chunks (Sec. 4.1, Sec. 4.2 graph
 *     equivalence): running short pieces one after another equals one long run.
 *   - Model family (Sec. 5.1 "Models"): Qwen2.5 / LLaMA-3.2 style decoders.
 *
 * Arithmetic: every floating-point value is fp32; every sum runs over its index
 * in ascending order into a single accumulator, so a row's result does not
 * depend on how many other rows are processed in the same call.  Weights are the
 * bf16 values handed in as bit patterns, widened exactly to fp32.
 *
 * Pinned by tests/test_oracle_*.py (fp64 restatements on tiny shapes, closed
 * forms, brute-force search, the lossless-decoding invariant).  The numerical
 * values of full-model logits have no value printed in the paper to compare
 * with: "parity unpinned" beyond those checks.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab, max_seq;
    int tied_lm_head, qkv_bias;
    float rope_theta, rms_eps;
} orc_config;

typedef struct {
    const uint16_t *wq, *wk, *wv, *wo, *wg, *wu, *wd; /* bf16 bits, [out][in] row-major */
    const float *norm1, *norm2;                       /* [d] */
    const float *bq, *bk, *bv;                        /* NULL unless qkv_bias */
} orc_layer;

typedef struct {
    const uint16_t *emb;      /* [V][d] */
    const uint16_t *lm_head;  /* [V][d]; NULL when tied */
    const float *final_norm;  /* [d] */
    const orc_layer *layers;  /* [n_layers] */
} orc_weights;

static inline float bf16_to_f32(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

/* Rows of x are handled MB at a time, and rows of w four at a time, purely so that the loop
 * over rows of x is the contiguous, vectorisable one and four independent sums are in flight;
 * each output still has its own accumulator summed over k ascending. */
#define NB 4
#define DEF_MATMUL(NAME, MB)                                                                              \
    static void NAME(const float *xt, const uint16_t *w, const float *bias, float *y, int M, int N, int K, \
                     int Mp) {                                                                            \
        _Pragma("omp parallel for schedule(static)") for (int n0 = 0; n0 < N; n0 += NB) {                 \
            const int nb = N - n0 < NB ? N - n0 : NB;                                                     \
            const uint16_t *wr[NB];                                                                       \
            for (int r = 0; r < NB; ++r) wr[r] = w + (size_t)(n0 + (r < nb ? r : 0)) * K;                 \
            for (int m0 = 0; m0 < Mp; m0 += MB) {                                                         \
                float acc[NB][MB];                                                                        \
                for (int r = 0; r < NB; ++r)                                                              \
                    for (int j = 0; j < MB; ++j) acc[r][j] = 0.0f;                                        \
                for (int k = 0; k < K; ++k) {                                                             \
                    const float *xr = xt + (size_t)k * Mp + m0;                                           \
                    for (int r = 0; r < NB; ++r) {                                                        \
                        const float wv = bf16_to_f32(wr[r][k]);                                           \
                        for (int j = 0; j < MB; ++j) acc[r][j] += wv * xr[j];                             \
                    }                                                                                     \
                }                                                                                         \
                for (int r = 0; r < nb; ++r)                                                              \
                    for (int j = 0; j < MB && m0 + j < M; ++j)                                            \
                        y[(size_t)(m0 + j) * N + n0 + r] = acc[r][j] + (bias ? bias[n0 + r] : 0.0f);      \
            }                                                                                             \
        }                                                                                                 \
    }
DEF_MATMUL(matmul_mb16, 16)
DEF_MATMUL(matmul_mb64, 64)

/* The definition written out: y[m][n] = sum_k x[m][k] * w[n][k]  (+ bias[n]), one accumulator per
 * output, k ascending; no blocking, no transposition, no threads.  orc_matmul below must equal it
 * bit for bit (tests/test_oracle_ops.py); it exists so that the arithmetic can be checked by eye. */
void orc_matmul_plain(const float *x, const uint16_t *w, const float *bias, float *y, int M, int N, int K) {
    for (int m = 0; m < M; ++m)
        for (int n = 0; n < N; ++n) {
            float acc = 0.0f;
            for (int k = 0; k < K; ++k) acc += bf16_to_f32(w[(size_t)n * K + k]) * x[(size_t)m * K + k];
            y[(size_t)m * N + n] = acc + (bias ? bias[n] : 0.0f);
        }
}

/* The same sums as orc_matmul_plain, arranged for speed (the full-size workloads need it).
 * y[m][n] = sum_k x[m][k] * w[n][k]  (+ bias[n]).  One accumulator per output, k ascending. */
void orc_matmul(const float *x, const uint16_t *w, const float *bias, float *y, int M, int N, int K) {
    const int MB = M > 32 ? 64 : 16;
    const int Mp = (M + MB - 1) / MB * MB;
    /* x transposed to [K][Mp] so the loop over rows of x is the contiguous one */
    float *xt = (float *)calloc((size_t)K * Mp, sizeof(float));
    for (int m = 0; m < M; ++m)
        for (int k = 0; k < K; ++k) xt[(size_t)k * Mp + m] = x[(size_t)m * K + k];
    if (MB == 64) matmul_mb64(xt, w, bias, y, M, N, K, Mp);
    else matmul_mb16(xt, w, bias, y, M, N, K, Mp);
    free(xt);
}

/* y = x * rsqrt(mean(x^2) + eps) * w, one row */
void orc_rmsnorm(const float *x, const float *w, float eps, float *y, int d) {
    float ss = 0.0f;
    for (int i = 0; i < d; ++i) ss += x[i] * x[i];
    const float r = 1.0f / sqrtf(ss / (float)d + eps);
    for (int i = 0; i < d; ++i) y[i] = x[i] * r * w[i];
}

/* Rotary embedding of one head vector at absolute position pos, pairing (i, i + hd/2),
 * angle pos * theta^(-2i/hd) evaluated in double. */
void orc_rope(float *v, int hd, int pos, float theta) {
    const int h = hd / 2;
    for (int i = 0; i < h; ++i) {
        const double ang = (double)pos * pow((double)theta, -2.0 * (double)i / (double)hd);
        const float c = (float)cos(ang), s = (float)sin(ang);
        const float a = v[i], b = v[i + h];
        v[i] = a * c - b * s;
        v[i + h] = b * c + a * s;
    }
}

/* Softmax attention of one query vector over keys 0..n_keys-1 (rows of k, v with stride hd). */
void orc_attention_row(const float *q, const float *k, const float *v, int n_keys, int hd, float *out,
                       float *scratch /* [n_keys] */) {
    const float scale = 1.0f / sqrtf((float)hd);
    float mx = -INFINITY;
    for (int t = 0; t < n_keys; ++t) {
        float s = 0.0f;
        for (int i = 0; i < hd; ++i) s += q[i] * k[(size_t)t * hd + i];
        s *= scale;
        scratch[t] = s;
        if (s > mx) mx = s;
    }
    float l = 0.0f;
    for (int t = 0; t < n_keys; ++t) {
        scratch[t] = expf(scratch[t] - mx);
        l += scratch[t];
    }
    for (int i = 0; i < hd; ++i) out[i] = 0.0f;
    for (int t = 0; t < n_keys; ++t) {
        const float p = scratch[t] / l;
        for (int i = 0; i < hd; ++i) out[i] += p * v[(size_t)t * hd + i];
    }
}

/* act = silu(g) * u */
void orc_swiglu(const float *g, const float *u, float *act, int n) {
    for (int i = 0; i < n; ++i) act[i] = (g[i] / (1.0f + expf(-g[i]))) * u[i];
}

/* Greedy choice: the largest value; among equal values the lowest index; NaN never wins. */
int orc_argmax(const float *x, int n) {
    int best = 0;
    float bv = -INFINITY;
    for (int i = 0; i < n; ++i)
        if (x[i] > bv) { bv = x[i]; best = i; }
    return best;
}

/*
 * Tree-structured drafts (paper Sec. 4.1 "Speculative decoding": drafts are trees, verified in one
 * pass): with parent != NULL token row j (j >= 1) continues row parent[j] < j (row 0 is the root, the
 * committed token).  Row j then sits at absolute position start_pos + depth(j), its K/V rows are
 * written at cache slot start_pos + j, and it attends to cache rows 0 .. start_pos-1 and to the rows
 * on its own path from the root (itself included), in that order.  parent == NULL is the linear
 * chain parent[j] = j-1, for which all of this reduces to the description below.
 *
 * Run the decoder over m tokens at absolute positions start_pos .. start_pos+m-1.
 * kcache/vcache: fp32 [layer][kv_head][max_seq][hd]; rows start_pos.. are written, rows
 * below start_pos are read.  Token row j attends to positions 0 .. start_pos+j.
 * logits: [m - logits_from][vocab] for rows logits_from..m-1 (NULL: skip the LM head).
 * hidden_out (optional): [m][d] residual stream after the last layer (before the final norm).
 * Returns 0, or -1 on a bad argument.
 */
int orc_forward_tree(const orc_config *c, const orc_weights *w, const int32_t *tokens, const int32_t *parent, int m,
                     int start_pos, float *kcache, float *vcache, float *logits, int logits_from, float *hidden_out) {
    const int d = c->d_model, hd = c->head_dim, nq = c->n_q_heads, nkv = c->n_kv_heads, f = c->d_ffn;
    const int g = nq / nkv, Nq = nq * hd, Nkv = nkv * hd;
    if (m <= 0 || start_pos < 0 || start_pos + m > c->max_seq) return -1;
    for (int j = 0; j < m; ++j)
        if (tokens[j] < 0 || tokens[j] >= c->vocab) return -1;
    int *depth = (int *)malloc(sizeof(int) * (size_t)m);
    for (int j = 0; j < m; ++j) {
        if (!parent) depth[j] = j;
        else if (j == 0) depth[j] = 0;
        else if (parent[j] < 0 || parent[j] >= j) { free(depth); return -1; }
        else depth[j] = depth[parent[j]] + 1;
    }

    float *h = (float *)malloc(sizeof(float) * (size_t)m * d);
    float *xn = (float *)malloc(sizeof(float) * (size_t)m * d);
    float *q = (float *)malloc(sizeof(float) * (size_t)m * Nq);
    float *kk = (float *)malloc(sizeof(float) * (size_t)m * Nkv);
    float *vv = (float *)malloc(sizeof(float) * (size_t)m * Nkv);
    float *o = (float *)malloc(sizeof(float) * (size_t)m * Nq);
    float *t1 = (float *)malloc(sizeof(float) * (size_t)m * d);
    float *gt = (float *)malloc(sizeof(float) * (size_t)m * f);
    float *up = (float *)malloc(sizeof(float) * (size_t)m * f);
    float *act = (float *)malloc(sizeof(float) * (size_t)m * f);

    for (int j = 0; j < m; ++j)
        for (int i = 0; i < d; ++i) h[(size_t)j * d + i] = bf16_to_f32(w->emb[(size_t)tokens[j] * d + i]);

    for (int l = 0; l < c->n_layers; ++l) {
        const orc_layer *L = &w->layers[l];
        float *kc = kcache + (size_t)l * nkv * c->max_seq * hd;
        float *vc = vcache + (size_t)l * nkv * c->max_seq * hd;
        for (int j = 0; j < m; ++j) orc_rmsnorm(h + (size_t)j * d, L->norm1, c->rms_eps, xn + (size_t)j * d, d);
        orc_matmul(xn, L->wq, c->qkv_bias ? L->bq : NULL, q, m, Nq, d);
        orc_matmul(xn, L->wk, c->qkv_bias ? L->bk : NULL, kk, m, Nkv, d);
        orc_matmul(xn, L->wv, c->qkv_bias ? L->bv : NULL, vv, m, Nkv, d);
        for (int j = 0; j < m; ++j) {
            const int pos = start_pos + depth[j]; /* rotary position */
            const int slot = start_pos + j;       /* cache row */
            for (int a = 0; a < nq; ++a) orc_rope(q + (size_t)j * Nq + a * hd, hd, pos, c->rope_theta);
            for (int a = 0; a < nkv; ++a) {
                orc_rope(kk + (size_t)j * Nkv + a * hd, hd, pos, c->rope_theta);
                memcpy(kc + ((size_t)a * c->max_seq + slot) * hd, kk + (size_t)j * Nkv + a * hd, sizeof(float) * hd);
                memcpy(vc + ((size_t)a * c->max_seq + slot) * hd, vv + (size_t)j * Nkv + a * hd, sizeof(float) * hd);
            }
        }
#pragma omp parallel
        {
            float *scr = (float *)malloc(sizeof(float) * (size_t)(start_pos + m));
            /* tree: the keys and values a row sees, gathered in order (cache rows, then its path from the root) */
            float *kg = parent ? (float *)malloc(sizeof(float) * (size_t)(start_pos + m) * hd) : NULL;
            float *vg = parent ? (float *)malloc(sizeof(float) * (size_t)(start_pos + m) * hd) : NULL;
            int *path = parent ? (int *)malloc(sizeof(int) * (size_t)m) : NULL;
#pragma omp for collapse(2) schedule(dynamic, 1)
            for (int j = 0; j < m; ++j)
                for (int a = 0; a < nq; ++a) {
                    const int kvh = a / g;
                    const float *kh = kc + (size_t)kvh * c->max_seq * hd, *vh = vc + (size_t)kvh * c->max_seq * hd;
                    if (!parent) {
                        orc_attention_row(q + (size_t)j * Nq + a * hd, kh, vh, start_pos + j + 1, hd,
                                          o + (size_t)j * Nq + a * hd, scr);
                    } else {
                        const int np = depth[j] + 1;
                        for (int r = j, i = np - 1; i >= 0; --i, r = (r > 0 ? parent[r] : 0)) path[i] = r;
                        memcpy(kg, kh, sizeof(float) * (size_t)start_pos * hd);
                        memcpy(vg, vh, sizeof(float) * (size_t)start_pos * hd);
                        for (int i = 0; i < np; ++i) {
                            memcpy(kg + (size_t)(start_pos + i) * hd, kh + (size_t)(start_pos + path[i]) * hd, sizeof(float) * hd);
                            memcpy(vg + (size_t)(start_pos + i) * hd, vh + (size_t)(start_pos + path[i]) * hd, sizeof(float) * hd);
                        }
                        orc_attention_row(q + (size_t)j * Nq + a * hd, kg, vg, start_pos + np, hd,
                                          o + (size_t)j * Nq + a * hd, scr);
                    }
                }
            free(scr); free(kg); free(vg); free(path);
        }
        orc_matmul(o, L->wo, NULL, t1, m, d, Nq);
        for (size_t i = 0; i < (size_t)m * d; ++i) h[i] += t1[i];
        for (int j = 0; j < m; ++j) orc_rmsnorm(h + (size_t)j * d, L->norm2, c->rms_eps, xn + (size_t)j * d, d);
        orc_matmul(xn, L->wg, NULL, gt, m, f, d);
        orc_matmul(xn, L->wu, NULL, up, m, f, d);
        orc_swiglu(gt, up, act, m * f);
        orc_matmul(act, L->wd, NULL, t1, m, d, f);
        for (size_t i = 0; i < (size_t)m * d; ++i) h[i] += t1[i];
    }
    if (hidden_out) memcpy(hidden_out, h, sizeof(float) * (size_t)m * d);
    if (logits && logits_from < m) {
        if (logits_from < 0) logits_from = 0;
        const int r = m - logits_from;
        for (int j = 0; j < r; ++j)
            orc_rmsnorm(h + (size_t)(logits_from + j) * d, w->final_norm, c->rms_eps, xn + (size_t)j * d, d);
        orc_matmul(xn, c->tied_lm_head ? w->emb : w->lm_head, NULL, logits, r, c->vocab, d);
    }
    free(h); free(xn); free(q); free(kk); free(vv); free(o); free(t1); free(gt); free(up); free(act); free(depth);
    return 0;
}

/* The linear chain: row j continues row j-1 (Sec. 3.2, the drafts of one retrieval are checked in one pass). */
int orc_forward(const orc_config *c, const orc_weights *w, const int32_t *tokens, int m, int start_pos,
                float *kcache, float *vcache, float *logits, int logits_from, float *hidden_out) {
    return orc_forward_tree(c, w, tokens, NULL, m, start_pos, kcache, vcache, logits, logits_from, hidden_out);
}

/*
 * Retrieval drafter: suffix match of the token history against a search array.
 * For every position p with a continuation (p+1 < n_search), m(p) is the length of the
 * longest common suffix of search[0..p] and hist[0..hist_len-1], capped at n, p+1 and
 * hist_len.  Positions with m(p) >= n_min are candidates; the winner maximises (m(p), p):
 * the longest match, and among equally long ones the latest.  The draft is the up-to-k
 * tokens that follow the winner.  Returns the draft length (0 when nothing matches).
 * exclude_from: positions p >= exclude_from are skipped (used when the search array is the
 * history itself, so that the suffix does not match itself); pass n_search otherwise.
 */
int orc_ngram_draft(const int32_t *search, int n_search, const int32_t *hist, int hist_len, int n, int n_min,
                    int k, int exclude_from, int32_t *draft, int *match_pos, int *match_len) {
    int best_m = 0, best_p = -1;
    for (int p = 0; p + 1 < n_search && p < exclude_from; ++p) {
        int cap = n;
        if (p + 1 < cap) cap = p + 1;
        if (hist_len < cap) cap = hist_len;
        int mlen = 0;
        while (mlen < cap && search[p - mlen] == hist[hist_len - 1 - mlen]) ++mlen;
        if (mlen >= n_min && mlen > 0 && (mlen > best_m || (mlen == best_m && p > best_p))) {
            best_m = mlen;
            best_p = p;
        }
    }
    if (match_pos) *match_pos = best_p;
    if (match_len) *match_len = best_m;
    if (best_p < 0) return 0;
    int dl = 0;
    for (int i = best_p + 1; i < n_search && dl < k; ++i) draft[dl++] = search[i];
    return dl;
}

/* Strict acceptance: the number of leading drafts x_i (i = 1..draft_len) equal to the model's
 * prediction y_i; y has draft_len + 1 entries. */
int orc_accept_len(const int32_t *x, const int32_t *y, int draft_len) {
    int a = 0;
    while (a < draft_len && x[a] == y[a]) ++a;
    return a;
}
