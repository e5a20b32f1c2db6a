/*
 * sdv — speculative-decoding verify path on one NVIDIA B200 (sm_100a).
 *
 * One sdv_ctx holds one sequence: the model weights (re-laid out for streaming), a bf16 KV
 * cache with a committed length L, the token history (request context followed by generated
 * tokens) and a small device-resident state block.  The calls follow the online workflow of
 * the paper (Sec. 4.1): chunked prefill of the request context, then repeatedly draft ->
 * verify -> accept/commit.
 *
 * Conventions
 *   - Every function returns an int status: SDV_OK (0) or a negative SDV_E* code.  Nothing
 *     throws, aborts or prints.  sdv_strerror() names a code; sdv_last_cuda_error() gives the
 *     CUDA runtime code behind the last SDV_ECUDA.
 *   - "host" pointers are ordinary CPU memory; "dev" pointers are CUDA device memory on the
 *     current device.  The caller owns every buffer it passes in, including the workspace,
 *     which must outlive the context and be 256-byte aligned.
 *   - All GPU work is ordered on the stream given to sdv_create (a cudaStream_t passed as
 *     void*; NULL = the legacy default stream).  Calls that hand values back to the host
 *     synchronise that stream; calls given NULL output pointers do not.
 *   - A context is not thread-safe.  There is no CPU fallback: without a usable CUDA device
 *     every call that would launch work returns SDV_ECUDA.
 */
#ifndef SDV_H_
#define SDV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    SDV_OK = 0,
    SDV_EINVAL = -1,    /* bad argument or unsupported shape */
    SDV_ENOMEM = -2,    /* workspace too small */
    SDV_ECAPACITY = -3, /* KV cache / history would exceed max_seq */
    SDV_ESTATE = -4,    /* call order: e.g. verify before prefill finished, commit without verify */
    SDV_ECUDA = -5,     /* CUDA runtime error, see sdv_last_cuda_error() */
    SDV_ETIMEOUT = -6,  /* a bounded device-side wait ran out; the context must be re-created */
    SDV_ETOOBIG = -7    /* sdv_gemm_noalloc: the problem exceeds its fixed scratch area */
};

#define SDV_NGRAM_MAX 4096 /* longest history suffix the drafter can be asked to match */
#define SDV_K_MAX 31 /* longest draft per verify step (M = k+1 <= 32 rows) */
#define SDV_CALIB_MAX 4 /* most successors sampled per context position by the calibration */

typedef struct sdv_ctx sdv_ctx;

/* Model shape and drafter settings.  Supported: head_dim 64 or 128; d_model and d_ffn multiples
 * of 64; vocab a multiple of 16; n_q_heads a multiple of n_kv_heads with at most 8 query heads
 * per KV head; 1 <= k_max <= SDV_K_MAX, further limited by shared memory (the k_max + 1 token rows
 * of d_model columns must fit next to the weight ring: sdv_create returns SDV_EINVAL otherwise);
 * 1 <= ngram_min <= ngram_n <= SDV_NGRAM_MAX.  ngram_n = SDV_NGRAM_MAX with search_history = 1 is
 * longest-suffix retrieval over the request context and the generated tokens: the match a suffix
 * automaton over that text returns (the retrieval algorithm the paper's baselines use, Sec. 5.1 (3)),
 * found here by a parallel scan of all end positions instead of an automaton. */
typedef struct {
    int n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
    int max_seq;        /* KV rows / history entries the context can hold */
    int k_max;          /* largest draft length that will be verified */
    int tied_lm_head;   /* LM head shares the embedding matrix */
    int qkv_bias;       /* q, k, v projections carry a bias */
    int ngram_n;        /* longest history suffix the drafter tries to match */
    int ngram_min;      /* shortest suffix match that still yields a draft */
    int search_history; /* 0: drafter searches the request context only; 1: context + generated tokens */
    float rope_theta, rms_eps;
} sdv_config;

/* Weights as the caller holds them: bf16 bit patterns, row-major [out_features][in_features]
 * (matrices) and fp32 vectors.  Pointers may be host or device memory.  Biases are read only
 * when qkv_bias is set; lm_head is read only when tied_lm_head is 0. */
typedef struct {
    const uint16_t *wq, *wk, *wv; /* [n_q*hd][d], [n_kv*hd][d], [n_kv*hd][d] */
    const uint16_t *wo;           /* [d][n_q*hd] */
    const uint16_t *wg, *wu;      /* [f][d] */
    const uint16_t *wd;           /* [d][f] */
    const float *norm1, *norm2;   /* [d] RMSNorm scales before attention / before the FFN */
    const float *bq, *bk, *bv;    /* [n_q*hd], [n_kv*hd], [n_kv*hd] or NULL */
} sdv_layer_weights;

typedef struct {
    const uint16_t *emb;             /* [vocab][d] */
    const uint16_t *lm_head;         /* [vocab][d] or NULL when tied */
    const float *final_norm;         /* [d] */
    const sdv_layer_weights *layers; /* [n_layers] */
} sdv_weights;

/* Bytes of device workspace sdv_create needs for this configuration (0 if it is invalid). */
size_t sdv_workspace_bytes(const sdv_config *cfg);

/* Creates a context inside caller-provided device memory (dev_workspace, bytes).  The context
 * keeps the pointer; it allocates only a small host structure and a pinned host staging page.
 * Errors: SDV_EINVAL (shape), SDV_ENOMEM (bytes too small), SDV_ECUDA. */
int sdv_create(const sdv_config *cfg, void *dev_workspace, size_t bytes, void *cuda_stream, sdv_ctx **out);

/* Copies the weights into the workspace, re-laid out in the order the kernels stream them.
 * Synchronises the stream.  May be called again to replace the weights. */
int sdv_load_weights(sdv_ctx *ctx, const sdv_weights *w);

/* Chunked prefill (paper Sec. 4.1: the prompt is cut into chunks of one fixed size; Sec. 4.2: graph
 * equivalence): appends n context tokens (host int32, each in [0, vocab)) to the history, runs
 * the decoder over them at positions L..L+n-1 and advances L by n.  Chunks of any length n >= 1
 * give the same cache as one long call.  With is_last != 0 the logits of the last token are
 * reduced to the first generated token T (greedy), which becomes the pending token and is
 * appended to the history; drafting and verification may start afterwards.  Synchronises.
 * Errors: SDV_ESTATE after the last chunk, SDV_ECAPACITY, SDV_EINVAL. */
int sdv_prefill_chunk(sdv_ctx *ctx, const int32_t *host_tokens, int n, int is_last);

/* Retrieval drafter (paper Sec. 3.2 / Sec. 5.5: drafts come from the request context by
 * matching the current suffix and copying what followed).  Finds the position p of the search
 * array whose preceding tokens share the longest suffix (at most ngram_n, at least ngram_min
 * tokens) with the history, preferring the latest among equally long matches, and copies up to
 * k tokens after p into the device draft buffer.  host_draft (k ints) and draft_len may be NULL;
 * if either is given the stream is synchronised.  draft_len may be less than k, or 0. */
int sdv_draft(sdv_ctx *ctx, int k, int32_t *host_draft, int *draft_len);

/* Extra token database for the drafter (paper Sec. 5.1 (3), Sec. 5.5: the retrieval algorithm of
 * the baselines searches the request context and an additional token corpus).  Copies n host tokens
 * (0 <= n <= max_seq; 0 removes the database) into the context; sdv_draft then searches them like
 * the request's text and copies the draft from wherever the longer suffix match ends (an equally
 * long match in the request's own text wins).  The database survives prefill and rollback.
 * Synchronises.  Errors: SDV_EINVAL (count, token range). */
int sdv_set_database(sdv_ctx *ctx, const int32_t *host_tokens, int n);

/* Verify step (paper Sec. 3.2: all drafts are checked in one parallel pass; Sec. 4.4: x = [T, x_1..x_n],
 * y = [y_1..y_{n+1}]): runs the decoder once over the pending token T and the drafts at
 * positions L..L+n, writing their KV rows speculatively, takes the greedy token y_{j+1} of
 * every row (lowest id wins ties) and the accept length a = number of leading x_i == y_i.
 * host_draft != NULL: verify these draft_len tokens (0 <= draft_len <= k_max).
 * host_draft == NULL: verify the draft left by the last sdv_draft (draft_len is ignored; k+1
 *   rows are computed, rows past the drafter's own draft length are padding and never accepted).
 * host_y (draft_len+1 ints; k_max+1 is always enough) and accept_len may be NULL; if either is
 * given the stream is synchronised.  Nothing is committed: L, T and the history are unchanged.
 * Errors: SDV_ESTATE before prefill has finished, SDV_ECAPACITY, SDV_EINVAL, SDV_ETIMEOUT. */
int sdv_verify(sdv_ctx *ctx, const int32_t *host_draft, int draft_len, int32_t *host_y, int *accept_len);

/* One whole step in one call with one synchronisation (paper Sec. 4.1: verify, accept, then the next draft):
 * verify host_draft (draft_len tokens, as sdv_verify; NULL: the draft on the device, left by sdv_draft or by
 * the previous sdv_step), accept, commit, and, when k_next > 0, draft k_next tokens for the next step as
 * sdv_draft would; accept scan, commit and draft are one launch behind the forward kernel.  The emitted tokens
 * (host_emitted: k_max + 1 ints are always enough), their number, the new KV length and the next draft
 * (host_next_draft: k_next ints; next_draft_len may be less than k_next, or 0) come back in one copy of the state
 * block; any of the output pointers may be NULL.  Synchronises.  The retained segment of the draft extension is
 * not updated by this call.  Errors: SDV_EINVAL, SDV_ESTATE (before the end of prefill; a tree draft pending),
 * SDV_ECAPACITY, SDV_ETIMEOUT. */
int sdv_step(sdv_ctx *ctx, const int32_t *host_draft, int draft_len, int k_next, int32_t *host_emitted,
             int *n_emitted, int32_t *host_next_draft, int *next_draft_len, int *kv_len);

/* A run of decoding steps without the host in between (paper Sec. 4.1, online workflow: draft -> verify ->
 * accept repeated until the answer ends).  Enqueues n_steps (1..4096) steps of sdv_draft(k) [+
 * sdv_extend_draft(ext_max_total) when ext_max_total > 0] -> sdv_verify -> [sdv_extension_update(ext_max_life)]
 * -> sdv_commit on the context's stream; every kernel takes the KV length, history and drafts from the
 * device state the step before left, so nothing is read back until the run ends.  Each verify computes
 * k + 1 rows (ext_max_total + 1 with the extension; k <= ext_max_total <= k_max); between two forward kernels one
 * launch does the accept scan, the commit and the next draft.  max_tokens > 0 ends the
 * run after that many emitted tokens: the step that reaches it is cut like sdv_commit's max_emit and the
 * steps enqueued behind it do nothing (they cost a few microseconds each); max_tokens <= 0: no limit.
 * The emitted tokens equal those of the same calls made one by one.  host_tokens (room for
 * min(max_tokens, n_steps * rows) ints), n_tokens and kv_len may be NULL.  Synchronises once, at the end.
 * Errors: SDV_EINVAL, SDV_ESTATE (before the end of prefill), SDV_ECAPACITY (n_steps * rows positions
 * must fit behind the current KV length and history), SDV_ETIMEOUT.
 *
 * sdv_run_kernel_ms: device times in milliseconds of the first n forward kernels of the last run (CUDA
 * events; a step enqueued behind the run's end shows a few microseconds).  Errors: SDV_ESTATE without a run
 * of at least n steps. */
int sdv_decode_steps(sdv_ctx *ctx, int k, int n_steps, int max_tokens, int ext_max_total, int ext_max_life,
                     int32_t *host_tokens, int *n_tokens, int *kv_len);
int sdv_run_kernel_ms(sdv_ctx *ctx, float *host_ms, int n);

/* Batched verify: several sequences share one pass over the weights.  The paper verifies one request at
 * a time; its utilisation argument (Sec. 2: the matrix units need a large batch or a long sequence per
 * weight read) is what this call applies across requests, and every sequence's result is what sdv_verify
 * on that sequence alone computes.
 *
 * sdv_follower_workspace_bytes / sdv_create_follower: a further sequence that reads `leader`'s weights
 * (the leader owns its weights, has loaded them and must outlive its followers).  The follower has the
 * leader's configuration and stream, its own KV cache, history and state in dev_workspace (256-byte
 * aligned, at least sdv_follower_workspace_bytes(cfg) bytes, owned by the caller), and takes every call
 * except sdv_load_weights and sdv_debug_gemm (SDV_ESTATE).  Errors: SDV_EINVAL (NULL, a leader that is
 * itself a follower, alignment), SDV_ESTATE (leader without weights), SDV_ENOMEM, SDV_ECUDA.
 *
 * sdv_verify_batch: one verify step over ctxs[0..n) (1 <= n <= 8, distinct, a leader and followers of it
 * or followers of one leader).  Each sequence contributes the rows sdv_verify(ctx, NULL, ...) would
 * compute for it: its pending token and, after sdv_draft / sdv_extend_draft, its chain draft (k + 1 rows);
 * the rows of all sequences together may not exceed 32.  The decoder runs once over all rows, every row
 * attending to its own sequence's KV cache and earlier rows only, each sequence's KV rows are written
 * speculatively into its own cache, and the accept scan runs per sequence; afterwards every context
 * is in the state sdv_verify leaves it in (sdv_commit, sdv_extension_update, sdv_get_logits per context).
 * The step runs on the scratch buffers of ctxs[0], whose sdv_last_verify_ms then times it.
 * accept_len (n ints) may be NULL; if given the stream is synchronised.
 * Errors: SDV_EINVAL (count, duplicates, unrelated contexts, more than 32 rows), SDV_ESTATE (a sequence
 * before the end of prefill, or with a tree draft pending), SDV_ECAPACITY, SDV_ETIMEOUT. */
/* Result of the outstanding verify step of one context (after sdv_verify, sdv_verify_tree or
 * sdv_verify_batch, before the commit): the greedy token of each of its rows into host_y (k_max + 1 ints
 * are always enough) and the accept length; either may be NULL.  Synchronises.  Errors: SDV_ESTATE when
 * no verify result is outstanding, SDV_ETIMEOUT. */
int sdv_get_verified(sdv_ctx *ctx, int32_t *host_y, int *accept_len);

size_t sdv_follower_workspace_bytes(const sdv_config *cfg);
int sdv_create_follower(sdv_ctx *leader, void *dev_workspace, size_t bytes, sdv_ctx **out);
int sdv_verify_batch(sdv_ctx *const *ctxs, int n, int *accept_len);

/* Draft extension (paper Sec. 4.4 "Reuse strategy", Eq. 3): drafts rejected by one verify step
 * are kept when they agree with the model's own predictions and are appended to later drafts.
 *
 * sdv_extend_draft: call after sdv_draft.  Appends the retained segment to the device draft when
 * the result has at most max_total tokens (1 <= max_total <= k_max; the paper's threshold is 32
 * rows); a segment that does not fit is dropped, not cut.  host_draft (max_total ints) and
 * draft_len may be NULL; if either is given the stream is synchronised and the next sdv_verify
 * computes exactly draft_len + 1 rows, otherwise it computes max_total + 1 rows (rows past the
 * draft are padding and never accepted).
 *
 * sdv_extension_update: call after sdv_verify, before sdv_commit.  Among the drafts beyond the
 * reject point e = a + 1 it finds the longest run with x_i == y_i (Eq. 3; the earliest among
 * equally long runs) and applies the retention rules: a segment that was appended ages by one
 * step; it is dropped when the accepted prefix reached into it or when its age exceeds max_life
 * (>= 1); the candidate replaces the retained segment when strictly longer.  host_segment
 * (k_max ints), segment_len and lifetime may be NULL; if any is given the stream is synchronised.
 * The segment is cleared by prefill, sdv_rollback and sdv_debug_set_history.
 * Errors: SDV_ESTATE without a pending draft / verify result, SDV_EINVAL. */
int sdv_extend_draft(sdv_ctx *ctx, int max_total, int32_t *host_draft, int *draft_len);
int sdv_extension_update(sdv_ctx *ctx, int max_life, int32_t *host_segment, int *segment_len, int *lifetime);

/* In-context distribution calibration (paper Sec. 4.3 "Workflow") and tree-structured drafts
 * (Sec. 4.1 "Speculative decoding": drafts are trees, verified in one pass).
 *
 * sdv_set_calibration: call before the first sdv_prefill_chunk.  With top_b in 1..SDV_CALIB_MAX every
 * prefill tile also runs the LM head and keeps, for each context position, the top_b token ids of
 * its logits (largest first, lowest id among equals): "Sample", the model-preferred anchors
 * <context token, prediction>.  After the last chunk each prediction is looked up in the request
 * ("Search": its latest position, -1 where it does not occur).  top_b = 0 switches it off.
 * sdv_get_calibration copies the two tables for the first n_positions context positions to the
 * host as int32 [n_positions][top_b] (either pointer may be NULL).
 *
 * sdv_draft_tree: the draft of one step as a tree with at most max_nodes (<= k_max) nodes.  The
 * retrieval drafter's chain of up to k tokens (k = 0: none) is its first path; then, with p the
 * latest position of the committed token T in the request, each sampled successor of p becomes a
 * child of the root, followed at once by the successors of the position where that anchor was
 * matched (two levels, depth first).  A token a node already has as a child is not added twice.
 * Node i (1-based) continues row host_parent[i-1] < i, row 0 being T; host_tokens / host_parent
 * (k_max ints each) and n_nodes may be NULL; if any is given the stream is synchronised and the
 * next sdv_verify_tree computes exactly n_nodes + 1 rows, else max_nodes + 1.
 *
 * sdv_verify_tree: one forward pass over [T, nodes]: node i sits at position L + depth(i), its K/V
 * rows go to cache slot L + i, and it attends to the cache and to its own path from the root.
 * host_tokens == NULL verifies the tree sdv_draft_tree left on the device.  Acceptance is strict: from
 * the root, step to the child (the lowest-numbered one) whose token equals the model's greedy
 * prediction at the current row, until no child does; the emitted tokens are the path's tokens and
 * the prediction at its last row.  host_y (n_nodes+1 ints), host_path (k_max ints: the accepted
 * rows) and path_len may be NULL.  sdv_commit then first moves the accepted rows' K/V to the
 * consecutive slots L+1.. before L advances.  A chain is the tree parent[i-1] = i-1.
 * Errors: SDV_ESTATE (order), SDV_EINVAL (a parent that is not an earlier row, token range),
 * SDV_ECAPACITY. */
int sdv_set_calibration(sdv_ctx *ctx, int top_b);
int sdv_get_calibration(sdv_ctx *ctx, int32_t *host_succ, int32_t *host_occ, int n_positions);
int sdv_draft_tree(sdv_ctx *ctx, int k, int max_nodes, int32_t *host_tokens, int32_t *host_parent, int *n_nodes);
int sdv_verify_tree(sdv_ctx *ctx, const int32_t *host_tokens, const int32_t *host_parent, int n_nodes,
                    int32_t *host_y, int32_t *host_path, int *path_len);

/* Commit / rollback (paper Sec. 3.2: tokens after the first mismatch are discarded; Sec. 4.4:
 * the accepted prefix is x_1..x_{e-1}, y_e): emits x_1..x_a, y_{a+1} of the last verify, cut to
 * max_emit tokens when max_emit > 0; appends them to the history; L += number emitted; the last
 * emitted token becomes the pending token.  KV rows beyond the new L are simply left behind.
 * host_emitted (k_max+1 ints), n_emitted and kv_len may be NULL.  Always synchronises.
 * Errors: SDV_ESTATE when no verify result is outstanding. */
int sdv_commit(sdv_ctx *ctx, int max_emit, int32_t *host_emitted, int *n_emitted, int *kv_len);

/* KV rollback (paper Sec. 3.2: everything behind the first mismatch is thrown away and computed
 * again; the cache rows stay where they are, only the committed length moves).  Sets L to
 * new_kv_len (1 <= new_kv_len <= current L): the history is cut to new_kv_len + 1 tokens and its
 * last token becomes the pending token again.  Errors: SDV_ESTATE before prefill, SDV_EINVAL. */
int sdv_rollback(sdv_ctx *ctx, int new_kv_len);

/* Current committed KV length L, or a negative error code. */
int sdv_kv_len(const sdv_ctx *ctx);

/* Parity mode: when on, every verify (and the last prefill chunk) also stores the fp32 logits of
 * all rows so that sdv_get_logits can return them.  Off by default (it adds rows x vocab x 4
 * bytes of writes per step). */
int sdv_set_parity_mode(sdv_ctx *ctx, int on);
int sdv_get_logits(sdv_ctx *ctx, float *host_logits, int rows); /* [rows][vocab] of the last verify */

/* Frees the host-side structure; never touches the workspace. */
int sdv_destroy(sdv_ctx *ctx);

const char *sdv_strerror(int code);
int sdv_last_cuda_error(const sdv_ctx *ctx);

/* Verify-step accounting: bytes a step over `rows` rows at KV length kv_len has to move once
 * (all linear weights; KV rows read + written), as defined by the shapes alone. */
int sdv_step_bytes(const sdv_ctx *ctx, int rows, int kv_len, double *weight_bytes, double *kv_bytes);

/* ---- entry points for tests and measurement ------------------------------------------------
 * They run the same device code as the calls above on caller-supplied state. */

/* Replaces the token history by hist[0..hist_len) of which the first n_ctx tokens are the request
 * context, without running the model (drafter tests).  L becomes hist_len - 1. */
int sdv_debug_set_history(sdv_ctx *ctx, const int32_t *host_hist, int hist_len, int n_ctx);

/* Plays the drafter: leaves draft_len host-given tokens as the device draft (extension tests). */
int sdv_debug_set_draft(sdv_ctx *ctx, const int32_t *host_draft, int draft_len);

/* Runs the accept scan on host-given predictions y (draft_len+1 ints) against host-given drafts
 * (host_draft == NULL: against the draft already on the device, whose length draft_len must be),
 * leaving the result where sdv_commit expects it. */
int sdv_debug_accept(sdv_ctx *ctx, const int32_t *host_draft, int draft_len, const int32_t *host_y,
                     int *accept_len);

/* Like sdv_commit, but with a caller-chosen accept length (<= draft_len of the last verify) and
 * next token: teacher forcing for step-by-step comparisons. */
int sdv_debug_force_commit(sdv_ctx *ctx, int accept_len, int32_t next_token);

/* The same after sdv_verify_tree: commits a caller-chosen accepted path (rows, ascending) and next token. */
int sdv_debug_force_commit_tree(sdv_ctx *ctx, const int32_t *host_path, int path_len, int32_t next_token);

/* Runs the calibration's top-successor kernel on caller-supplied logits rows (host fp32 [rows][vocab],
 * rows <= 32) and returns int32 [rows][top_b]: the integer part of "Sample" on its own. */
int sdv_debug_top_successors(sdv_ctx *ctx, const float *host_logits, int rows, int top_b, int32_t *host_out);

/* Copies rows [pos0, pos0+n) of one layer's key (which = 0) or value (which = 1) cache to the
 * host as fp32 [n_kv_heads][n][head_dim]. */
int sdv_debug_read_kv(sdv_ctx *ctx, int layer, int which, int pos0, int n, float *host_out);

/* Copies the residual stream of the last forward pass, fp32 [rows][d_model]. */
int sdv_debug_read_hidden(sdv_ctx *ctx, int rows, float *host_out);

/* Y[M][N] = X[M][K] * W[N][K]^T with the verify path's weight-streaming GEMM (bf16 operands, fp32
 * accumulate).  host_x fp32 [M][K] (rounded to bf16 on the way in), host_w bf16 bits [N][K],
 * host_y fp32 [M][N]; M <= 32, N % 16 == 0, K % 64 == 0, K <= max(d_model, d_ffn, n_q*hd) and
 * N*K*2 bytes no larger than max(64 MiB, one layer's gate+up matrices).  dev_ms (optional)
 * receives the kernel's device time in milliseconds. */
int sdv_debug_gemm(sdv_ctx *ctx, const float *host_x, const uint16_t *host_w, float *host_y, int M, int N, int K,
                   float *dev_ms);

/* Launches a one-thread kernel that waits, with a limit of a few milliseconds, on a flag nothing
 * ever sets; returns SDV_ETIMEOUT when the bounded wait reported its expiry as designed (the
 * context stays usable), SDV_OK if the wait wrongly succeeded. */
int sdv_debug_timeout_probe(sdv_ctx *ctx);

/* Per-phase timing of the forward kernel.  host_out != NULL: copies what the last profiled launch
 * recorded, uint64 [n_phases][blocks][12] per thread block (phase 0 = embedding, then 4 per layer:
 * qkv, attention, o, gate|up + down; last = LM head).  Words 0, 1: phase work begin and end
 * (nanoseconds of the global timer).  GEMM phases: 2 token operand built, 3 last tensor-core
 * instruction issued, 4 epilogue done, 5 / 6 wait for the SwiGLU operand begins / ends (gate|up +
 * down only), 10 last accumulator seen complete by the epilogue (nanoseconds); 7, 8, 9 cycles the
 * tensor-core warp waited for weights, waited for a free accumulator, and spent in its loop.
 * Attention phase: 2 unit begins, 3 query tile built, 4 first key block in place, 5 key loop done,
 * 6 unit done, 7 whether the unit was a new-rows unit.  Then switches recording on or off for
 * later launches (it adds a block-wide barrier per phase, so timed runs keep it off).  Returns the
 * number of thread blocks, or an error. */
int sdv_debug_profile(sdv_ctx *ctx, int on, unsigned long long *host_out, int n_phases);

/* Host-only self-check of the weight streaming layout (no GPU needed): walks every thread block's
 * share of an operation the way the kernel does and checks that every 16-byte unit of the matrix
 * is met exactly once at the offset the packing step writes it to.  desc and gu_desc are
 * {row tiles, column steps, row partitions, column partitions, tiles per pass, steps per stage,
 * row granularity, follow flag}; gu_desc (the gate|up operation) is only read when the follow flag
 * of desc is set.  Returns SDV_OK, SDV_EINVAL for a malformed description, or a code <= -100. */
int sdv_debug_layout_check(const int *desc, const int *gu_desc, int n_blocks);

/* Host-only: the work partition and the shared-memory plan a context of this configuration uses
 * with n_blocks thread blocks and `rows` token rows.  out[8 * op + 0..7] as in
 * sdv_debug_layout_check for QKV, O, gate|up, down, LM head; out[40..45] = row groups of the token
 * operand, N of the tensor-core instruction, ring slots, operand region bytes, dynamic shared
 * memory bytes, 1 if the plan fits. */
int sdv_debug_plan(const sdv_config *cfg, int n_blocks, int rows, int *out);

/* Number of kernels launched by this context since creation. */
long long sdv_launch_count(const sdv_ctx *ctx);

/* Device time in milliseconds of the last forward kernel launched by sdv_verify (CUDA events on
 * the context's stream; synchronises on the closing event). */
int sdv_last_verify_ms(sdv_ctx *ctx, float *ms);

/* The same GEMM as sdv_debug_gemm, Y[M][N] = X[M][K] * W[N][K]^T (operands rounded to bf16, fp32
 * accumulate), for callers that may not allocate.  The paper has no counterpart: this is a
 * library convenience.  It needs no context and asks the CUDA runtime for no memory at any point,
 * so it can be used where an allocation is unwelcome or impossible: inside a serving loop whose
 * memory is fully handed out to the KV cache, from a plug-in that was given a fixed budget, or at
 * a point where the implicit device synchronisation of cudaMalloc / cudaFree would stall other
 * streams.
 *
 * All three buffers are DEVICE pointers on the current device and stay owned by the caller:
 * dev_x fp32 [M][K], dev_w bf16 bits [N][K] row-major, dev_y fp32 [M][N] (overwritten).  dev_x and
 * dev_w are read with 16-byte vector loads and must be 16-byte aligned, dev_y 4-byte aligned (a
 * view into a larger tensor that starts at an odd element offset is not); a misaligned pointer
 * returns SDV_EINVAL before anything runs.  Where the runtime can tell, a pointer that is not device
 * memory of the current device is refused the same way.
 * cuda_stream is a cudaStream_t (NULL = the default stream); the work is queued on it and the
 * call returns after it has finished (it synchronises that stream).
 *
 * Scratch (the weights in streaming order, the accumulators, an error word)
 * lives in a fixed array of about 2.5 MB inside the library's device image, present on every GPU
 * that loads the library for as long as it stays loaded.  Hence the limits: M <= 32, N <= 4096,
 * K <= 4096, N % 16 == 0, K % 64 == 0 and N * K * 2 <= 2 MiB; a larger problem returns
 * SDV_ETOOBIG and touches nothing, a malformed one SDV_EINVAL.  The array keeps whatever the last
 * call left in it; each call clears the parts that must start at zero (accumulators, error word)
 * itself.  There is one array per GPU, so two calls that overlap in time on one GPU (different
 * streams or threads) race on it: serialise them.
 *
 * The first call on each device looks up the array's device address (a one-time set-up step that
 * also makes the runtime load the library's device code if it has not yet); make that first call
 * before starting any stream capture.  Returns SDV_OK, SDV_EINVAL, SDV_ETOOBIG, SDV_ECUDA, or
 * SDV_ETIMEOUT if a bounded device-side wait ran out. */
int sdv_gemm_noalloc(const float *dev_x, const uint16_t *dev_w, float *dev_y, int M, int N, int K,
                     void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SDV_H_ */
