// C-ABI of the verify-path library (see include/sdv.h): context set-up, the static work
// partition, weight re-layout, and the launch sequences of prefill / draft / verify / commit.
#include "../../include/sdv.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>
#include <vector>

#include "dense.cuh"
#include "forward.cuh"
#include "layout.cuh"
#include "small_kernels.cuh"

using namespace sdv;

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Regions {
    size_t state, bstate, bar, never, hist, db, rope, norm_w, bias, wlayers, wlm, emb, kcache, vcache, h, qkv_acc, sumsq, part_o,
        part_ml, cand_val, cand_idx, logits, raw_out, staging, wraw, xstage, prof, succ, occ, dw, dh, dxn, dqkv, dq, datt, dact, dtok, total;
    size_t layer_stride, staging_bytes, raw_kmax;
};

constexpr int kMaxGrid = 256;  // per-block candidate arrays are sized for this many blocks

bool config_ok(const sdv_config* c) {
    if (!c) return false;
    if (c->n_layers < 1 || c->d_model < 64 || c->d_model % 64 || c->d_ffn < 64 || c->d_ffn % 64) return false;
    if (c->vocab < 16 || c->vocab % 16) return false;
    if (c->head_dim != 64 && c->head_dim != 128) return false;
    if (c->n_kv_heads < 1 || c->n_q_heads < 1 || c->n_q_heads % c->n_kv_heads) return false;
    const int g = c->n_q_heads / c->n_kv_heads;
    if (g > 8) return false;
    if (c->k_max < 1 || c->k_max > SDV_K_MAX) return false;
    if (c->max_seq < c->k_max + 2) return false;
    if (c->ngram_n < 1 || c->ngram_n > SDV_NGRAM_MAX || c->ngram_min < 1 || c->ngram_min > c->ngram_n) return false;
    if (!(c->rope_theta > 0.f) || !(c->rms_eps > 0.f)) return false;
    return true;
}

// `own_weights` false: a context that reads another context's weights carves none of the weight regions
// (nor the staging areas only weight loading and the stand-alone GEMM use).
Regions carve(const sdv_config* c, bool own_weights = true) {
    Regions r;
    memset(&r, 0, sizeof(r));
    const size_t d = c->d_model, f = c->d_ffn, V = c->vocab, hd = c->head_dim;
    const size_t nq = (size_t)c->n_q_heads * hd, nkv = (size_t)c->n_kv_heads * hd, nqkv = nq + 2 * nkv;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        const size_t o = off;
        off = align_up(off + bytes, 256);
        return o;
    };
    auto take_w = [&](size_t bytes) { return take(own_weights ? bytes : 0); };
    r.state = take(ST_WORDS * 4);
    r.bstate = take(ST_WORDS * 4);  // state block a batched verify step runs on
    r.bar = take(256);
    r.never = take(256);
    r.hist = take(((size_t)c->max_seq + 64) * 4);
    r.db = take(((size_t)c->max_seq + 64) * 4);
    r.rope = take((size_t)c->max_seq * (hd / 2) * sizeof(float2));
    r.norm_w = take_w(((size_t)c->n_layers * 2 + 1) * d * 4);
    r.bias = take_w((size_t)c->n_layers * nqkv * 4);
    r.layer_stride = (nqkv * d + d * nq + 2 * f * d + d * f) * 2;
    r.wlayers = take_w(r.layer_stride * c->n_layers);
    r.wlm = take_w(V * d * 2);
    r.emb = take_w(V * d * 2);
    const size_t kvb = (size_t)c->n_layers * c->n_kv_heads * c->max_seq * hd * 2;
    r.kcache = take(kvb);
    r.vcache = take(kvb);
    r.h = take((size_t)kMaxRows * d * 4);
    r.qkv_acc = take((size_t)kMaxRows * nqkv * 4);
    r.sumsq = take(2 * kMaxRows * 4);
    size_t raw_kmax = f;  // the stand-alone GEMM takes operands of any K up to max(f, d, nq)
    if (d > raw_kmax) raw_kmax = d;
    if (nq > raw_kmax) raw_kmax = nq;
    r.raw_kmax = raw_kmax;
    r.part_o = take((size_t)c->n_q_heads * (kMaxSplits + 1) * kMaxRows * hd * 4);
    r.part_ml = take((size_t)c->n_q_heads * (kMaxSplits + 1) * kMaxRows * 2 * 4);
    r.cand_val = take((size_t)kMaxGrid * kMaxRows * 4);
    r.cand_idx = take((size_t)kMaxGrid * kMaxRows * 4);
    r.logits = take((size_t)kMaxRows * V * 4);
    size_t st = 2 * f * d * 2;  // gate | up of one layer, the largest per-layer group
    if (nqkv * d * 2 > st) st = nqkv * d * 2;
    if (d * nq * 2 > st) st = d * nq * 2;
    if (st < ((size_t)64 << 20)) st = (size_t)64 << 20;
    r.staging_bytes = st;
    r.staging = take_w(st);
    r.wraw = take_w(st);
    r.raw_out = take_w((size_t)kMaxRows * (st / 128) * 4);  // N <= staging / (2 bytes * 64 columns)
    r.xstage = take((size_t)kMaxRows * raw_kmax * 4);
    r.prof = take((size_t)(3 + kPhasesPerLayer * c->n_layers) * kMaxGrid * kProfWords * 8);
    // dense prefill path: row-major weight copies and the activations of one sub-chunk
    r.dw = take_w(r.layer_stride * c->n_layers);
    r.dh = take((size_t)kDenseMaxRows * d * 4);
    r.dxn = take((size_t)kDenseMaxRows * d * 2);
    r.dqkv = take((size_t)kDenseMaxRows * nqkv * 4);
    r.dq = take((size_t)kDenseMaxRows * nq * 2);
    r.datt = take((size_t)kDenseMaxRows * nq * 2);
    r.dact = take((size_t)kDenseMaxRows * f * 2);
    r.dtok = take((size_t)kDenseMaxRows * 4);
    r.succ = take((size_t)c->max_seq * SDV_CALIB_MAX * 4);  // calibration: sampled successors per context position
    r.occ = take((size_t)c->max_seq * SDV_CALIB_MAX * 4);   // and where each occurs in the context
    r.total = off;
    return r;
}

// Chooses how an operation's grid of row tiles x column steps is cut among the blocks and how a
// block walks its share (RW row tiles per pass, SK column steps per stage).  Model of a block's
// time in microseconds: streaming its share at a fair share of HBM bandwidth or walking its
// stages and passes, whichever is longer, plus building its token operand (the bytes it reads from
// L2: residual rows, or split-KV partial results when `merge`) and, when partial sums meet in L2
// (column partitions, or the residual add), the reductions of all blocks.
void choose_partition(OpDesc& o, int G, int rows, bool merge, bool always_add) {
    double best_t = -1.0;
    o.RW = 16;
    o.SK = kStageBytes / kStepBytes / 16;
    o.P_row = 1;
    o.P_k = 1;
    o.unit = 1;
    o.follow = 0;
    for (int RW = 16; RW >= 1; RW /= 2) {
        const int SK = kStageBytes / kStepBytes / RW;
        for (int pr = 1; pr <= o.T && pr <= G; ++pr) {
            const int pk_max = G / pr < o.K16 ? G / pr : o.K16;
            for (int pk = 1; pk <= pk_max; ++pk) {
                const int tiles = (o.T + pr - 1) / pr, ks = (o.K16 + pk - 1) / pk;
                const int passes = (tiles + RW - 1) / RW;
                const int stages = passes * ((ks + SK - 1) / SK);
                const double stream = (double)tiles * ks * kStepBytes / 44000.0;
                const double walk = 0.06 * stages + 0.25 * passes;
                const double operand_bytes =
                    merge ? (double)rows * ks * 2 * (kMaxSplits + 1) * 40.0 : (double)rows * ks * 16 * 4.0;
                double t = (stream > walk ? stream : walk) + 0.8 + operand_bytes / 60000.0;
                if (pk > 1 || always_add) t += 0.7 + 0.016 * pk * (rows / 9.0);
                if (best_t < 0 || t < best_t - 1e-9) {
                    best_t = t;
                    o.RW = RW;
                    o.SK = SK;
                    o.P_row = pr;
                    o.P_k = pk;
                }
            }
        }
    }
}
// A block whose share has fewer row tiles than a pass may hold walks it in one pass all the same:
// RW then only sets the stage length.  Shrinking RW to the tiles a block really has (a power of two)
// doubles SK until a stage is back at the ring slot's size, i.e. fewer, longer bulk copies.
void fit_pass_width(OpDesc& o) {
    if (o.follow) return;
    const int per = o.unit * ((o.T / o.unit + o.P_row - 1) / o.P_row);  // row tiles of the largest share
    while (o.RW > 1 && o.RW / 2 >= per) o.RW /= 2;
    o.SK = kStageBytes / kStepBytes / o.RW;
}

// Operations whose epilogue needs complete sums: all columns in one block, rows spread evenly.
void full_k_partition(OpDesc& o, int G, int unit) {
    o.RW = 16;
    o.SK = kStageBytes / kStepBytes / 16;
    o.unit = unit;
    o.follow = 0;
    o.P_k = 1;
    o.P_row = o.T / unit < G ? o.T / unit : G;
}

// Shared-memory plan of a launch over `rows` token rows: ring of weight stages | operand region |
// SwiGLU operand | bookkeeping.  The operand region holds the token operand of the widest GEMM
// share (or the attention tiles); the ring takes what is left.
struct SmemPlan {
    int NG, NB, nstage, u_off, act_off, misc_off, total;
    bool ok;
};
SmemPlan plan_smem(const FwdParams& P, int rows, bool raw_only) {
    SmemPlan s;
    s.NG = (rows + 7) / 8;
    s.NB = rows > 16 ? 32 : 16;
    const int step_bytes = 32 * rows;  // token operand bytes per column step: 16 columns x rows x bf16
    int max_ks = 0;
    for (int i = 0; i < OP_COUNT; ++i) {
        const OpDesc& o = P.op[i];
        if (o.T == 0 || o.follow || (raw_only != (i == OP_RAW))) continue;
        const int ks = (o.K16 + o.P_k - 1) / o.P_k;
        if (ks > max_ks) max_ks = ks;
    }
    int u = max_ks * step_bytes;
    if (!raw_only && u < kAttnSmemBytes) u = kAttnSmemBytes;
    u = (u + 1023) / 1024 * 1024;
    s.ok = true;
    int act = 1024;
    if (!raw_only) {
        const OpDesc& gu = P.op[OP_GU];
        const int units = (gu.T / gu.unit + gu.P_row - 1) / gu.P_row;  // SwiGLU column steps per block at most
        act = (units * step_bytes + 1023) / 1024 * 1024;
        if (act > kActSmemMax) s.ok = false;
    }
    const int ring = kSmemBudget - 1024 - kMiscSmemBytes - act - u;
    s.nstage = ring / kStageBytes;
    if (s.nstage > kMaxStages) s.nstage = kMaxStages;
    if (s.nstage < 2) s.ok = false;
    s.u_off = s.nstage * kStageBytes;
    s.act_off = s.u_off + u;
    s.misc_off = s.act_off + act;
    s.total = s.misc_off + kMiscSmemBytes + 1024;  // + slack for 1024-byte alignment
    return s;
}

// The operations of one layer, in streaming order, and the LM head: shapes, partitions, offsets.
void setup_ops(FwdParams& P, const sdv_config* cfg, int G) {
    const int d = cfg->d_model, f = cfg->d_ffn, hd = cfg->head_dim;
    const int nq = cfg->n_q_heads * hd, nkv = cfg->n_kv_heads * hd, nqkv = nq + 2 * nkv;
    struct { int idx, N, K; } ops[5] = {{OP_QKV, nqkv, d}, {OP_O, d, nq}, {OP_GU, 2 * f, d}, {OP_DOWN, d, f},
                                        {OP_LM, cfg->vocab, d}};
    unsigned long long woff = 0;
    int rot = 0;
    const int rows_max = cfg->k_max + 1;
    for (int i = 0; i < 5; ++i) {
        OpDesc& o = P.op[ops[i].idx];
        memset(&o, 0, sizeof(o));
        o.T = ops[i].N / 16;
        o.K16 = ops[i].K / 16;
        switch (ops[i].idx) {
            case OP_QKV: choose_partition(o, G, rows_max, false, false); break;
            case OP_O: choose_partition(o, G, rows_max, true, true); break;
            case OP_GU: full_k_partition(o, G, 2); break;   // pairs of tiles: 16 SwiGLU columns = one column step of down
            case OP_LM: full_k_partition(o, G, 1); break;
            default:  // down: every block multiplies the SwiGLU columns it produced
                o.RW = 16; o.SK = kStageBytes / kStepBytes / 16; o.unit = 1; o.follow = 1; o.P_row = 1; o.P_k = P.op[OP_GU].P_row;
                break;
        }
        fit_pass_width(o);
        if (ops[i].idx == OP_DOWN) {
            o.rot = P.op[OP_GU].rot;
        } else {
            o.rot = rot % G;
            rot += o.P_row * o.P_k;
        }
        o.w_off = (ops[i].idx == OP_LM) ? 0 : woff;
        if (ops[i].idx != OP_LM) woff += (unsigned long long)ops[i].N * ops[i].K * 2;
    }
}

}  // namespace

struct sdv_ctx {
    sdv_config cfg;
    uint8_t* ws;
    size_t ws_bytes;
    Regions r;
    cudaStream_t stream;
    int G;
    FwdParams P;  // template; per-launch fields are filled at launch
    int* pinned;  // host staging for the state block
    cudaEvent_t ev0, ev1;
    // host mirror of the device state
    int kv_len, hist_len, n_ctx;
    bool prefill_done, weights_loaded, verified, draft_pending;
    int draft_k;    // k of the pending sdv_draft
    int last_rows;  // rows of the last verify
    unsigned bar_base;  // grid-barrier counter value before the next launch (wraps; only differences are used)
    int parity;
    int profile;
    int last_cuda;
    long long launches;
    bool have_verify_time;
    bool poisoned;
    std::vector<CUtensorMap>* maps;  // dense path: [0..2] activations (normalised rows, attention output, SwiGLU output), then 4 per layer
    bool dense_ok;       // the tensor maps could be built (else every chunk takes the small-row path)
    int calib_b;         // successors sampled per context position during prefill (0: calibration off)
    bool calibrated;     // the calibration tables cover the whole context
    bool tree_pending;   // the device draft is a tree
    bool tree_verified;  // the outstanding verify result is a tree's
    std::vector<cudaEvent_t>* run_ev;  // event pairs around the forward kernels of the last run of enqueued steps
    int run_steps;       // steps of that run
    sdv_ctx* leader;     // the context whose weights this one reads (nullptr: its own)
    const float* logits_src;  // where the rows of this context's last verify step lie (a batched step leaves them in the first context's buffer)
};

namespace {

int cuda_fail(sdv_ctx* ctx, cudaError_t e) {
    if (ctx) ctx->last_cuda = (int)e;
    return SDV_ECUDA;
}
#define CK(call)                                          \
    do {                                                  \
        cudaError_t e_ = (call);                          \
        if (e_ != cudaSuccess) return cuda_fail(ctx, e_); \
    } while (0)

cudaError_t launch_kernel(const FwdParams& P, int smem_bytes, cudaStream_t stream) {
    cudaError_t e = cudaFuncSetAttribute(sdv_forward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e != cudaSuccess) return e;
    void* args[] = {(void*)&P};
    // phases meet at grid barriers, so more than one phase needs all blocks co-resident
    if (P.ph_end - P.ph_begin > 1)
        return cudaLaunchCooperativeKernel((const void*)sdv_forward_kernel, dim3(P.G), dim3(kThreads), args, smem_bytes, stream);
    return cudaLaunchKernel((const void*)sdv_forward_kernel, dim3(P.G), dim3(kThreads), args, smem_bytes, stream);
}

bool apply_plan(FwdParams& P, int rows, bool raw_only, int* smem_bytes) {
    const SmemPlan sp = plan_smem(P, rows, raw_only);
    if (!sp.ok) return false;
    P.M = rows;
    P.NB = sp.NB;
    P.nstage = sp.nstage;
    P.u_off = sp.u_off;
    P.act_off = sp.act_off;
    P.misc_off = sp.misc_off;
    *smem_bytes = sp.total;
    return true;
}

// Attention split of a launch: heads per unit (a unit's rows, heads x M, fill at most four 16-row
// tiles), number of key ranges and keys per range (a multiple of 64).  Cost of a choice = the
// 16-key steps a warp walks one after another: blocks of 64 keys per range x steps per block; with
// more units than blocks (several sequences, each with its own units) the blocks take them in rounds,
// each round paying a unit's fixed cost (about three such steps) again.
void plan_attention(FwdParams& P, int rows, int L, int nseq = 1) {
    P.att_gh = 1;
    if (P.g < 1) return;
    int best = -1;
    for (int gh = 1; gh <= P.g; ++gh) {
        if (gh * rows > 64 && gh > 1) break;
        const int MT = (gh * rows + 15) / 16, KG = MT <= 2 ? 4 : (MT == 3 ? 3 : 2);
        const int QG = (P.g + gh - 1) / gh;
        int cap = P.G / (P.n_kv * QG) - 1;
        if (cap > kMaxSplits) cap = kMaxSplits;
        if (cap < 1) cap = 1;
        int cost = 1, S = 0;
        if (L > 0) {
            const int kps = ((L + cap - 1) / cap + 63) / 64 * 64;
            S = (L + kps - 1) / kps;
            cost = (kps / 64) * ((4 + KG - 1) / KG);
        }
        const int rounds = (P.n_kv * QG * (S + 1) * nseq + P.G - 1) / P.G;
        cost = rounds * (3 + cost);
        if (best < 0 || cost <= best) {  // ties: more heads per unit (fewer reloads of the keys)
            best = cost;
            P.att_gh = gh;
        }
    }
}

// `batch`: the sequences of a batched step (then `rows` is their total, `L` the longest length, and the launch
// reads its tokens from the batch state block).
struct BatchPlan {
    int n, max_rows;
    BatchSeq seq[kMaxBatch];
};
int launch_forward(sdv_ctx* ctx, int rows, int L, int mode, int ph_begin, int ph_end, bool timed, bool force_logits = false,
                   bool tree = false, const BatchPlan* batch = nullptr, bool l_from_state = false, cudaEvent_t* run_ev = nullptr) {
    FwdParams P = ctx->P;
    P.l_from_state = l_from_state ? 1 : 0;
    int smem_bytes = 0;
    const bool raw_only = (ph_begin == 2 + kPhasesPerLayer * ctx->cfg.n_layers);
    if (!apply_plan(P, rows, raw_only, &smem_bytes)) return SDV_EINVAL;
    P.L = L;
    plan_attention(P, batch ? batch->max_rows : rows, L, batch ? batch->n : 1);
    P.nseq = 0;
    if (batch) {
        P.nseq = batch->n;
        for (int b = 0; b < batch->n; ++b) P.seq[b] = batch->seq[b];
        P.state = (int*)(ctx->ws + ctx->r.bstate);
    }
    ctx->logits_src = P.logits;
    P.mode = mode;
    P.ph_begin = ph_begin;
    P.ph_end = ph_end;
    P.bar_base = ctx->bar_base;
    P.store_logits = (ctx->parity || force_logits) ? 1 : 0;
    P.tree = tree ? 1 : 0;
    P.prof = ctx->profile ? (unsigned long long*)(ctx->ws + ctx->r.prof) : nullptr;
    const int nbar = ph_end - ph_begin - 1;
    ctx->bar_base += (unsigned)(nbar * ctx->G);
    if (timed) CK(cudaEventRecord(run_ev ? run_ev[0] : ctx->ev0, ctx->stream));
    cudaError_t e = launch_kernel(P, smem_bytes, ctx->stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    ctx->launches++;
    if (timed) {
        CK(cudaEventRecord(run_ev ? run_ev[1] : ctx->ev1, ctx->stream));
        if (!run_ev) ctx->have_verify_time = true;
    }
    return SDV_OK;
}

int read_state(sdv_ctx* ctx) {
    CK(cudaMemcpyAsync(ctx->pinned, ctx->ws + ctx->r.state, ST_WORDS * 4, cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    if (ctx->pinned[ST_ERR] == 1) {
        ctx->poisoned = true;
        return SDV_ETIMEOUT;
    }
    return SDV_OK;
}

int pack_op(sdv_ctx* ctx, const OpDesc& o, uint8_t* dst_base, const uint16_t* s0, int rows0, const uint16_t* s1,
            int rows1, const uint16_t* s2, int K, int mode, int t_begin, int t_end, int row_base) {
    const long long total = (long long)(t_end - t_begin) * 16 * (K / 8);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 148 * 16) blocks = 148 * 16;
    pack_weights_kernel<<<blocks, 256, 0, ctx->stream>>>(o, ctx->P.op[OP_GU], dst_base, s0, rows0, s1, rows1, s2, K, mode,
                                                       t_begin, t_end, row_base);
    ctx->launches++;
    CK(cudaGetLastError());
    return SDV_OK;
}

void fill_draft_arg(DraftArg& a, const int32_t* tok, int n) {
    memset(&a, 0, sizeof(a));
    a.n = n;
    for (int i = 0; i < n; ++i) a.tok[i] = tok[i];
}

int commit_common(sdv_ctx* ctx, int max_emit, int force_accept, int force_token, int32_t* host_emitted, int* n_emitted,
                  int* kv_len) {
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    if (ctx->tree_verified) {
        // the accepted path's K/V rows move to consecutive cache slots before the length advances
        kv_compact_kernel<<<dim3(ctx->cfg.n_layers * ctx->cfg.n_kv_heads, 2), 128, 0, ctx->stream>>>(
            ctx->P.state, ctx->P.kcache, ctx->P.vcache, ctx->cfg.max_seq, ctx->cfg.head_dim, max_emit);
        ctx->launches++;
        ctx->tree_verified = false;
    }
    commit_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, hist, max_emit, force_accept, force_token, 0);
    ctx->launches++;
    CK(cudaGetLastError());
    int rc = read_state(ctx);
    if (rc) return rc;
    const int n = ctx->pinned[ST_N_EMITTED];
    ctx->kv_len = ctx->pinned[ST_KV_LEN];
    ctx->hist_len = ctx->pinned[ST_HIST_LEN];
    ctx->verified = false;
    ctx->draft_pending = false;
    ctx->tree_pending = false;
    if (n_emitted) *n_emitted = n;
    if (kv_len) *kv_len = ctx->kv_len;
    if (host_emitted)
        for (int i = 0; i < n; ++i) host_emitted[i] = ctx->pinned[ST_EMITTED + i];
    return SDV_OK;
}

// ---- dense prefill path (csrc/dense.cuh)
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}
// bf16 matrix [rows][K] row-major on this GPU; box = 128 rows x 64 columns, 128-byte swizzle, zeros outside.
bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t K) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {K, rows};
    const cuuint64_t strides[1] = {K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kDenseBK, (cuuint32_t)kDenseBM};
    const cuuint32_t estr[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int EPI>
cudaError_t launch_dense_gemm(sdv_ctx* ctx, const CUtensorMap& a, const CUtensorMap& b, int M, int N, int K, float* out_f32, int ld_f32,
                              const float* bias, __nv_bfloat16* out_bf16, int ld_bf16) {
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(dense_gemm_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDenseSmemBytes);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    dim3 grid((N + kDenseBN - 1) / kDenseBN, (M + kDenseBM - 1) / kDenseBM, 1);
    if (EPI != EPI_SWIGLU) {
        // few tiles and a long K (the down projection): split K so that about one block per SM runs; every share
        // keeps at least six stages
        const int tiles = (int)(grid.x * grid.y), nkb = K / kDenseBK;
        int sp = ctx->G / tiles;
        if (sp > nkb / 6) sp = nkb / 6;
        if (sp < 1) sp = 1;
        grid.z = (unsigned)sp;
        if (EPI == EPI_STORE && sp > 1) {
            cudaError_t e = cudaMemsetAsync(out_f32, 0, (size_t)M * ld_f32 * 4, ctx->stream);
            if (e != cudaSuccess) return e;
        }
    }
    dense_gemm_kernel<EPI><<<grid, kDenseThreads, kDenseSmemBytes, ctx->stream>>>(a, b, M, N, K, out_f32, ld_f32, bias, out_bf16, ld_bf16,
                                                                               ctx->P.state + ST_ERR, 2000000000ull);
    ctx->launches++;
    return cudaGetLastError();
}

// One sub-chunk of `rows` (32..256) context tokens at positions L..L+rows-1 through every layer:
// fills their K/V rows.  The tokens are hist[L .. L+rows).
int dense_prefill_rows(sdv_ctx* ctx, int rows, int L) {
    const sdv_config& c = ctx->cfg;
    const int d = c.d_model, f = c.d_ffn, hd = c.head_dim, nq = c.n_q_heads * hd, nkv = c.n_kv_heads * hd, nqkv = nq + 2 * nkv;
    uint8_t* ws = ctx->ws;
    cudaStream_t s = ctx->stream;
    float* h = (float*)(ws + ctx->r.dh);
    __nv_bfloat16* xn = (__nv_bfloat16*)(ws + ctx->r.dxn);
    float* qkv = (float*)(ws + ctx->r.dqkv);
    __nv_bfloat16* q = (__nv_bfloat16*)(ws + ctx->r.dq);
    __nv_bfloat16* att = (__nv_bfloat16*)(ws + ctx->r.datt);
    __nv_bfloat16* act = (__nv_bfloat16*)(ws + ctx->r.dact);
    const int* hist = (const int*)(ws + ctx->r.hist);
    const std::vector<CUtensorMap>& maps = *ctx->maps;
    const float* norm_w = ctx->P.norm_w;
    const float* bias = ctx->P.bias;
    const size_t att_smem = (size_t)(16 * hd * 2 + 4 * 64 * hd * 2 + 128);  // query tile + two K|V blocks
    static bool att_attr = false;
    if (!att_attr) {
        CK(cudaFuncSetAttribute(dense_attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16 * 128 * 2 + 4 * 64 * 128 * 2 + 128));
        CK(cudaFuncSetAttribute(dense_attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, 16 * 64 * 2 + 4 * 64 * 64 * 2 + 128));
        att_attr = true;
    }
    dense_embed_kernel<<<rows, 128, 0, s>>>(hist + L, ctx->P.emb, h, d, c.vocab);
    ctx->launches++;
    for (int l = 0; l < c.n_layers; ++l) {
        const CUtensorMap* mb = &maps[3 + 4 * l];
        const size_t layer_off = (size_t)l * c.n_kv_heads * c.max_seq * hd;
        dense_rmsnorm_kernel<<<rows, 256, 0, s>>>(h, norm_w + (size_t)(2 * l) * d, xn, d, c.rms_eps);
        CK(launch_dense_gemm<EPI_STORE>(ctx, maps[0], mb[0], rows, nqkv, d, qkv, nqkv, bias ? bias + (size_t)l * nqkv : nullptr, nullptr, 0));
        dense_rope_append_kernel<<<dim3(rows, c.n_q_heads + c.n_kv_heads), hd / 2, 0, s>>>(
            qkv, nqkv, ctx->P.rope, q, c.n_q_heads, c.n_kv_heads, hd, ctx->P.kcache, ctx->P.vcache, layer_off, c.max_seq, L);
        const dim3 ag(c.n_q_heads, (rows + 15) / 16);
        if (hd == 128)
            dense_attention_kernel<128><<<ag, 128, att_smem, s>>>(q, ctx->P.kcache, ctx->P.vcache, layer_off, c.max_seq, c.n_q_heads,
                                                                   ctx->P.g, rows, L, ctx->P.scale_log2e, att);
        else
            dense_attention_kernel<64><<<ag, 128, att_smem, s>>>(q, ctx->P.kcache, ctx->P.vcache, layer_off, c.max_seq, c.n_q_heads,
                                                                  ctx->P.g, rows, L, ctx->P.scale_log2e, att);
        CK(launch_dense_gemm<EPI_RESIDUAL>(ctx, maps[1], mb[1], rows, d, nq, h, d, nullptr, nullptr, 0));
        dense_rmsnorm_kernel<<<rows, 256, 0, s>>>(h, norm_w + (size_t)(2 * l + 1) * d, xn, d, c.rms_eps);
        CK(launch_dense_gemm<EPI_SWIGLU>(ctx, maps[0], mb[2], rows, 2 * f, d, nullptr, 0, nullptr, act, f));
        CK(launch_dense_gemm<EPI_RESIDUAL>(ctx, maps[2], mb[3], rows, d, f, h, d, nullptr, nullptr, 0));
        ctx->launches += 4;  // norms, rotary + append, attention
    }
    CK(cudaGetLastError());
    return SDV_OK;
}

}  // namespace

extern "C" {

const char* sdv_strerror(int code) {
    switch (code) {
        case SDV_OK: return "ok";
        case SDV_EINVAL: return "invalid argument or unsupported shape";
        case SDV_ENOMEM: return "workspace too small";
        case SDV_ECAPACITY: return "KV cache or history capacity exceeded";
        case SDV_ESTATE: return "call not valid in the current state";
        case SDV_ECUDA: return "CUDA runtime error";
        case SDV_ETIMEOUT: return "a bounded device-side wait ran out";
        case SDV_ETOOBIG: return "problem larger than the fixed scratch area of the no-allocation entry point";
        default: return "unknown error";
    }
}

size_t sdv_workspace_bytes(const sdv_config* cfg) {
    if (!config_ok(cfg)) return 0;
    return carve(cfg).total;
}

int sdv_last_cuda_error(const sdv_ctx* ctx) { return ctx ? ctx->last_cuda : 0; }
long long sdv_launch_count(const sdv_ctx* ctx) { return ctx ? ctx->launches : 0; }
int sdv_kv_len(const sdv_ctx* ctx) { return ctx ? ctx->kv_len : SDV_EINVAL; }

}  // extern "C"

namespace {
// A context over `dev_workspace`; with a `leader` it reads that context's weights instead of holding its own.
int create_context(const sdv_config* cfg, void* dev_workspace, size_t bytes, cudaStream_t stream, sdv_ctx* leader, sdv_ctx** out) {
    if (!out) return SDV_EINVAL;
    *out = nullptr;
    if (!config_ok(cfg) || !dev_workspace || ((uintptr_t)dev_workspace & 255)) return SDV_EINVAL;
    if (bytes < carve(cfg, leader == nullptr).total) return SDV_ENOMEM;
    sdv_ctx* ctx = new (std::nothrow) sdv_ctx();
    if (!ctx) return SDV_ENOMEM;
    memset(ctx, 0, sizeof(*ctx));
    ctx->cfg = *cfg;
    ctx->ws = (uint8_t*)dev_workspace;
    ctx->ws_bytes = bytes;
    ctx->stream = stream;
    ctx->leader = leader;
    int sms = 0, dev = 0, coop = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev);
    if (e != cudaSuccess || sms <= 0 || !coop) {
        delete ctx;
        return SDV_ECUDA;
    }
    if (sms > kMaxGrid) sms = kMaxGrid;
    ctx->G = sms;  // one persistent block per SM
    ctx->r = carve(cfg, leader == nullptr);
    // every failure below leaves through this: what was created so far is released
    auto fail = [&](int code) {
        if (ctx->pinned) cudaFreeHost(ctx->pinned);
        if (ctx->ev0) cudaEventDestroy(ctx->ev0);
        if (ctx->ev1) cudaEventDestroy(ctx->ev1);
        delete ctx;
        return code;
    };
    e = cudaHostAlloc((void**)&ctx->pinned, 4096, cudaHostAllocDefault);
    if (e == cudaSuccess) e = cudaEventCreate(&ctx->ev0);
    if (e == cudaSuccess) e = cudaEventCreate(&ctx->ev1);
    if (e != cudaSuccess) return fail(SDV_ECUDA);

    const int d = cfg->d_model, f = cfg->d_ffn, hd = cfg->head_dim;
    const int nq = cfg->n_q_heads * hd, nkv = cfg->n_kv_heads * hd, nqkv = nq + 2 * nkv;
    FwdParams& P = ctx->P;
    P.n_layers = cfg->n_layers; P.d = d; P.n_q = cfg->n_q_heads; P.n_kv = cfg->n_kv_heads; P.hd = hd; P.f = f;
    P.V = cfg->vocab; P.max_seq = cfg->max_seq; P.g = cfg->n_q_heads / cfg->n_kv_heads; P.n_qkv = nqkv;
    P.eps = cfg->rms_eps;
    P.scale_log2e = (float)((1.0 / sqrt((double)hd)) * 1.4426950408889634);
    P.G = ctx->G;
    setup_ops(P, cfg, ctx->G);
    const int rows_max = cfg->k_max + 1;
    P.layer_stride = ctx->r.layer_stride;
    uint8_t* ws = ctx->ws;
    if (leader) {
        P.wlayers = leader->P.wlayers;
        P.wlm = leader->P.wlm;
        P.wraw = nullptr;  // no stand-alone GEMM on a context without weight regions
        P.emb = leader->P.emb;
        P.norm_w = leader->P.norm_w;
        P.bias = leader->P.bias;
    } else {
        P.wlayers = ws + ctx->r.wlayers;
        P.wlm = ws + ctx->r.wlm;
        P.wraw = ws + ctx->r.wraw;
        P.emb = (const __nv_bfloat16*)(ws + ctx->r.emb);
        P.norm_w = (const float*)(ws + ctx->r.norm_w);
        P.bias = cfg->qkv_bias ? (const float*)(ws + ctx->r.bias) : nullptr;
    }
    P.rope = (const float2*)(ws + ctx->r.rope);
    P.kcache = (__nv_bfloat16*)(ws + ctx->r.kcache);
    P.vcache = (__nv_bfloat16*)(ws + ctx->r.vcache);
    P.h = (float*)(ws + ctx->r.h);
    P.qkv_acc = (float*)(ws + ctx->r.qkv_acc);
    P.sumsq = (float*)(ws + ctx->r.sumsq);
    P.part_o = (float*)(ws + ctx->r.part_o);
    P.part_ml = (float*)(ws + ctx->r.part_ml);
    P.cand_val = (float*)(ws + ctx->r.cand_val);
    P.cand_idx = (int*)(ws + ctx->r.cand_idx);
    P.logits = (float*)(ws + ctx->r.logits);
    P.raw_out = (float*)(ws + ctx->r.raw_out);
    P.raw_x = (const float*)(ws + ctx->r.xstage);
    P.raw_N = 0;
    P.raw_K = 0;
    P.state = (int*)(ws + ctx->r.state);
    P.hist = (const int*)(ws + ctx->r.hist);
    P.bar = (unsigned*)(ws + ctx->r.bar);
    P.wait_limit_ns = 2000000000ull;
    {
        // the widest verify step must fit the shared-memory plan
        FwdParams probe = P;
        int smem_bytes = 0;
        if (!apply_plan(probe, rows_max, false, &smem_bytes)) return fail(SDV_EINVAL);
    }

    // rotary table in double, rounded once to fp32
    {
        const size_t n = (size_t)cfg->max_seq * (hd / 2);
        std::vector<float2> tab(n);
        for (int i = 0; i < hd / 2; ++i) {
            const double inv = pow((double)cfg->rope_theta, -2.0 * (double)i / (double)hd);
            for (int p = 0; p < cfg->max_seq; ++p) {
                const double a = (double)p * inv;
                tab[(size_t)p * (hd / 2) + i] = make_float2((float)cos(a), (float)sin(a));
            }
        }
        e = cudaMemcpyAsync(ws + ctx->r.rope, tab.data(), n * sizeof(float2), cudaMemcpyHostToDevice, ctx->stream);
        if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    }
    if (e == cudaSuccess) e = cudaMemsetAsync(ws + ctx->r.state, 0, ST_WORDS * 4, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ws + ctx->r.bstate, 0, ST_WORDS * 4, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ws + ctx->r.bar, 0, 256, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ws + ctx->r.never, 0, 256, ctx->stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(ws + ctx->r.hist, 0, ((size_t)cfg->max_seq + 64) * 4, ctx->stream);
    // activations: h .. part_ml are contiguous regions
    if (e == cudaSuccess) e = cudaMemsetAsync(ws + ctx->r.h, 0, ctx->r.cand_val - ctx->r.h, ctx->stream);
    if (e == cudaSuccess) {
        fill_f32_kernel<<<8, 256, 0, ctx->stream>>>(P.cand_val, -INFINITY, (long long)kMaxGrid * kMaxRows);
        fill_i32_kernel<<<8, 256, 0, ctx->stream>>>(P.cand_idx, 0x7fffffff, (long long)kMaxGrid * kMaxRows);
        ctx->launches += 2;
        e = cudaGetLastError();
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->stream);
    if (e != cudaSuccess) return fail(SDV_ECUDA);
    // dense prefill path: tensor maps over its activation buffers and its weight copies
    ctx->maps = new (std::nothrow) std::vector<CUtensorMap>(3 + 4 * (size_t)cfg->n_layers);
    ctx->dense_ok = ctx->maps != nullptr;
    if (ctx->dense_ok) {
        std::vector<CUtensorMap>& m = *ctx->maps;
        ctx->dense_ok = make_map(&m[0], ws + ctx->r.dxn, kDenseMaxRows, d) && make_map(&m[1], ws + ctx->r.datt, kDenseMaxRows, nq) &&
                        make_map(&m[2], ws + ctx->r.dact, kDenseMaxRows, f);
        if (leader) {  // the weight copies of the dense path are the leader's as well
            ctx->dense_ok = ctx->dense_ok && leader->dense_ok;
            for (size_t i = 3; i < m.size() && ctx->dense_ok; ++i) m[i] = (*leader->maps)[i];
        }
        for (int l = 0; l < cfg->n_layers && ctx->dense_ok && !leader; ++l) {
            uint8_t* lb = ws + ctx->r.dw + (size_t)l * ctx->r.layer_stride;
            const size_t o1 = (size_t)nqkv * d * 2, o2 = o1 + (size_t)d * nq * 2, o3 = o2 + (size_t)2 * f * d * 2;
            ctx->dense_ok = make_map(&m[3 + 4 * l], lb, nqkv, d) && make_map(&m[4 + 4 * l], lb + o1, d, nq) &&
                            make_map(&m[5 + 4 * l], lb + o2, 2 * (uint64_t)f, d) && make_map(&m[6 + 4 * l], lb + o3, d, f);
        }
    }
    ctx->logits_src = P.logits;
    ctx->weights_loaded = leader != nullptr;
    *out = ctx;
    return SDV_OK;
}
}  // namespace

extern "C" {

int sdv_create(const sdv_config* cfg, void* dev_workspace, size_t bytes, void* cuda_stream, sdv_ctx** out) {
    return create_context(cfg, dev_workspace, bytes, (cudaStream_t)cuda_stream, nullptr, out);
}

size_t sdv_follower_workspace_bytes(const sdv_config* cfg) {
    if (!config_ok(cfg)) return 0;
    return carve(cfg, false).total;
}

int sdv_create_follower(sdv_ctx* leader, void* dev_workspace, size_t bytes, sdv_ctx** out) {
    if (out) *out = nullptr;
    if (!leader || leader->leader) return SDV_EINVAL;  // followers follow a context that owns its weights
    if (!leader->weights_loaded) return SDV_ESTATE;
    return create_context(&leader->cfg, dev_workspace, bytes, leader->stream, leader, out);
}

int sdv_destroy(sdv_ctx* ctx) {
    if (!ctx) return SDV_EINVAL;
    cudaStreamSynchronize(ctx->stream);
    if (ctx->pinned) cudaFreeHost(ctx->pinned);
    cudaEventDestroy(ctx->ev0);
    cudaEventDestroy(ctx->ev1);
    delete ctx->maps;
    if (ctx->run_ev) {
        for (cudaEvent_t ev : *ctx->run_ev) cudaEventDestroy(ev);
        delete ctx->run_ev;
    }
    delete ctx;
    return SDV_OK;
}

int sdv_load_weights(sdv_ctx* ctx, const sdv_weights* w) {
    if (!ctx || !w || !w->emb || !w->final_norm || !w->layers) return SDV_EINVAL;
    if (ctx->leader) return SDV_ESTATE;
    const sdv_config& c = ctx->cfg;
    if (!c.tied_lm_head && !w->lm_head) return SDV_EINVAL;
    const size_t d = c.d_model, f = c.d_ffn, hd = c.head_dim, V = c.vocab;
    const size_t nq = c.n_q_heads * hd, nkv = c.n_kv_heads * hd, nqkv = nq + 2 * nkv;
    uint8_t* ws = ctx->ws;
    uint16_t* stg = (uint16_t*)(ws + ctx->r.staging);
    float* norm_w = (float*)(ws + ctx->r.norm_w);
    float* bias = (float*)(ws + ctx->r.bias);
    cudaStream_t s = ctx->stream;
    for (int l = 0; l < c.n_layers; ++l) {
        const sdv_layer_weights& L = w->layers[l];
        if (!L.wq || !L.wk || !L.wv || !L.wo || !L.wg || !L.wu || !L.wd || !L.norm1 || !L.norm2) return SDV_EINVAL;
        if (c.qkv_bias && (!L.bq || !L.bk || !L.bv)) return SDV_EINVAL;
        uint8_t* lbase = ws + ctx->r.wlayers + (size_t)l * ctx->r.layer_stride;
        int rc;
        // q | k | v stacked
        CK(cudaMemcpyAsync(stg, L.wq, nq * d * 2, cudaMemcpyDefault, s));
        CK(cudaMemcpyAsync(stg + nq * d, L.wk, nkv * d * 2, cudaMemcpyDefault, s));
        CK(cudaMemcpyAsync(stg + (nq + nkv) * d, L.wv, nkv * d * 2, cudaMemcpyDefault, s));
        rc = pack_op(ctx, ctx->P.op[OP_QKV], lbase + ctx->P.op[OP_QKV].w_off, stg, (int)nq, stg + nq * d, (int)nkv,
                     stg + (nq + nkv) * d, (int)d, 0, 0, ctx->P.op[OP_QKV].T, 0);
        if (rc) return rc;
        // row-major copies for the dense prefill path: q|k|v, o, gate|up (interleaved by 64), down
        uint16_t* dbase = (uint16_t*)(ws + ctx->r.dw + (size_t)l * ctx->r.layer_stride);
        CK(cudaMemcpyAsync(dbase, stg, nqkv * d * 2, cudaMemcpyDeviceToDevice, s));
        CK(cudaStreamSynchronize(s));
        // o
        CK(cudaMemcpyAsync(stg, L.wo, d * nq * 2, cudaMemcpyDefault, s));
        rc = pack_op(ctx, ctx->P.op[OP_O], lbase + ctx->P.op[OP_O].w_off, stg, (int)d, nullptr, 0, nullptr, (int)nq, 0, 0,
                     ctx->P.op[OP_O].T, 0);
        if (rc) return rc;
        CK(cudaMemcpyAsync(dbase + nqkv * d, stg, d * nq * 2, cudaMemcpyDeviceToDevice, s));
        CK(cudaStreamSynchronize(s));
        // gate | up, interleaved 8 + 8 rows per tile
        CK(cudaMemcpyAsync(stg, L.wg, f * d * 2, cudaMemcpyDefault, s));
        CK(cudaMemcpyAsync(stg + f * d, L.wu, f * d * 2, cudaMemcpyDefault, s));
        rc = pack_op(ctx, ctx->P.op[OP_GU], lbase + ctx->P.op[OP_GU].w_off, stg, (int)f, stg + f * d, (int)f, nullptr,
                     (int)d, 1, 0, ctx->P.op[OP_GU].T, 0);
        if (rc) return rc;
        dense_copy_weights_kernel<<<148 * 8, 256, 0, s>>>(dbase + nqkv * d + d * nq, stg, stg + f * d, (int)(2 * f), (int)d, 1);
        ctx->launches++;
        CK(cudaGetLastError());
        CK(cudaStreamSynchronize(s));
        // down
        CK(cudaMemcpyAsync(stg, L.wd, d * f * 2, cudaMemcpyDefault, s));
        rc = pack_op(ctx, ctx->P.op[OP_DOWN], lbase + ctx->P.op[OP_DOWN].w_off, stg, (int)d, nullptr, 0, nullptr, (int)f,
                     0, 0, ctx->P.op[OP_DOWN].T, 0);
        if (rc) return rc;
        CK(cudaMemcpyAsync(dbase + nqkv * d + d * nq + 2 * f * d, stg, d * f * 2, cudaMemcpyDeviceToDevice, s));
        CK(cudaStreamSynchronize(s));
        CK(cudaMemcpyAsync(norm_w + ((size_t)l * 2 + 0) * d, L.norm1, d * 4, cudaMemcpyDefault, s));
        CK(cudaMemcpyAsync(norm_w + ((size_t)l * 2 + 1) * d, L.norm2, d * 4, cudaMemcpyDefault, s));
        if (c.qkv_bias) {
            CK(cudaMemcpyAsync(bias + (size_t)l * nqkv, L.bq, nq * 4, cudaMemcpyDefault, s));
            CK(cudaMemcpyAsync(bias + (size_t)l * nqkv + nq, L.bk, nkv * 4, cudaMemcpyDefault, s));
            CK(cudaMemcpyAsync(bias + (size_t)l * nqkv + nq + nkv, L.bv, nkv * 4, cudaMemcpyDefault, s));
        }
    }
    CK(cudaMemcpyAsync(norm_w + (size_t)c.n_layers * 2 * d, w->final_norm, d * 4, cudaMemcpyDefault, s));
    CK(cudaMemcpyAsync(ws + ctx->r.emb, w->emb, V * d * 2, cudaMemcpyDefault, s));
    // LM head: packed from row blocks that fit the staging area
    {
        const uint16_t* src = c.tied_lm_head ? w->emb : w->lm_head;
        const OpDesc& o = ctx->P.op[OP_LM];
        const size_t tiles_per = ctx->r.staging_bytes / (16 * d * 2);
        if (tiles_per < 1) return SDV_ENOMEM;
        for (size_t t0 = 0; t0 < (size_t)o.T; t0 += tiles_per) {
            const size_t t1 = (t0 + tiles_per < (size_t)o.T) ? t0 + tiles_per : (size_t)o.T;
            const size_t rows = (t1 - t0) * 16;
            CK(cudaMemcpyAsync(stg, src + t0 * 16 * d, rows * d * 2, cudaMemcpyDefault, s));
            int rc = pack_op(ctx, o, ws + ctx->r.wlm, stg, (int)rows, nullptr, 0, nullptr, (int)d, 0, (int)t0, (int)t1,
                             (int)(t0 * 16));
            if (rc) return rc;
            CK(cudaStreamSynchronize(s));
        }
    }
    CK(cudaStreamSynchronize(s));
    ctx->weights_loaded = true;
    return SDV_OK;
}

int sdv_set_parity_mode(sdv_ctx* ctx, int on) {
    if (!ctx) return SDV_EINVAL;
    ctx->parity = on ? 1 : 0;
    return SDV_OK;
}

int sdv_prefill_chunk(sdv_ctx* ctx, const int32_t* host_tokens, int n, int is_last) {
    if (!ctx || !host_tokens || n < 1) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->weights_loaded || ctx->prefill_done) return SDV_ESTATE;
    const sdv_config& c = ctx->cfg;
    if (ctx->kv_len + n + 1 + c.k_max + 1 > c.max_seq) return SDV_ECAPACITY;
    for (int i = 0; i < n; ++i)
        if (host_tokens[i] < 0 || host_tokens[i] >= c.vocab) return SDV_EINVAL;
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    CK(cudaMemcpyAsync(hist + ctx->hist_len, host_tokens, (size_t)n * 4, cudaMemcpyDefault, ctx->stream));
    // rows per launch
    int tile = 24;
    {
        // wide models: fewer rows per launch so that the token operand leaves room for the weight ring
        FwdParams probe = ctx->P;
        int smem_bytes = 0;
        while (tile > 8 && (!apply_plan(probe, tile, false, &smem_bytes) || probe.nstage < 4)) tile -= 8;
    }
    const int n_ph = 1 + kPhasesPerLayer * c.n_layers;
    int done = 0;
    while (done < n) {
        // sub-chunks of 32..256 rows go through the dense path (tokens on the tensor cores' M side, every weight
        // streamed once); the last token of the request (its logits give the first generated token), short
        // remainders and calibrated prefill (logits of every row) take the small-row kernel
        const int dense_rows_avail = n - done - (is_last ? 1 : 0);
        if (ctx->dense_ok && ctx->calib_b == 0 && dense_rows_avail >= 32) {
            const int rows = dense_rows_avail < kDenseMaxRows ? dense_rows_avail : kDenseMaxRows;
            int rc = dense_prefill_rows(ctx, rows, ctx->kv_len);
            if (rc) return rc;
            ctx->kv_len += rows;
            ctx->hist_len += rows;
            done += rows;
            if (done == n) {   // the chunk ended here (never the last one: its final token takes the path below)
                ctx->n_ctx = ctx->hist_len;
                set_state_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, ctx->kv_len, ctx->hist_len, ctx->n_ctx, 0, hist);
                ctx->launches++;
                CK(cudaGetLastError());
            }
            continue;
        }
        const int rows = (n - done < tile) ? n - done : tile;
        const bool last_tile = is_last && (done + rows == n);
        const bool calib = ctx->calib_b > 0;
        int rc = launch_forward(ctx, rows, ctx->kv_len, 1, 0, (last_tile || calib) ? n_ph + 1 : n_ph, false, calib);
        if (rc) return rc;
        if (calib) {
            // "Sample": the best successors of every row of this tile, from the logits the LM head just stored
            top_successors_kernel<<<rows, 1024, 0, ctx->stream>>>(ctx->P.logits, c.vocab, ctx->calib_b,
                                                               (int*)(ctx->ws + ctx->r.succ) + (size_t)ctx->kv_len * ctx->calib_b);
            ctx->launches++;
            CK(cudaGetLastError());
        }
        ctx->kv_len += rows;
        ctx->hist_len += rows;
        done += rows;
        if (done == n) {
            // the context now covers everything prefilled so far
            ctx->n_ctx = ctx->hist_len;
            set_state_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, ctx->kv_len, ctx->hist_len, ctx->n_ctx, 0, hist);
            ctx->launches++;
            CK(cudaGetLastError());
            if (last_tile) {
                // greedy token of the last context row: appended to the history as the pending token T
                prefill_final_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, hist, ctx->P.cand_val, ctx->P.cand_idx,
                                                              ctx->G, rows - 1);
                ctx->launches++;
                CK(cudaGetLastError());
                ctx->hist_len += 1;
                ctx->prefill_done = true;
                if (ctx->calib_b > 0) {
                    // "Search": where each sampled successor occurs in the request
                    const int total = ctx->n_ctx * ctx->calib_b;
                    anchor_search_kernel<<<(total + 255) / 256, 256, 0, ctx->stream>>>(
                        hist, ctx->n_ctx, ctx->calib_b, (const int*)(ctx->ws + ctx->r.succ), (int*)(ctx->ws + ctx->r.occ));
                    ctx->launches++;
                    CK(cudaGetLastError());
                    ctx->calibrated = true;
                }
            }
        }
    }
    return read_state(ctx);
}

int sdv_draft(sdv_ctx* ctx, int k, int32_t* host_draft, int* draft_len) {
    if (!ctx || k < 1 || k > ctx->cfg.k_max) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done) return SDV_ESTATE;
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    ngram_draft_kernel<<<1, 1024, 0, ctx->stream>>>(ctx->P.state, hist, (const int*)(ctx->ws + ctx->r.db), ctx->cfg.ngram_n,
                                                    ctx->cfg.ngram_min, k, ctx->cfg.search_history, 0);
    ctx->launches++;
    CK(cudaGetLastError());
    ctx->draft_pending = true;
    ctx->tree_pending = false;
    ctx->draft_k = k;
    ctx->verified = false;
    if (host_draft || draft_len) {
        int rc = read_state(ctx);
        if (rc) return rc;
        const int dl = ctx->pinned[ST_DRAFT_LEN];
        if (draft_len) *draft_len = dl;
        if (host_draft)
            for (int i = 0; i < dl; ++i) host_draft[i] = ctx->pinned[ST_DRAFT + i];
    }
    return SDV_OK;
}

int sdv_verify(sdv_ctx* ctx, const int32_t* host_draft, int draft_len, int32_t* host_y, int* accept_len) {
    if (!ctx) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done || !ctx->weights_loaded) return SDV_ESTATE;
    const sdv_config& c = ctx->cfg;
    int rows;
    if (host_draft) {
        if (draft_len < 0 || draft_len > c.k_max) return SDV_EINVAL;
        for (int i = 0; i < draft_len; ++i)
            if (host_draft[i] < 0 || host_draft[i] >= c.vocab) return SDV_EINVAL;
        rows = draft_len + 1;
    } else {
        rows = ctx->draft_pending ? ctx->draft_k + 1 : 1;
    }
    if (ctx->kv_len + rows > c.max_seq) return SDV_ECAPACITY;
    if (host_draft) {
        DraftArg a;
        fill_draft_arg(a, host_draft, draft_len);
        set_draft_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, a);
        ctx->launches++;
        CK(cudaGetLastError());
    }
    const bool tree = !host_draft && ctx->tree_pending;
    int rc = launch_forward(ctx, rows, ctx->kv_len, 0, 0, 2 + kPhasesPerLayer * c.n_layers, true, false, tree);
    if (rc) return rc;
    accept_kernel<<<1, 32 * rows, 0, ctx->stream>>>(ctx->P.state, ctx->P.cand_val, ctx->P.cand_idx, ctx->G, 0, 0, nullptr, 0);
    ctx->launches++;
    CK(cudaGetLastError());
    ctx->verified = true;
    ctx->tree_verified = tree;
    ctx->last_rows = rows;
    if (host_y || accept_len) {
        rc = read_state(ctx);
        if (rc) return rc;
        const int dl = ctx->pinned[ST_DRAFT_LEN];
        if (accept_len) *accept_len = ctx->pinned[ST_ACCEPT_LEN];
        if (host_y)
            for (int i = 0; i <= dl; ++i) host_y[i] = ctx->pinned[ST_Y + i];
    }
    return SDV_OK;
}

int sdv_verify_batch(sdv_ctx* const* ctxs, int n, int* accept_len) {
    if (!ctxs || n < 1 || n > kMaxBatch) return SDV_EINVAL;
    sdv_ctx* ctx = ctxs[0];  // the launch runs on the first context's scratch buffers and stream
    if (!ctx) return SDV_EINVAL;
    sdv_ctx* owner = ctx->leader ? ctx->leader : ctx;
    BatchPlan bp;
    BatchGatherArg ga;
    memset(&bp, 0, sizeof(bp));
    memset(&ga, 0, sizeof(ga));
    bp.n = ga.n = n;
    int rows = 0, Lmax = 0;
    for (int b = 0; b < n; ++b) {
        sdv_ctx* c = ctxs[b];
        if (!c) return SDV_EINVAL;
        for (int a = 0; a < b; ++a)
            if (ctxs[a] == c) return SDV_EINVAL;
        if ((c->leader ? c->leader : c) != owner || c->stream != ctx->stream) return SDV_EINVAL;
        if (c->poisoned) return SDV_ETIMEOUT;
        if (!c->prefill_done || !c->weights_loaded || c->tree_pending) return SDV_ESTATE;  // chains only
        const int m = c->draft_pending ? c->draft_k + 1 : 1;
        if (c->kv_len + m > c->cfg.max_seq) return SDV_ECAPACITY;
        bp.seq[b].kcache = c->P.kcache;
        bp.seq[b].vcache = c->P.vcache;
        bp.seq[b].r0 = ga.r0[b] = rows;
        bp.seq[b].M = ga.M[b] = m;
        bp.seq[b].L = c->kv_len;
        ga.state[b] = c->P.state;
        if (m > bp.max_rows) bp.max_rows = m;
        if (c->kv_len > Lmax) Lmax = c->kv_len;
        rows += m;
    }
    if (rows > kMaxRows) return SDV_EINVAL;
    int* bstate = (int*)(ctx->ws + ctx->r.bstate);
    batch_gather_kernel<<<1, kMaxRows, 0, ctx->stream>>>(bstate, ga);
    ctx->launches++;
    CK(cudaGetLastError());
    int rc = launch_forward(ctx, rows, Lmax, 0, 0, 2 + kPhasesPerLayer * ctx->cfg.n_layers, true, false, false, &bp);
    if (rc) return rc;
    for (int b = 0; b < n; ++b) {
        sdv_ctx* c = ctxs[b];
        accept_kernel<<<1, 32 * bp.seq[b].M, 0, ctx->stream>>>(c->P.state, ctx->P.cand_val, ctx->P.cand_idx, ctx->G, 0, bp.seq[b].r0,
                                                              bstate, 0);
        ctx->launches++;
        c->verified = true;
        c->tree_verified = false;
        c->last_rows = bp.seq[b].M;
        c->logits_src = ctx->P.logits + (size_t)bp.seq[b].r0 * ctx->cfg.vocab;
    }
    CK(cudaGetLastError());
    if (accept_len) {
        for (int b = 0; b < n; ++b) {
            sdv_ctx* c = ctxs[b];
            rc = read_state(c);
            if (rc) return rc;
            accept_len[b] = c->pinned[ST_ACCEPT_LEN];
        }
    }
    return SDV_OK;
}

int sdv_get_verified(sdv_ctx* ctx, int32_t* host_y, int* accept_len) {
    if (!ctx) return SDV_EINVAL;
    if (!ctx->verified) return SDV_ESTATE;
    int rc = read_state(ctx);
    if (rc) return rc;
    if (accept_len) *accept_len = ctx->pinned[ST_ACCEPT_LEN];
    if (host_y)
        for (int i = 0; i < ctx->last_rows; ++i) host_y[i] = ctx->pinned[ST_Y + i];
    return SDV_OK;
}

int sdv_set_database(sdv_ctx* ctx, const int32_t* host_tokens, int n) {
    if (!ctx || n < 0 || n > ctx->cfg.max_seq || (n && !host_tokens)) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    for (int i = 0; i < n; ++i)
        if (host_tokens[i] < 0 || host_tokens[i] >= ctx->cfg.vocab) return SDV_EINVAL;
    if (n) CK(cudaMemcpyAsync(ctx->ws + ctx->r.db, host_tokens, (size_t)n * 4, cudaMemcpyDefault, ctx->stream));
    set_word_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, ST_DB_LEN, n);
    ctx->launches++;
    CK(cudaGetLastError());
    CK(cudaStreamSynchronize(ctx->stream));  // the caller's buffer may go away
    return SDV_OK;
}

int sdv_extend_draft(sdv_ctx* ctx, int max_total, int32_t* host_draft, int* draft_len) {
    if (!ctx || max_total < 1 || max_total > ctx->cfg.k_max) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done || !ctx->draft_pending) return SDV_ESTATE;
    extend_draft_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, max_total, 0);
    ctx->launches++;
    CK(cudaGetLastError());
    // rows of the next verify: the exact draft length when the caller reads it, else the bound
    if (ctx->draft_k < max_total) ctx->draft_k = max_total;
    if (host_draft || draft_len) {
        int rc = read_state(ctx);
        if (rc) return rc;
        const int dl = ctx->pinned[ST_DRAFT_LEN];
        ctx->draft_k = dl;
        if (draft_len) *draft_len = dl;
        if (host_draft)
            for (int i = 0; i < dl; ++i) host_draft[i] = ctx->pinned[ST_DRAFT + i];
    }
    return SDV_OK;
}

int sdv_extension_update(sdv_ctx* ctx, int max_life, int32_t* host_segment, int* segment_len, int* lifetime) {
    if (!ctx || max_life < 1) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->verified) return SDV_ESTATE;
    extension_update_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, max_life, 0);
    ctx->launches++;
    CK(cudaGetLastError());
    if (host_segment || segment_len || lifetime) {
        int rc = read_state(ctx);
        if (rc) return rc;
        const int sl = ctx->pinned[ST_SEG_LEN];
        if (segment_len) *segment_len = sl;
        if (lifetime) *lifetime = ctx->pinned[ST_SEG_LIFE];
        if (host_segment)
            for (int i = 0; i < sl; ++i) host_segment[i] = ctx->pinned[ST_SEG + i];
    }
    return SDV_OK;
}

int sdv_step(sdv_ctx* ctx, const int32_t* host_draft, int draft_len, int k_next, int32_t* host_emitted, int* n_emitted,
             int32_t* host_next_draft, int* next_draft_len, int* kv_len) {
    if (!ctx || k_next < 0 || k_next > ctx->cfg.k_max) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done || !ctx->weights_loaded) return SDV_ESTATE;
    const sdv_config& c = ctx->cfg;
    int rows;
    if (host_draft) {
        if (draft_len < 0 || draft_len > c.k_max) return SDV_EINVAL;
        for (int i = 0; i < draft_len; ++i)
            if (host_draft[i] < 0 || host_draft[i] >= c.vocab) return SDV_EINVAL;
        rows = draft_len + 1;
    } else {
        if (ctx->tree_pending) return SDV_ESTATE;  // chains only
        rows = ctx->draft_pending ? ctx->draft_k + 1 : 1;
    }
    if (ctx->kv_len + rows > c.max_seq || ctx->hist_len + rows > c.max_seq + 64) return SDV_ECAPACITY;
    int* state = ctx->P.state;
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    if (host_draft) {
        DraftArg a;
        fill_draft_arg(a, host_draft, draft_len);
        set_draft_kernel<<<1, 32, 0, ctx->stream>>>(state, a);
        ctx->launches++;
    }
    int rc = launch_forward(ctx, rows, ctx->kv_len, 0, 0, 2 + kPhasesPerLayer * c.n_layers, true);
    if (rc) return rc;
    step_tail_kernel<<<1, 1024, 0, ctx->stream>>>(state, hist, (const int*)(ctx->ws + ctx->r.db), ctx->P.cand_val, ctx->P.cand_idx,
                                                  ctx->G, c.ngram_n, c.ngram_min, k_next, c.search_history, 0, 0, k_next > 0 ? 1 : 0, 0);
    ctx->launches++;
    CK(cudaGetLastError());
    ctx->last_rows = rows;
    ctx->verified = false;
    ctx->tree_pending = false;
    ctx->tree_verified = false;
    ctx->draft_pending = k_next > 0;
    ctx->draft_k = k_next;
    rc = read_state(ctx);  // one copy of the state block: emitted tokens, lengths and the next draft
    if (rc) return rc;
    const int n = ctx->pinned[ST_N_EMITTED];
    ctx->kv_len = ctx->pinned[ST_KV_LEN];
    ctx->hist_len = ctx->pinned[ST_HIST_LEN];
    if (n_emitted) *n_emitted = n;
    if (kv_len) *kv_len = ctx->kv_len;
    if (host_emitted)
        for (int i = 0; i < n; ++i) host_emitted[i] = ctx->pinned[ST_EMITTED + i];
    const int dl = k_next > 0 ? ctx->pinned[ST_DRAFT_LEN] : 0;
    if (next_draft_len) *next_draft_len = dl;
    if (host_next_draft)
        for (int i = 0; i < dl; ++i) host_next_draft[i] = ctx->pinned[ST_DRAFT + i];
    return SDV_OK;
}

int sdv_decode_steps(sdv_ctx* ctx, int k, int n_steps, int max_tokens, int ext_max_total, int ext_max_life, int32_t* host_tokens,
                     int* n_tokens, int* kv_len) {
    if (!ctx || k < 1 || k > ctx->cfg.k_max || n_steps < 1 || n_steps > 4096) return SDV_EINVAL;
    if (ext_max_total < 0 || ext_max_total > ctx->cfg.k_max || (ext_max_total > 0 && (ext_max_total < k || ext_max_life < 1)))
        return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done || !ctx->weights_loaded) return SDV_ESTATE;
    const sdv_config& c = ctx->cfg;
    const int rows = (ext_max_total > 0 ? ext_max_total : k) + 1;
    // every step may write `rows` KV rows beyond the length it starts from and emit up to `rows` tokens
    if ((long long)ctx->kv_len + (long long)n_steps * rows > c.max_seq) return SDV_ECAPACITY;
    if ((long long)ctx->hist_len + (long long)n_steps * rows > c.max_seq + 64) return SDV_ECAPACITY;
    if (!ctx->run_ev) ctx->run_ev = new (std::nothrow) std::vector<cudaEvent_t>();
    if (!ctx->run_ev) return SDV_ENOMEM;
    while (ctx->run_ev->size() < 2 * (size_t)n_steps) {
        cudaEvent_t ev;
        CK(cudaEventCreate(&ev));
        ctx->run_ev->push_back(ev);
    }
    int* state = ctx->P.state;
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    const int hist_before = ctx->hist_len;
    fill_i32_kernel<<<1, 32, 0, ctx->stream>>>(state + ST_BUDGET, max_tokens > 0 ? max_tokens : -1, 1);
    const int* db = (const int*)(ctx->ws + ctx->r.db);
    ngram_draft_kernel<<<1, 1024, 0, ctx->stream>>>(state, hist, db, c.ngram_n, c.ngram_min, k, c.search_history, 1);
    if (ext_max_total > 0) extend_draft_kernel<<<1, 32, 0, ctx->stream>>>(state, ext_max_total, 1);
    ctx->launches += ext_max_total > 0 ? 3 : 2;
    const int all_phases = 2 + kPhasesPerLayer * c.n_layers;
    for (int i = 0; i < n_steps; ++i) {
        // the kernel reads the KV length from the state block; the host's value (a lower bound) only shapes the attention split
        int rc = launch_forward(ctx, rows, ctx->kv_len, 0, 0, all_phases, true, false, false, nullptr, true,
                                ctx->run_ev->data() + 2 * i);
        if (rc) return rc;
        // accept, commit and the next step's draft in one launch
        step_tail_kernel<<<1, 1024, 0, ctx->stream>>>(state, hist, db, ctx->P.cand_val, ctx->P.cand_idx, ctx->G, c.ngram_n,
                                                      c.ngram_min, k, c.search_history, ext_max_total, ext_max_life,
                                                      i + 1 < n_steps ? 1 : 0, 1);
        ctx->launches++;
    }
    CK(cudaGetLastError());
    ctx->run_steps = n_steps;
    ctx->verified = false;
    ctx->draft_pending = false;
    ctx->tree_pending = false;
    ctx->tree_verified = false;
    int rc = read_state(ctx);
    if (rc) return rc;
    ctx->kv_len = ctx->pinned[ST_KV_LEN];
    ctx->hist_len = ctx->pinned[ST_HIST_LEN];
    const int n = ctx->hist_len - hist_before;
    if (n_tokens) *n_tokens = n;
    if (kv_len) *kv_len = ctx->kv_len;
    if (host_tokens && n > 0) {
        CK(cudaMemcpyAsync(host_tokens, hist + hist_before, (size_t)n * 4, cudaMemcpyDeviceToHost, ctx->stream));
        CK(cudaStreamSynchronize(ctx->stream));
    }
    return SDV_OK;
}

int sdv_run_kernel_ms(sdv_ctx* ctx, float* host_ms, int n) {
    if (!ctx || !host_ms || n < 1) return SDV_EINVAL;
    if (!ctx->run_ev || n > ctx->run_steps) return SDV_ESTATE;
    CK(cudaStreamSynchronize(ctx->stream));
    for (int i = 0; i < n; ++i) CK(cudaEventElapsedTime(&host_ms[i], (*ctx->run_ev)[2 * i], (*ctx->run_ev)[2 * i + 1]));
    return SDV_OK;
}

int sdv_set_calibration(sdv_ctx* ctx, int top_b) {
    if (!ctx || top_b < 0 || top_b > SDV_CALIB_MAX) return SDV_EINVAL;
    if (ctx->kv_len > 0 || ctx->prefill_done) return SDV_ESTATE;  // the tables are filled while the context is prefilled
    ctx->calib_b = top_b;
    ctx->calibrated = false;
    return SDV_OK;
}

int sdv_get_calibration(sdv_ctx* ctx, int32_t* host_succ, int32_t* host_occ, int n_positions) {
    if (!ctx || n_positions < 1 || (!host_succ && !host_occ)) return SDV_EINVAL;
    if (!ctx->calibrated) return SDV_ESTATE;
    if (n_positions > ctx->n_ctx) return SDV_EINVAL;
    const size_t bytes = (size_t)n_positions * ctx->calib_b * 4;
    if (host_succ) CK(cudaMemcpyAsync(host_succ, ctx->ws + ctx->r.succ, bytes, cudaMemcpyDeviceToHost, ctx->stream));
    if (host_occ) CK(cudaMemcpyAsync(host_occ, ctx->ws + ctx->r.occ, bytes, cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    return SDV_OK;
}

int sdv_draft_tree(sdv_ctx* ctx, int k, int max_nodes, int32_t* host_tokens, int32_t* host_parent, int* n_nodes) {
    if (!ctx || k < 0 || k > ctx->cfg.k_max || max_nodes < 1 || max_nodes > ctx->cfg.k_max) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done) return SDV_ESTATE;
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    if (k > 0) {
        ngram_draft_kernel<<<1, 1024, 0, ctx->stream>>>(ctx->P.state, hist, (const int*)(ctx->ws + ctx->r.db), ctx->cfg.ngram_n,
                                                        ctx->cfg.ngram_min, k, ctx->cfg.search_history, 0);
    } else {
        DraftArg none;
        fill_draft_arg(none, nullptr, 0);
        set_draft_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, none);
    }
    tree_draft_kernel<<<1, 1024, 0, ctx->stream>>>(ctx->P.state, hist, (const int*)(ctx->ws + ctx->r.succ),
                                                   (const int*)(ctx->ws + ctx->r.occ), ctx->calibrated ? ctx->calib_b : 0, max_nodes);
    ctx->launches += 2;
    CK(cudaGetLastError());
    ctx->draft_pending = true;
    ctx->tree_pending = true;
    ctx->draft_k = max_nodes;   // rows of the next verify: the bound, or the exact count when the caller reads it
    ctx->verified = false;
    if (host_tokens || host_parent || n_nodes) {
        int rc = read_state(ctx);
        if (rc) return rc;
        const int n = ctx->pinned[ST_DRAFT_LEN];
        ctx->draft_k = n;
        if (n_nodes) *n_nodes = n;
        for (int i = 0; i < n; ++i) {
            if (host_tokens) host_tokens[i] = ctx->pinned[ST_DRAFT + i];
            if (host_parent) host_parent[i] = ctx->pinned[ST_PARENT + 1 + i];
        }
    }
    return SDV_OK;
}

int sdv_verify_tree(sdv_ctx* ctx, const int32_t* host_tokens, const int32_t* host_parent, int n_nodes, int32_t* host_y,
                    int32_t* host_path, int* path_len) {
    if (!ctx) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done || !ctx->weights_loaded) return SDV_ESTATE;
    const sdv_config& c = ctx->cfg;
    int rows;
    if (host_tokens) {
        if (!host_parent || n_nodes < 0 || n_nodes > c.k_max) return SDV_EINVAL;
        for (int i = 0; i < n_nodes; ++i) {
            if (host_tokens[i] < 0 || host_tokens[i] >= c.vocab) return SDV_EINVAL;
            if (host_parent[i] < 0 || host_parent[i] > i) return SDV_EINVAL;  // node i + 1 continues an earlier row
        }
        rows = n_nodes + 1;
    } else {
        if (!ctx->tree_pending) return SDV_ESTATE;
        rows = ctx->draft_k + 1;
    }
    if (ctx->kv_len + rows > c.max_seq) return SDV_ECAPACITY;
    if (host_tokens) {
        DraftArg t, p;
        fill_draft_arg(t, host_tokens, n_nodes);
        fill_draft_arg(p, host_parent, n_nodes);
        set_tree_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, t, p);
        ctx->launches++;
        CK(cudaGetLastError());
    }
    int rc = launch_forward(ctx, rows, ctx->kv_len, 0, 0, 2 + kPhasesPerLayer * c.n_layers, true, false, true);
    if (rc) return rc;
    accept_kernel<<<1, 32 * rows, 0, ctx->stream>>>(ctx->P.state, ctx->P.cand_val, ctx->P.cand_idx, ctx->G, 0, 0, nullptr, 0);
    ctx->launches++;
    CK(cudaGetLastError());
    ctx->verified = true;
    ctx->tree_verified = true;
    ctx->last_rows = rows;
    if (host_y || host_path || path_len) {
        rc = read_state(ctx);
        if (rc) return rc;
        const int n = ctx->pinned[ST_DRAFT_LEN], a = ctx->pinned[ST_PATH_LEN];
        if (path_len) *path_len = a;
        if (host_path)
            for (int i = 0; i < a; ++i) host_path[i] = ctx->pinned[ST_PATH + i];
        if (host_y)
            for (int i = 0; i <= n; ++i) host_y[i] = ctx->pinned[ST_Y + i];
    }
    return SDV_OK;
}

int sdv_debug_force_commit_tree(sdv_ctx* ctx, const int32_t* host_path, int path_len, int32_t next_token) {
    if (!ctx || path_len < 0 || (path_len && !host_path)) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->verified || !ctx->tree_verified) return SDV_ESTATE;
    if (path_len + 1 > ctx->last_rows || next_token < 0 || next_token >= ctx->cfg.vocab) return SDV_EINVAL;
    for (int i = 0; i < path_len; ++i)
        if (host_path[i] < 1 || host_path[i] >= ctx->last_rows || (i && host_path[i] <= host_path[i - 1])) return SDV_EINVAL;
    DraftArg p;
    fill_draft_arg(p, host_path, path_len);
    set_path_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, p, next_token);
    ctx->launches++;
    CK(cudaGetLastError());
    return commit_common(ctx, 0, -1, 0, nullptr, nullptr, nullptr);
}

int sdv_commit(sdv_ctx* ctx, int max_emit, int32_t* host_emitted, int* n_emitted, int* kv_len) {
    if (!ctx) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->verified) return SDV_ESTATE;
    return commit_common(ctx, max_emit, -1, 0, host_emitted, n_emitted, kv_len);
}

int sdv_debug_force_commit(sdv_ctx* ctx, int accept_len, int32_t next_token) {
    if (!ctx) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->verified) return SDV_ESTATE;
    if (accept_len < 0 || accept_len + 1 > ctx->last_rows || next_token < 0 || next_token >= ctx->cfg.vocab)
        return SDV_EINVAL;
    return commit_common(ctx, 0, accept_len, next_token, nullptr, nullptr, nullptr);
}

int sdv_rollback(sdv_ctx* ctx, int new_kv_len) {
    if (!ctx) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (!ctx->prefill_done) return SDV_ESTATE;
    if (new_kv_len < 1 || new_kv_len > ctx->kv_len) return SDV_EINVAL;
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    ctx->kv_len = new_kv_len;
    ctx->hist_len = new_kv_len + 1;
    set_state_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, ctx->kv_len, ctx->hist_len, ctx->n_ctx, 1, hist);
    ctx->launches++;
    CK(cudaGetLastError());
    ctx->verified = false;
    ctx->draft_pending = false;
    ctx->tree_pending = false;
    ctx->tree_verified = false;
    CK(cudaStreamSynchronize(ctx->stream));
    return SDV_OK;
}

int sdv_get_logits(sdv_ctx* ctx, float* host_logits, int rows) {
    if (!ctx || !host_logits || rows < 1 || rows > kMaxRows) return SDV_EINVAL;
    if (!ctx->parity) return SDV_ESTATE;
    CK(cudaMemcpyAsync(host_logits, ctx->logits_src, (size_t)rows * ctx->cfg.vocab * 4, cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    return SDV_OK;
}

int sdv_step_bytes(const sdv_ctx* ctx, int rows, int kv_len, double* weight_bytes, double* kv_bytes) {
    if (!ctx || rows < 1) return SDV_EINVAL;
    const sdv_config& c = ctx->cfg;
    const double hd = c.head_dim, nq = c.n_q_heads * hd, nkv = c.n_kv_heads * hd, d = c.d_model, f = c.d_ffn;
    const double per_layer = (nq + 2 * nkv) * d + d * nq + 3 * d * f;
    if (weight_bytes) *weight_bytes = 2.0 * (c.n_layers * per_layer + (double)c.vocab * d);
    if (kv_bytes) *kv_bytes = (double)c.n_layers * 2.0 * nkv * 2.0 * ((double)kv_len + rows);
    return SDV_OK;
}

int sdv_last_verify_ms(sdv_ctx* ctx, float* ms) {
    if (!ctx || !ms) return SDV_EINVAL;
    if (!ctx->have_verify_time) return SDV_ESTATE;
    CK(cudaEventSynchronize(ctx->ev1));
    CK(cudaEventElapsedTime(ms, ctx->ev0, ctx->ev1));
    return SDV_OK;
}

// ------------------------------------------------------------------------------------------ debug
int sdv_debug_set_history(sdv_ctx* ctx, const int32_t* host_hist, int hist_len, int n_ctx) {
    if (!ctx || !host_hist || hist_len < 1 || n_ctx < 0 || n_ctx > hist_len) return SDV_EINVAL;
    if (hist_len > ctx->cfg.max_seq) return SDV_ECAPACITY;
    int* hist = (int*)(ctx->ws + ctx->r.hist);
    CK(cudaMemcpyAsync(hist, host_hist, (size_t)hist_len * 4, cudaMemcpyDefault, ctx->stream));
    ctx->hist_len = hist_len;
    ctx->kv_len = hist_len - 1;
    ctx->n_ctx = n_ctx;
    set_state_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, ctx->kv_len, ctx->hist_len, ctx->n_ctx, 1, hist);
    ctx->launches++;
    CK(cudaGetLastError());
    ctx->prefill_done = true;
    ctx->verified = false;
    ctx->draft_pending = false;
    ctx->tree_pending = false;
    ctx->tree_verified = false;
    CK(cudaStreamSynchronize(ctx->stream));
    return SDV_OK;
}

int sdv_debug_set_draft(sdv_ctx* ctx, const int32_t* host_draft, int draft_len) {
    if (!ctx || draft_len < 0 || draft_len > ctx->cfg.k_max || (draft_len && !host_draft)) return SDV_EINVAL;
    DraftArg a;
    fill_draft_arg(a, host_draft, draft_len);
    set_draft_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, a);
    ctx->launches++;
    CK(cudaGetLastError());
    ctx->draft_pending = true;
    ctx->tree_pending = false;
    ctx->draft_k = draft_len;
    ctx->verified = false;
    return SDV_OK;
}

int sdv_debug_accept(sdv_ctx* ctx, const int32_t* host_draft, int draft_len, const int32_t* host_y, int* accept_len) {
    if (!ctx || !host_y || draft_len < 0 || draft_len > ctx->cfg.k_max) return SDV_EINVAL;
    DraftArg a, y;
    fill_draft_arg(y, host_y, draft_len + 1);
    if (host_draft) {
        // host_draft == NULL: the draft already on the device (draft_len must be its length)
        fill_draft_arg(a, host_draft, draft_len);
        set_draft_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, a);
        ctx->launches++;
    }
    set_y_kernel<<<1, 32, 0, ctx->stream>>>(ctx->P.state, y);
    accept_kernel<<<1, 32 * (draft_len + 1), 0, ctx->stream>>>(ctx->P.state, ctx->P.cand_val, ctx->P.cand_idx, ctx->G, 1, 0, nullptr, 0);
    ctx->launches += 2;
    CK(cudaGetLastError());
    ctx->verified = true;
    ctx->last_rows = draft_len + 1;
    int rc = read_state(ctx);
    if (rc) return rc;
    if (accept_len) *accept_len = ctx->pinned[ST_ACCEPT_LEN];
    return SDV_OK;
}

int sdv_debug_top_successors(sdv_ctx* ctx, const float* host_logits, int rows, int top_b, int32_t* host_out) {
    if (!ctx || !host_logits || !host_out || rows < 1 || rows > kMaxRows || top_b < 1 || top_b > SDV_CALIB_MAX)
        return SDV_EINVAL;
    const size_t V = ctx->cfg.vocab;
    CK(cudaMemcpyAsync(ctx->ws + ctx->r.logits, host_logits, (size_t)rows * V * 4, cudaMemcpyDefault, ctx->stream));
    int* out = (int*)(ctx->ws + ctx->r.xstage);  // scratch of the stand-alone GEMM: at least 32 * d floats
    top_successors_kernel<<<rows, 1024, 0, ctx->stream>>>(ctx->P.logits, (int)V, top_b, out);
    ctx->launches++;
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(host_out, out, (size_t)rows * top_b * 4, cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    return SDV_OK;
}

int sdv_debug_read_kv(sdv_ctx* ctx, int layer, int which, int pos0, int n, float* host_out) {
    if (!ctx || !host_out || layer < 0 || layer >= ctx->cfg.n_layers || pos0 < 0 || n < 1 ||
        pos0 + n > ctx->cfg.max_seq)
        return SDV_EINVAL;
    const sdv_config& c = ctx->cfg;
    const size_t hd = c.head_dim;
    std::vector<uint16_t> tmp((size_t)n * hd);
    const uint8_t* base = ctx->ws + (which ? ctx->r.vcache : ctx->r.kcache);
    for (int a = 0; a < c.n_kv_heads; ++a) {
        const size_t off = (((size_t)layer * c.n_kv_heads + a) * c.max_seq + pos0) * hd * 2;
        CK(cudaMemcpyAsync(tmp.data(), base + off, tmp.size() * 2, cudaMemcpyDeviceToHost, ctx->stream));
        CK(cudaStreamSynchronize(ctx->stream));
        for (size_t i = 0; i < tmp.size(); ++i) {
            const uint32_t u = (uint32_t)tmp[i] << 16;
            memcpy(&host_out[(size_t)a * n * hd + i], &u, 4);
        }
    }
    return SDV_OK;
}

int sdv_debug_read_hidden(sdv_ctx* ctx, int rows, float* host_out) {
    if (!ctx || !host_out || rows < 1 || rows > kMaxRows) return SDV_EINVAL;
    CK(cudaMemcpyAsync(host_out, ctx->ws + ctx->r.h, (size_t)rows * ctx->cfg.d_model * 4, cudaMemcpyDeviceToHost,
                       ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    return SDV_OK;
}

int sdv_debug_gemm(sdv_ctx* ctx, const float* host_x, const uint16_t* host_w, float* host_y, int M, int N, int K,
                   float* dev_ms) {
    if (!ctx || !host_x || !host_w || !host_y) return SDV_EINVAL;
    if (ctx->poisoned) return SDV_ETIMEOUT;
    if (ctx->leader) return SDV_ESTATE;  // no staging areas without weight regions
    if (M < 1 || M > kMaxRows || N < 16 || N % 16 || K < 64 || K % 64) return SDV_EINVAL;
    if ((size_t)K > ctx->r.raw_kmax || (size_t)N * K * 2 > ctx->r.staging_bytes || (size_t)N > ctx->r.staging_bytes / 128)
        return SDV_EINVAL;
    const sdv_config& c = ctx->cfg;
    uint8_t* ws = ctx->ws;
    cudaStream_t s = ctx->stream;
    OpDesc o;
    memset(&o, 0, sizeof(o));
    o.T = N / 16;
    o.K16 = K / 16;
    choose_partition(o, ctx->G, M, false, false);
    fit_pass_width(o);
    CK(cudaMemcpyAsync(ws + ctx->r.staging, host_w, (size_t)N * K * 2, cudaMemcpyDefault, s));
    int rc = pack_op(ctx, o, ws + ctx->r.wraw, (const uint16_t*)(ws + ctx->r.staging), N, nullptr, 0, nullptr, K, 0, 0,
                     o.T, 0);
    if (rc) return rc;
    CK(cudaMemcpyAsync(ws + ctx->r.xstage, host_x, (size_t)M * K * 4, cudaMemcpyDefault, s));
    CK(cudaMemsetAsync(ws + ctx->r.raw_out, 0, (size_t)kMaxRows * N * 4, s));
    const OpDesc saved = ctx->P.op[OP_RAW];
    const int saved_N = ctx->P.raw_N, saved_K = ctx->P.raw_K;
    ctx->P.op[OP_RAW] = o;
    ctx->P.raw_N = N;
    ctx->P.raw_K = K;
    const int ph = 2 + kPhasesPerLayer * c.n_layers;
    rc = launch_forward(ctx, M, 0, 1, ph, ph + 1, true);
    ctx->P.op[OP_RAW] = saved;
    ctx->P.raw_N = saved_N;
    ctx->P.raw_K = saved_K;
    if (rc) return rc;
    CK(cudaMemcpyAsync(host_y, ws + ctx->r.raw_out, (size_t)M * N * 4, cudaMemcpyDeviceToHost, s));
    rc = read_state(ctx);
    if (rc) return rc;
    if (dev_ms) CK(cudaEventElapsedTime(dev_ms, ctx->ev0, ctx->ev1));
    return SDV_OK;
}

int sdv_debug_profile(sdv_ctx* ctx, int on, unsigned long long* host_out, int n_phases) {
    if (!ctx) return SDV_EINVAL;
    if (host_out) {
        if (n_phases < 1 || n_phases > 3 + kPhasesPerLayer * ctx->cfg.n_layers) return SDV_EINVAL;
        CK(cudaMemcpyAsync(host_out, ctx->ws + ctx->r.prof, (size_t)n_phases * ctx->G * kProfWords * 8, cudaMemcpyDeviceToHost,
                           ctx->stream));
        CK(cudaStreamSynchronize(ctx->stream));
    }
    if (on)
        CK(cudaMemsetAsync(ctx->ws + ctx->r.prof, 0,
                           (size_t)(3 + kPhasesPerLayer * ctx->cfg.n_layers) * kMaxGrid * kProfWords * 8, ctx->stream));
    ctx->profile = on ? 1 : 0;
    return ctx->G;
}

// Host-only self-check of the streaming layout: walks every block's share of an operation the way
// the weight streamer and the tensor-core thread do (pass by pass, stage by stage, the addresses the
// shared-memory descriptors generate) and checks that each 16-byte unit of the matrix is met exactly
// once, at the offset the packing function gives.  desc = {T, K16, P_row, P_k, RW, SK, unit, follow};
// gu_desc likewise (only read when follow is set).  Returns 0, or a negative code.
int sdv_debug_layout_check(const int* desc, const int* gu_desc, int G) {
    if (!desc || !gu_desc || G < 1) return SDV_EINVAL;
    OpDesc o, gu;
    memset(&o, 0, sizeof(o));
    memset(&gu, 0, sizeof(gu));
    o.T = desc[0]; o.K16 = desc[1]; o.P_row = desc[2]; o.P_k = desc[3]; o.RW = desc[4]; o.SK = desc[5]; o.unit = desc[6];
    o.follow = desc[7];
    gu.T = gu_desc[0]; gu.K16 = gu_desc[1]; gu.P_row = gu_desc[2]; gu.P_k = gu_desc[3]; gu.RW = gu_desc[4]; gu.SK = gu_desc[5];
    gu.unit = gu_desc[6];
    if (o.T < 1 || o.K16 < 1 || o.RW < 1 || o.SK < 1 || o.RW * o.SK * kStepBytes > kStageBytes || o.unit < 1 || o.T % o.unit) return SDV_EINVAL;
    const size_t units = (size_t)o.T * 16 * o.K16 * 2;  // 16-byte units of the matrix
    std::vector<unsigned char> seen(units, 0);
    for (int cta = 0; cta < G; ++cta) {
        const Part pt = get_part(o, gu, cta, G);
        if (pt.ntiles == 0 || pt.nk == 0) continue;
        unsigned long long src = pt.off;  // the streamer's running offset
        for (int p = 0; p < pt.npass; ++p) {
            const int pcount = pass_count(pt, p), pstart = pass_start(pt, p);
            if (pcount < 1 || pcount > 16) return -100;
            for (int st = 0; st < pt.nst; ++st) {
                const int nks = (pt.SK < pt.nk - st * pt.SK) ? pt.SK : pt.nk - st * pt.SK;
                const unsigned long long bytes = (unsigned long long)pcount * nks * kStepBytes;
                if (bytes > (unsigned long long)kStageBytes) return -101;
                const unsigned lbo = 2u * pcount * 128u, astep = 2u * lbo;
                for (int ks = 0; ks < nks; ++ks)
                    for (int half = 0; half < 2; ++half)
                        for (int r = 0; r < 16 * pcount; ++r) {
                            const unsigned long long in_slot = (unsigned long long)ks * astep + half * lbo + (r >> 3) * 128 + (r & 7) * 16;
                            if (in_slot + 16 > bytes) return -102;
                            const int row = (pt.tile0 + pstart) * 16 + r;
                            const int k8 = (pt.k0 + st * pt.SK + ks) * 2 + half;
                            const unsigned long long want = weight_offset(o, gu, row, k8);
                            if (want != src + in_slot) return -103;
                            const size_t u = want / 16;
                            if (u >= units || seen[u]) return -104;
                            seen[u] = 1;
                        }
                src += bytes;
            }
        }
    }
    for (size_t u = 0; u < units; ++u)
        if (!seen[u]) return -105;
    return 0;
}

// Host-only: the work partition and shared-memory plan a context of this configuration would use
// with G thread blocks and `rows` token rows.  out[op * 8 + {0..7}] = {T, K16, P_row, P_k, RW, SK,
// unit, follow} for the five operations (QKV, O, gate|up, down, LM head), then out[40..45] =
// {NG, NB, ring slots, operand region bytes, total dynamic shared memory, plan ok}.
int sdv_debug_plan(const sdv_config* cfg, int G, int rows, int* out) {
    if (!config_ok(cfg) || !out || G < 1 || G > kMaxGrid || rows < 1 || rows > kMaxRows) return SDV_EINVAL;
    FwdParams P;
    memset(&P, 0, sizeof(P));
    P.d = cfg->d_model;
    setup_ops(P, cfg, G);
    for (int i = 0; i < 5; ++i) {
        const OpDesc& o = P.op[i];
        const int v[8] = {o.T, o.K16, o.P_row, o.P_k, o.RW, o.SK, o.unit, o.follow};
        for (int j = 0; j < 8; ++j) out[i * 8 + j] = v[j];
    }
    const SmemPlan sp = plan_smem(P, rows, false);
    out[40] = sp.NG; out[41] = sp.NB; out[42] = sp.nstage; out[43] = sp.act_off - sp.u_off; out[44] = sp.total; out[45] = sp.ok ? 1 : 0;
    return SDV_OK;
}

int sdv_debug_timeout_probe(sdv_ctx* ctx) {
    if (!ctx) return SDV_EINVAL;
    timeout_probe_kernel<<<1, 1, 0, ctx->stream>>>(ctx->P.state, (const int*)(ctx->ws + ctx->r.never), 5000000ull);
    ctx->launches++;
    CK(cudaGetLastError());
    CK(cudaMemcpyAsync(ctx->pinned, ctx->ws + ctx->r.state, ST_WORDS * 4, cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    const int err = ctx->pinned[ST_ERR];
    CK(cudaMemsetAsync(ctx->P.state + ST_ERR, 0, 4, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    return err == 2 ? SDV_ETIMEOUT : SDV_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Stand-alone GEMM without any allocation (see include/sdv.h, sdv_gemm_noalloc).
//
// For callers that have no memory left to give or cannot afford the device-wide stall an
// allocation or a free brings (a serving loop whose memory is all KV cache, a plug-in with a fixed
// budget): nothing below asks the runtime for memory.  Its scratch memory is a fixed array in the library's device image.  Host code must not hand the
// array's name to a kernel (there it is only a host-side stand-in); the device address is looked
// up once per device with cudaGetSymbolAddress and passed on.
namespace {
constexpr size_t kNaWeightBytes = (size_t)2 << 20;              // packed weights: N * K * 2 <= 2 MiB
constexpr int kNaMaxK = 4096, kNaMaxN = 4096;
constexpr size_t kNaOutOff = kNaWeightBytes;                    // fp32 accumulators [32][N]
constexpr size_t kNaOutBytes = (size_t)kMaxRows * kNaMaxN * 4;
constexpr size_t kNaStateOff = kNaOutOff + kNaOutBytes;         // state words (error flag)
constexpr size_t kNaTotal = kNaStateOff + 1024;
constexpr int kNaMaxDevices = 64;
uint8_t* g_na_ptr[kNaMaxDevices];  // device address of the scratch array, per device (0 = not looked up yet)
}  // namespace

static __device__ __align__(256) uint8_t g_na_scratch[kNaTotal];  // ~2.5 MB per GPU that loads the library

extern "C" {

int sdv_gemm_noalloc(const float* dev_x, const uint16_t* dev_w, float* dev_y, int M, int N, int K, void* cuda_stream) {
    if (!dev_x || !dev_w || !dev_y) return SDV_EINVAL;
    if (M < 1 || N < 16 || N % 16 || K < 64 || K % 64) return SDV_EINVAL;
    if (M > kMaxRows || N > kNaMaxN || K > kNaMaxK || (size_t)N * K * 2 > kNaWeightBytes) return SDV_ETOOBIG;
    // the kernels read x and w with 16-byte vector loads
    if ((((uintptr_t)dev_x | (uintptr_t)dev_w) & 15) || ((uintptr_t)dev_y & 3)) return SDV_EINVAL;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kNaMaxDevices) return SDV_ECUDA;
    {
        // host memory or another device's memory would fault inside the kernel: refuse it here
        const void* ptrs[3] = {dev_x, dev_w, dev_y};
        for (int i = 0; i < 3; ++i) {
            cudaPointerAttributes at;
            if (cudaPointerGetAttributes(&at, ptrs[i]) != cudaSuccess) {
                cudaGetLastError();
                return SDV_EINVAL;
            }
            if (at.type == cudaMemoryTypeManaged) continue;
            if (at.type != cudaMemoryTypeDevice || at.device != dev) return SDV_EINVAL;
        }
    }
    if (!g_na_ptr[dev]) {
        // first call on this device: look the array's device address up (do this before any stream capture)
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_na_scratch) != cudaSuccess || !p) return SDV_ECUDA;
        g_na_ptr[dev] = (uint8_t*)p;
    }
    uint8_t* sc = g_na_ptr[dev];
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return SDV_ECUDA;
    if (sms > kMaxGrid) sms = kMaxGrid;

    FwdParams P;
    memset(&P, 0, sizeof(P));
    P.G = sms;
    OpDesc& o = P.op[OP_RAW];
    o.T = N / 16;
    o.K16 = K / 16;
    choose_partition(o, sms, M, false, false);
    fit_pass_width(o);
    P.wraw = sc;
    P.raw_x = dev_x;  // the caller's rows are read in place
    P.raw_out = (float*)(sc + kNaOutOff);
    P.raw_N = N;
    P.raw_K = K;
    P.state = (int*)(sc + kNaStateOff);
    P.bar = (unsigned*)(P.state + 200);  // unused by a one-phase launch, kept inside the cleared words
    P.mode = 1;
    P.ph_begin = 2;  // with n_layers = 0 phase 2 is the stand-alone GEMM
    P.ph_end = 3;
    P.wait_limit_ns = 2000000000ull;
    int smem_bytes = 0;
    if (!apply_plan(P, M, true, &smem_bytes)) return SDV_EINVAL;

    // the array keeps the previous call's contents: clear what must start at zero
    if (cudaMemsetAsync(sc + kNaOutOff, 0, (size_t)kMaxRows * N * 4, s) != cudaSuccess) return SDV_ECUDA;
    if (cudaMemsetAsync(sc + kNaStateOff, 0, 1024, s) != cudaSuccess) return SDV_ECUDA;
    const long long total = (long long)o.T * 16 * (K / 8);
    int blocks = (int)((total + 255) / 256);
    if (blocks > 148 * 16) blocks = 148 * 16;
    pack_weights_kernel<<<blocks, 256, 0, s>>>(o, o, sc, dev_w, N, nullptr, 0, nullptr, K, 0, 0, o.T, 0);
    if (cudaGetLastError() != cudaSuccess) return SDV_ECUDA;
    if (launch_kernel(P, smem_bytes, s) != cudaSuccess) return SDV_ECUDA;
    if (cudaMemcpyAsync(dev_y, sc + kNaOutOff, (size_t)M * N * 4, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return SDV_ECUDA;
    int err = 0;
    if (cudaMemcpyAsync(&err, sc + kNaStateOff + ST_ERR * 4, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return SDV_ECUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return SDV_ECUDA;
    return err ? SDV_ETIMEOUT : SDV_OK;
}

}  // extern "C"
