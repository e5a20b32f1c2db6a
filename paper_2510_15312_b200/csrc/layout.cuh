// Shapes, buffer pointers and the static work partition shared by host code and kernels.
//
// Weight streaming layout.  Every linear layer W[N][K] (bf16) is seen as a grid of T = N/16 row
// tiles by K16 = K/16 column steps (one step = the 16 input features of one tensor-core
// instruction).  The grid is split into P_row x P_k rectangular partitions, one per thread
// block.  A block walks its partition in passes of at most RW row tiles (RW <= 16: one pass is
// one or two 128-row accumulators in tensor memory, rows past the pass are don't-care) and, inside a
// pass, in stages of at most SK column steps (RW * SK <= 64, i.e. <= 32 KB).  A stage is stored
// as the shared-memory image the tensor core reads: column step by column step, the two
// 8-column halves of a step one after the other, each a run of 8-row x 16-byte core matrices
//     [step][half][8-row group][row][8 bf16]
// with no padding.  Stages follow each other pass by pass, so every stage is one contiguous
// bulk copy and a block's whole share of an operation is one contiguous byte range.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace sdv {

constexpr int kWorkerWarps = 11;                       // every warp but the weight streamer
constexpr int kWorkerThreads = kWorkerWarps * 32;      // 352
constexpr int kThreads = kWorkerThreads + 32;          // 384 with the weight-streaming warp
constexpr int kBuilderWarps = 10;                      // warps 0..9 build the token operand of a GEMM
constexpr int kEpilogueWarps = 8;                      // warps 0..7 read the accumulators: warp w lanes 32(w%4)..+31 of accumulator w/4
constexpr int kMmaWarp = 10;                           // its lane 0 issues the tensor-core instructions
constexpr int kProducerWarp = 11;
constexpr int kStepBytes = 512;                        // one row tile x one column step: 16 x 16 bf16
constexpr int kStageBytes = 32768;                     // ring slot
constexpr int kMaxStages = 8;                          // ring slots at most
constexpr int kMaxRows = 32;                           // token rows a buffer is sized for
constexpr int kMaxBatch = 8;                           // sequences one batched verify step takes at most
constexpr int kMaxSplits = 19;                         // KV key ranges per head (+1 partial result for the new rows)
constexpr int kSmemBudget = 232448;                    // 227 KB
constexpr int kAttnSmemBytes = 81920;                  // Q tile (up to 16 KB) + two K|V blocks of 64 keys (64 KB)
constexpr int kActSmemMax = 32768;                     // SwiGLU output of this block (operand of its down-projection slice) at most
constexpr int kMiscSmemBytes = 4096;
constexpr int kMaxDraftWords = 32;
constexpr int kProfWords = 12;                         // timestamps per (phase, block)
constexpr int kTmemCols = 128;                         // two buffers of two 128-row accumulators of up to 32 fp32 columns

enum OpIndex { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_DOWN = 3, OP_LM = 4, OP_RAW = 5, OP_COUNT = 6 };

struct OpDesc {
    int T;       // row tiles (16 weight rows each)
    int K16;     // column steps (16 input features each)
    int P_row;   // partitions along rows
    int P_k;     // partitions along columns (> 1: partial sums meet by reductions in L2)
    int rot;     // block index that owns partition 0 (spreads idle blocks over operations)
    int RW;      // row tiles per pass at most (16, 8, 4, 2 or 1)
    int SK;      // column steps per stage at most (RW * SK <= 64)
    int unit;    // row partitions are multiples of this many tiles (2 for gate|up: 16 SwiGLU columns)
    int follow;  // 1: one row partition; block i takes the columns that partition i of `gate|up` produces
    int pad;
    unsigned long long w_off;  // byte offset of the operation inside its weight region
};

struct Part {
    int tile0, ntiles, k0, nk, pr, pk;
    unsigned long long off;  // byte offset of this partition from the operation's base
    int npass, nst;          // passes over the row tiles; stages per pass
    int pbase, prem;         // tiles per pass: pbase + (p < prem)
    int SK, pad;
};
__host__ __device__ inline int pass_count(const Part& p, int i) { return p.pbase + (i < p.prem ? 1 : 0); }
__host__ __device__ inline int pass_start(const Part& p, int i) { return i * p.pbase + (i < p.prem ? i : p.prem); }

__host__ __device__ inline int even_start(int total, int parts, int i) {
    const int b = total / parts, r = total % parts;
    return i * b + (i < r ? i : r);
}
__host__ __device__ inline int even_count(int total, int parts, int i) {
    return total / parts + (i < total % parts ? 1 : 0);
}
// Inverse of even_start: which part holds element x.
__host__ __device__ inline int even_find(int total, int parts, int x) {
    const int b = total / parts, r = total % parts;
    if (x < r * (b + 1)) return x / (b + 1);
    return r + (x - r * (b + 1)) / b;
}

__host__ __device__ inline void finish_part(Part& p, const OpDesc& o) {
    p.off = (unsigned long long)kStepBytes *
            ((unsigned long long)p.tile0 * o.K16 + (unsigned long long)p.ntiles * p.k0);
    p.SK = o.SK;
    p.npass = (p.ntiles + o.RW - 1) / o.RW;
    p.nst = (p.nk + o.SK - 1) / o.SK;
    p.pbase = p.npass ? p.ntiles / p.npass : 0;
    p.prem = p.npass ? p.ntiles % p.npass : 0;
}

// Partition (pr, pk) of an operation; `gu` is the gate|up operation (used when o.follow).
__host__ __device__ inline Part make_part(const OpDesc& o, const OpDesc& gu, int pr, int pk) {
    Part p;
    p.pr = pr;
    p.pk = pk;
    p.pad = 0;
    if (o.follow) {
        p.tile0 = 0;
        p.ntiles = o.T;
        p.k0 = even_start(gu.T / gu.unit, gu.P_row, pk);
        p.nk = even_count(gu.T / gu.unit, gu.P_row, pk);
    } else {
        p.tile0 = o.unit * even_start(o.T / o.unit, o.P_row, pr);
        p.ntiles = o.unit * even_count(o.T / o.unit, o.P_row, pr);
        p.k0 = even_start(o.K16, o.P_k, pk);
        p.nk = even_count(o.K16, o.P_k, pk);
    }
    finish_part(p, o);
    return p;
}

__host__ __device__ inline Part get_part(const OpDesc& o, const OpDesc& gu, int cta, int G) {
    const int rot = o.follow ? gu.rot : o.rot;
    const int nparts = o.follow ? gu.P_row : o.P_row * o.P_k;
    int idx = cta - rot;
    if (idx < 0) idx += G;
    if (idx >= nparts) {
        Part p;
        p.tile0 = p.ntiles = p.k0 = p.nk = p.pr = p.pk = p.npass = p.nst = p.pbase = p.prem = p.pad = 0;
        p.SK = o.SK;
        p.off = 0;
        return p;
    }
    if (o.follow) return make_part(o, gu, 0, idx);
    return make_part(o, gu, idx / o.P_k, idx % o.P_k);
}

// Byte offset (from the operation's base) of the 16-byte unit holding columns 8*k8 .. 8*k8+7 of
// weight row `row`: the inverse view used when packing.
__host__ __device__ inline unsigned long long weight_offset(const OpDesc& o, const OpDesc& gu, int row, int k8) {
    const int t = row >> 4, ks = k8 >> 1, half = k8 & 1;
    int pr, pk;
    if (o.follow) {
        pr = 0;
        pk = even_find(gu.T / gu.unit, gu.P_row, ks);
    } else {
        pr = even_find(o.T / o.unit, o.P_row, t / o.unit);
        pk = even_find(o.K16, o.P_k, ks);
    }
    const Part p = make_part(o, gu, pr, pk);
    const int lt = t - p.tile0;
    const int pass = even_find(p.ntiles, p.npass, lt);
    const int start = pass_start(p, pass), pcount = pass_count(p, pass);
    const int tip = lt - start, lk = ks - p.k0;
    const int st = lk / p.SK, kin = lk % p.SK;
    const unsigned long long stage_base =
        p.off + (unsigned long long)kStepBytes * ((unsigned long long)start * p.nk + (unsigned long long)pcount * st * p.SK);
    const unsigned long long in_stage =
        ((unsigned long long)(kin * 2 + half) * (2 * pcount) + (tip * 2 + ((row & 15) >> 3))) * 128 + (row & 7) * 16;
    return stage_base + in_stage;
}

// Device state block (int32 words).
enum StateWord {
    ST_KV_LEN = 0, ST_HIST_LEN, ST_N_CTX, ST_PENDING, ST_DRAFT_LEN, ST_ACCEPT_LEN, ST_N_EMITTED, ST_ERR,
    ST_VERIFIED,      // 1 when a verify result awaits commit
    ST_MATCH_POS, ST_MATCH_LEN,
    ST_SEG_LEN,       // retained segment of rejected drafts (draft extension): tokens,
    ST_SEG_LIFE,      //   verify steps it has been appended to,
    ST_SEG_USED,      //   1 while it is part of the draft under verification,
    ST_BASE_LEN,      //   and that draft's length before it was appended
    ST_DB_LEN,        // tokens in the extra token database the drafter also searches (0: none)
    ST_DRAFT = 16,    // [32]
    ST_Y = 48,        // [33]
    ST_TREE_ON = 82,  // 1: the draft is a tree (ST_PARENT .. ST_ANC hold its shape), 0: a chain
    ST_PATH_LEN = 83, // nodes on the accepted path of the last tree verify
    ST_BUDGET = 84,   // tokens a run of enqueued steps may still emit (-1: no limit; 0: the remaining steps do nothing)
    ST_EMITTED = 96,  // [33]
    ST_SEG = 160,     // [32]
    ST_PARENT = 192,  // [32] row that row j continues (row 0 = the committed token; draft node i is row i)
    ST_DEPTH = 224,   // [32] distance of row j from the root = its position minus the KV length
    ST_ANC = 256,     // [32] bit r set: row r lies on row j's path from the root (j itself included)
    ST_PATH = 288,    // [32] accepted path (rows), root excluded
    ST_WORDS = 320
};

// One sequence of a batched verify step: its rows [r0, r0 + M) of the launch, its committed length
// and its own KV cache.
struct BatchSeq {
    __nv_bfloat16* kcache;
    __nv_bfloat16* vcache;
    int r0, M, L, pad;
};

struct FwdParams {
    // model
    int n_layers, d, n_q, n_kv, hd, f, V, max_seq, g, n_qkv;
    float eps, scale_log2e;  // softmax scale 1/sqrt(hd) times log2(e)
    int G;                   // thread blocks in the grid
    OpDesc op[OP_COUNT];
    unsigned long long layer_stride;  // bytes of streamed weights per layer
    const uint8_t* wlayers;           // streamed weights of layer 0 (qkv, o, gate|up, down)
    const uint8_t* wlm;               // streamed LM head
    const uint8_t* wraw;              // streamed matrix of the stand-alone GEMM entry point
    const __nv_bfloat16* emb;         // [V][d] row-major (embedding gather)
    const float* norm_w;              // [n_layers][2][d], then the final norm [d]
    const float* bias;                // [n_layers][n_qkv] or nullptr
    const float2* rope;               // [max_seq][hd/2] (cos, sin)
    __nv_bfloat16* kcache;            // [layer][kv head][max_seq][hd]
    __nv_bfloat16* vcache;
    // activations (global, L2 resident)
    float* h;          // [kMaxRows][d] residual stream
    float* qkv_acc;    // [kMaxRows][n_qkv] un-normalised q|k|v sums
    float* sumsq;      // [2][kMaxRows] sum of squares of h rows for the attention-side norm
    float* part_o;     // [n_q][kMaxSplits+1][kMaxRows][hd] un-normalised split outputs
    float* part_ml;    // [n_q][kMaxSplits+1][kMaxRows][2]  (running max in log2 units, sum)
    float* cand_val;   // [G][kMaxRows] per-block best logit
    int* cand_idx;     // [G][kMaxRows] and its token id
    float* logits;     // [kMaxRows][V]
    const float* raw_x;  // [M][raw_K] operand of the stand-alone GEMM
    float* raw_out;    // [kMaxRows][raw_N] output of the stand-alone GEMM
    int raw_N, raw_K;
    int* state;
    const int* hist;
    unsigned* bar;     // grid barrier counter (wraps round; only differences are compared)
    unsigned long long* prof;  // optional [phase][block][kProfWords] timestamps (ns)
    // per launch
    int L;             // committed KV length = position of row 0
    int M;             // rows computed (1..kMaxRows)
    int NB;            // N of the tensor-core instruction: 16, or 32 when M > 16
    int att_gh;        // attention split: query heads per unit (the key ranges follow from it)
    int att_S, att_kps;  // key ranges and keys per range: derived from L and att_gh by the kernel when it starts
    int att_QG, att_per_seq;            // head groups per KV head; attention units per sequence
    int att_b0, att_hk0, att_qg0, att_s0;  // the block's first attention unit, decoded (each block works this out for itself)
    int mode;          // 0: rows are [pending, draft...]; 1: rows are hist[L..L+M)
    int ph_begin, ph_end;
    unsigned bar_base; // barrier counter value before this launch
    int store_logits;
    int tree;          // 1: the rows form a tree (positions, masks from the state block), 0: a chain
    // shared-memory plan of this launch (bytes from the 1024-aligned base)
    int nstage;        // ring slots of kStageBytes, at offset 0
    int u_off;         // operand region (token operand of the running GEMM; attention tiles)
    int act_off;       // SwiGLU output operand
    int misc_off;
    unsigned long long wait_limit_ns;
    int l_from_state;  // 1: L is read from the state block when the kernel starts (steps enqueued without the host in between)
    // batched verify: nseq > 0 sequences share the launch (chains only); L is then the longest length
    int nseq;
    BatchSeq seq[kMaxBatch];
};

}  // namespace sdv
