// Shapes, buffer pointers and the static work partition shared by host code and kernels.
//
// Weight streaming layout.  Every linear layer W[N][K] (bf16) is cut into tiles of 16 rows x 64
// columns (2 KB, 128-byte rows with XOR-swizzled 16-byte units).  An operation's tile grid
// (T = N/16 row tiles, C = K/64 column chunks) is split into P_row x P_k rectangular
// partitions, one per thread block.  The block's 8 MMA warps form an RW x KW grid (RW * KW = 8):
// it walks its partition in passes of at most RW row tiles and, inside a pass, in stages of KW
// consecutive chunks, so one stage is RW x KW tiles (<= 16 KB), one per warp.  Tiles are stored
// pass by pass, chunk by chunk, tile by tile: every stage is one contiguous bulk copy and a
// block's whole share of an operation is one contiguous byte range.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace sdv {

constexpr int kConsumerWarps = 8;
constexpr int kLoaderWarps = 3;
constexpr int kWorkerThreads = (kConsumerWarps + kLoaderWarps) * 32;  // 352: every warp but the producer
constexpr int kThreads = kWorkerThreads + 32;                        // 384 with the weight-streaming warp
constexpr int kTileBytes = 2048;                                     // 16 rows x 64 cols bf16
constexpr int kStageWeightBytes = kConsumerWarps * kTileBytes;       // 16 KB
constexpr int kMaxRows = 32;                                         // token rows a buffer is sized for
constexpr int kMaxSplits = 40;                                       // KV splits per head (+1 unit for new rows)
constexpr int kMaxKW = 4;                                             // chunks per stage at most
constexpr int kSmemBudget = 232448;                                  // 227 KB
constexpr int kAttnSmemBytes = 49152 + 4096;                         // Q tile + K and V blocks (48 KB), row statistics
constexpr int kMiscSmemBytes = 4096;
constexpr int kMaxDraftWords = 32;
constexpr int kProfWords = 12;                                       // timestamps per (phase, block)

enum OpIndex { OP_QKV = 0, OP_O = 1, OP_GU = 2, OP_DOWN = 3, OP_LM = 4, OP_RAW = 5, OP_COUNT = 6 };

struct OpDesc {
    int T;       // row tiles (16 weight rows each)
    int C;       // column chunks (64 input features each)
    int P_row;   // partitions along rows
    int P_k;     // partitions along columns (> 1: partial sums meet by atomic adds)
    int rot;     // block index that owns partition 0 (spreads idle blocks over operations)
    int RW;      // row tiles per pass (8, 4 or 2); KW = 8 / RW chunks per stage
    unsigned long long w_off;  // byte offset of the operation inside its weight region
};

struct Part {
    int tile0, ntiles, chunk0, nchunks, pr, pk;
    unsigned long long off;  // byte offset of this partition from the operation's base
    // derived once per launch so that the per-stage code needs no integer division
    int npass, nst;          // passes over the row tiles; stages (groups of KW chunks) per pass
    int pbase, prem;         // tiles per pass: pbase + (p < prem)
    int lkw;                 // log2(KW)
    int pad;
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

__host__ __device__ inline Part get_part(const OpDesc& o, int cta, int G) {
    Part p;
    int idx = cta - o.rot;
    if (idx < 0) idx += G;
    p.npass = p.nst = p.pbase = p.prem = p.lkw = p.pad = 0;
    if (idx >= o.P_row * o.P_k) {
        p.tile0 = p.ntiles = p.chunk0 = p.nchunks = p.pr = p.pk = 0;
        p.off = 0;
        return p;
    }
    p.pr = idx / o.P_k;
    p.pk = idx % o.P_k;
    p.tile0 = even_start(o.T, o.P_row, p.pr);
    p.ntiles = even_count(o.T, o.P_row, p.pr);
    p.chunk0 = even_start(o.C, o.P_k, p.pk);
    p.nchunks = even_count(o.C, o.P_k, p.pk);
    p.off = (unsigned long long)kTileBytes *
            ((unsigned long long)p.tile0 * o.C + (unsigned long long)p.ntiles * p.chunk0);
    const int KW = kConsumerWarps / o.RW;
    p.lkw = KW == 4 ? 2 : (KW == 2 ? 1 : 0);
    p.npass = (p.ntiles + o.RW - 1) / o.RW;
    p.nst = (p.nchunks + KW - 1) / KW;
    p.pbase = p.ntiles / p.npass;
    p.prem = p.ntiles % p.npass;
    return p;
}
__host__ __device__ inline int part_passes(const Part& p, int RW) { return (p.ntiles + RW - 1) / RW; }

// Byte offset (from the operation's base) of tile t, chunk c: the inverse view used when packing.
__host__ __device__ inline unsigned long long tile_offset(const OpDesc& o, int t, int c) {
    const int pr = even_find(o.T, o.P_row, t), pk = even_find(o.C, o.P_k, c);
    const int tile0 = even_start(o.T, o.P_row, pr), ntiles = even_count(o.T, o.P_row, pr);
    const int chunk0 = even_start(o.C, o.P_k, pk), nchunks = even_count(o.C, o.P_k, pk);
    const int npass = (ntiles + o.RW - 1) / o.RW;
    const int lt = t - tile0;
    const int p = even_find(ntiles, npass, lt);
    const int start = even_start(ntiles, npass, p), cnt = even_count(ntiles, npass, p);
    const unsigned long long tiles_before = (unsigned long long)tile0 * o.C + (unsigned long long)ntiles * chunk0 +
                                            (unsigned long long)start * nchunks +
                                            (unsigned long long)cnt * (c - chunk0) + (lt - start);
    return tiles_before * kTileBytes;
}

// Device state block (int32 words).
enum StateWord {
    ST_KV_LEN = 0, ST_HIST_LEN, ST_N_CTX, ST_PENDING, ST_DRAFT_LEN, ST_ACCEPT_LEN, ST_N_EMITTED, ST_ERR,
    ST_VERIFIED,      // 1 when a verify result awaits commit
    ST_MATCH_POS, ST_MATCH_LEN,
    ST_DRAFT = 16,    // [32]
    ST_Y = 48,        // [33]
    ST_EMITTED = 96,  // [33]
    ST_WORDS = 160
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
    uint8_t* act;      // bf16 [f/64][rows][64] swizzled: SwiGLU output, the down projection's operand
    uint8_t* attn_op;  // bf16 [n_q*hd/64][rows][64] swizzled: attention output, the o projection's operand
    float* part_o;     // [n_q][kMaxSplits+1][kMaxRows][hd] un-normalised split outputs
    float* part_ml;    // [n_q][kMaxSplits+1][kMaxRows][2]  (running max in log2 units, sum)
    float* cand_val;   // [G][kMaxRows] per-block best logit
    int* cand_idx;     // [G][kMaxRows] and its token id
    float* logits;     // [kMaxRows][V]
    float* raw_out;    // [kMaxRows][raw_N] output of the stand-alone GEMM
    int raw_N;
    int* state;
    const int* hist;
    int* bar;          // grid barrier counter
    unsigned long long* prof;  // optional [phase][block][kProfWords] timestamps (ns)
    // per launch
    int L;             // committed KV length = position of row 0
    int M;             // rows computed (1..8*NT)
    int mode;          // 0: rows are [pending, draft...]; 1: rows are hist[L..L+M)
    int ph_begin, ph_end;
    int bar_base;      // barrier counter value before this launch
    int store_logits;
    int ahead;         // weight stages the streamer may run ahead of the MMA warps (<= ring size)
    unsigned long long wait_limit_ns;
};

}  // namespace sdv
