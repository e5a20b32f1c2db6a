// The integer kernels of the path (n-gram drafter, accept scan, commit) and set-up helpers
// (weight re-layout, fills).
#pragma once
#include <math_constants.h>

#include "layout.cuh"
#include "ptx.cuh"

namespace sdv {

// ------------------------------------------------------------------------------------------
// Weight re-layout: row-major bf16 [rows][K] -> streaming order (see layout.cuh).  One thread per
// 16-byte unit (8 columns of one row).
// mode 0: the operation's rows are src0 | src1 | src2 stacked (the sources hold the rows from
// row_base on); mode 1: every 16-row tile holds 8 rows of src0 (gate) followed by the 8 matching
// rows of src1 (up).  Only tiles [t_begin, t_end) are written.
__global__ void pack_weights_kernel(OpDesc o, OpDesc gu, uint8_t* dst_base, const uint16_t* src0, int rows0,
                                    const uint16_t* src1, int rows1, const uint16_t* src2, int K, int mode,
                                    int t_begin, int t_end, int row_base) {
    const int K8 = K / 8;
    const long long total = (long long)(t_end - t_begin) * 16 * K8;
    for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < total;
         u += (long long)gridDim.x * blockDim.x) {
        const int k8 = (int)(u % K8);
        const int row = t_begin * 16 + (int)(u / K8);  // row of the operation
        const int t = row >> 4, r = row & 15;
        const uint16_t* src;
        if (mode == 1) {
            src = (r < 8) ? src0 + (size_t)(8 * t + r) * K : src1 + (size_t)(8 * t + r - 8) * K;
        } else {
            const int lr = row - row_base;
            if (lr < rows0) src = src0 + (size_t)lr * K;
            else if (lr < rows0 + rows1) src = src1 + (size_t)(lr - rows0) * K;
            else src = src2 + (size_t)(lr - rows0 - rows1) * K;
        }
        const uint4 v = *reinterpret_cast<const uint4*>(src + k8 * 8);
        *reinterpret_cast<uint4*>(dst_base + weight_offset(o, gu, row, k8)) = v;
    }
}

__global__ void fill_f32_kernel(float* p, float v, long long n) {
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        p[i] = v;
}
__global__ void fill_i32_kernel(int* p, int v, long long n) {
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x)
        p[i] = v;
}

// ------------------------------------------------------------------------------------------
// Retrieval drafter.  One block; thread p tests search position p: the length m(p) of the common
// suffix of search[0..p] and the history (capped at n), then a block-wide maximum of (m(p), p)
// picks the longest and, among those, the latest match; up to k following tokens are the draft.
// The search array is the history's own prefix: the request context (first n_ctx tokens), or,
// with search_history, everything but the last token (the suffix must not match itself).  A second
// array, the extra token database, is searched the same way; an equally long match in the request's
// own text wins over one in the database (bit 32 of the key).  ST_MATCH_POS reports a database
// position p as -(p + 2).
__device__ __forceinline__ unsigned long long suffix_scan(const int* search, int n_search, int exclude_from,
                                                          const int* hist, int hist_len, int n, int n_min,
                                                          unsigned long long src_bit) {
    unsigned long long best = 0;
    for (int p = threadIdx.x; p + 1 < n_search && p < exclude_from; p += blockDim.x) {
        int cap = n;
        if (p + 1 < cap) cap = p + 1;
        if (hist_len < cap) cap = hist_len;
        int mlen = 0;
        while (mlen < cap && search[p - mlen] == hist[hist_len - 1 - mlen]) ++mlen;
        if (mlen >= n_min && mlen > 0) {
            const unsigned long long key = ((unsigned long long)mlen << 33) | src_bit | (unsigned)p;
            if (key > best) best = key;
        }
    }
    return best;
}

// `in_run` (all kernels of a step): the step was enqueued as part of a run with a token budget and does nothing
// once the budget is used up.
__device__ __forceinline__ void ngram_draft_body(int* state, const int* hist, const int* db, int n, int n_min, int k,
                                                 int search_history) {
    __shared__ unsigned long long best_s[32];
    const int hist_len = state[ST_HIST_LEN];
    const int n_search = search_history ? hist_len : state[ST_N_CTX];
    const int exclude_from = search_history ? hist_len - 1 : n_search;
    const int db_len = state[ST_DB_LEN];
    unsigned long long best = suffix_scan(hist, n_search, exclude_from, hist, hist_len, n, n_min, 1ull << 32);
    if (db_len > 1) {
        const unsigned long long b2 = suffix_scan(db, db_len, db_len, hist, hist_len, n, n_min, 0ull);
        if (b2 > best) best = b2;
    }
    for (int off = 16; off; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, off);
        if (o > best) best = o;
    }
    if ((threadIdx.x & 31) == 0) best_s[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x < 32) {
        best = (threadIdx.x < (blockDim.x >> 5)) ? best_s[threadIdx.x] : 0ull;
        for (int off = 16; off; off >>= 1) {
            const unsigned long long o = __shfl_xor_sync(0xffffffffu, best, off);
            if (o > best) best = o;
        }
        int dl = 0, pos = -1, mlen = 0;
        if (best != 0) {
            const bool own = ((best >> 32) & 1ull) != 0;
            const int* src = own ? hist : db;
            const int n_src = own ? n_search : db_len;
            const int p = (int)(best & 0xffffffffu);
            mlen = (int)(best >> 33);
            pos = own ? p : -(p + 2);
            dl = n_src - 1 - p;
            if (dl > k) dl = k;
            if ((int)threadIdx.x < dl) state[ST_DRAFT + threadIdx.x] = src[p + 1 + threadIdx.x];
        }
        if (threadIdx.x == 0) {
            state[ST_DRAFT_LEN] = dl;
            state[ST_BASE_LEN] = dl;
            state[ST_SEG_USED] = 0;
            state[ST_MATCH_POS] = pos;
            state[ST_MATCH_LEN] = mlen;
            state[ST_TREE_ON] = 0;
        }
    }
}
__global__ void ngram_draft_kernel(int* state, const int* hist, const int* db, int n, int n_min, int k,
                                   int search_history, int in_run) {
    if (in_run && state[ST_BUDGET] == 0) return;
    ngram_draft_body(state, hist, db, n, n_min, k, search_history);
}

__global__ void set_word_kernel(int* state, int word, int value) {
    if (threadIdx.x == 0) state[word] = value;
}

struct DraftArg {
    int n;
    int tok[kMaxDraftWords];
};

// Caller-supplied drafts (by value: no host buffer has to outlive the call).
__global__ void set_draft_kernel(int* state, DraftArg a) {
    if ((int)threadIdx.x < a.n) state[ST_DRAFT + threadIdx.x] = a.tok[threadIdx.x];
    if (threadIdx.x == 0) {
        state[ST_DRAFT_LEN] = a.n;
        state[ST_BASE_LEN] = a.n;
        state[ST_SEG_USED] = 0;
        state[ST_TREE_ON] = 0;
    }
}

// ------------------------------------------------------------------------------------------
// Tree-structured drafts.  Row 0 is the committed token, draft node i is row i; ST_PARENT[i] < i is
// the row it continues.  One thread derives what the forward pass reads: the depth of every row
// (its position relative to the KV length) and the bit mask of the rows on its path from the root.
// Rows past the tree (padding up to the launch's row count) hang off the root on their own.
__device__ __forceinline__ void tree_finish(int* state, int n_nodes) {
    state[ST_PARENT] = -1;
    state[ST_DEPTH] = 0;
    state[ST_ANC] = 1;
    for (int j = 1; j < kMaxRows; ++j) {
        int par = (j <= n_nodes) ? state[ST_PARENT + j] : 0;
        if (par < 0 || par >= j) par = 0;
        state[ST_PARENT + j] = par;
        state[ST_DEPTH + j] = state[ST_DEPTH + par] + 1;
        state[ST_ANC + j] = state[ST_ANC + par] | (int)(1u << j);
    }
    state[ST_TREE_ON] = 1;
}

// Caller-supplied tree: tokens of the draft nodes and, for node i (1-based), the row it continues.
__global__ void set_tree_kernel(int* state, DraftArg tok, DraftArg par) {
    if ((int)threadIdx.x < tok.n) {
        state[ST_DRAFT + threadIdx.x] = tok.tok[threadIdx.x];
        state[ST_PARENT + 1 + threadIdx.x] = par.tok[threadIdx.x];
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        state[ST_DRAFT_LEN] = tok.n;
        state[ST_BASE_LEN] = tok.n;
        state[ST_SEG_USED] = 0;
        tree_finish(state, tok.n);
    }
}

// In-context calibration, "Sample": the b best token ids of every logits row (largest logit first,
// lowest id among equals: the greedy rule applied b times).  One block per row.
__global__ void top_successors_kernel(const float* logits, int V, int b, int* succ /* [rows][b] */) {
    __shared__ float bv_s[32];
    __shared__ int bi_s[32];
    __shared__ int taken[8];
    const float* row = logits + (size_t)blockIdx.x * V;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    for (int r = 0; r < b; ++r) {
        float bv = -CUDART_INF_F;
        int bi = 0x7fffffff;
        for (int i = threadIdx.x; i < V; i += blockDim.x) {
            bool skip = false;
            for (int t = 0; t < r; ++t) skip |= (taken[t] == i);
            const float v = row[i];
            if (!skip && (v > bv || (v == bv && i < bi))) { bv = v; bi = i; }
        }
        for (int off = 16; off; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        if (lane == 0) { bv_s[warp] = bv; bi_s[warp] = bi; }
        __syncthreads();
        if (warp == 0) {
            bv = lane < nw ? bv_s[lane] : -CUDART_INF_F;
            bi = lane < nw ? bi_s[lane] : 0x7fffffff;
            for (int off = 16; off; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (lane == 0) {
                if (bi == 0x7fffffff) bi = 0;
                taken[r] = bi;
                succ[(size_t)blockIdx.x * b + r] = bi;
            }
        }
        __syncthreads();
    }
}

// "Search": where in the context each sampled successor occurs (the latest position; -1: nowhere).
__global__ void anchor_search_kernel(const int* hist, int n_ctx, int b, const int* succ, int* occ) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= n_ctx * b) return;
    const int tok = succ[idx];
    int q = n_ctx - 1;
    while (q >= 0 && hist[q] != tok) --q;
    occ[idx] = q;
}

// Tree draft of one step: the retrieval chain the drafter left in the state block becomes one path;
// then the calibrated tree of the committed token T: its sampled successors as children of the
// root, each followed at once by its own successors where the anchor was matched in the context
// (two levels, depth first).  A token a node already has as a child is not added twice; at most
// max_nodes draft nodes.  One block: all threads look for the latest position of T in the context,
// one thread builds.
__global__ void tree_draft_kernel(int* state, const int* hist, const int* succ, const int* occ, int b, int max_nodes) {
    __shared__ int best_s[32];
    const int n_ctx = state[ST_N_CTX], T = state[ST_PENDING];
    int best = -1;
    for (int q = threadIdx.x; q < n_ctx; q += blockDim.x)
        if (hist[q] == T) best = q;   // ascending per thread: the last hit is the thread's latest
    for (int off = 16; off; off >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
    if ((threadIdx.x & 31) == 0) best_s[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x != 0) return;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) best = max(best, best_s[w]);
    const int p = best;
    int n = state[ST_DRAFT_LEN];            // the chain: node i continues node i - 1
    if (n > max_nodes) n = max_nodes;
    for (int i = 1; i <= n; ++i) state[ST_PARENT + i] = i - 1;
    auto add = [&](int node, int tok) -> int {
        for (int c = 1; c <= n; ++c)
            if (state[ST_PARENT + c] == node && state[ST_DRAFT + c - 1] == tok) return c;
        if (n >= max_nodes) return -1;
        ++n;
        state[ST_DRAFT + n - 1] = tok;
        state[ST_PARENT + n] = node;
        return n;
    };
    if (p >= 0) {
        for (int i = 0; i < b; ++i) {
            const int c = add(0, succ[p * b + i]);
            const int q = occ[p * b + i];
            if (c >= 0 && q >= 0)
                for (int i2 = 0; i2 < b; ++i2) add(c, succ[q * b + i2]);
        }
    }
    state[ST_DRAFT_LEN] = n;
    state[ST_BASE_LEN] = n;
    state[ST_SEG_USED] = 0;
    tree_finish(state, n);
}

// The accepted path given by the caller (teacher forcing in tests): emitted = its tokens + next_token.
__global__ void set_path_kernel(int* state, DraftArg path, int next_token) {
    if (threadIdx.x != 0) return;
    for (int i = 0; i < path.n; ++i) {
        state[ST_PATH + i] = path.tok[i];
        state[ST_EMITTED + i] = state[ST_DRAFT + path.tok[i] - 1];
    }
    state[ST_EMITTED + path.n] = next_token;
    state[ST_PATH_LEN] = path.n;
    state[ST_ACCEPT_LEN] = path.n;
    state[ST_N_EMITTED] = path.n + 1;
}

// Before the commit of a tree step: the accepted path's K/V rows, written at cache slots L + row,
// move to the consecutive slots L + 1 .. L + a (ascending, sources never lie below their
// destinations: a row's index is at least its depth).  Rows of emitted tokens that the commit will
// cut off (max_emit) are not needed.  grid = (layers * KV heads, 2): K and V.
__global__ void kv_compact_kernel(const int* state, __nv_bfloat16* kcache, __nv_bfloat16* vcache, int max_seq, int hd,
                                  int max_emit) {
    if (!state[ST_TREE_ON]) return;
    const int L = state[ST_KV_LEN], a = state[ST_PATH_LEN];
    int n = state[ST_N_EMITTED];
    if (max_emit > 0 && n > max_emit) n = max_emit;
    const int keep = min(a, n - 1);
    __nv_bfloat16* base = (blockIdx.y ? vcache : kcache) + (size_t)blockIdx.x * max_seq * hd;
    for (int i = 1; i <= keep; ++i) {
        const int src = L + state[ST_PATH + i - 1], dst = L + i;
        if (src != dst)
            for (int e = threadIdx.x; e < hd; e += blockDim.x) base[(size_t)dst * hd + e] = base[(size_t)src * hd + e];
        __syncthreads();
    }
}
// Caller-supplied predictions for the stand-alone accept scan.
__global__ void set_y_kernel(int* state, DraftArg a) {
    if ((int)threadIdx.x < a.n) state[ST_Y + threadIdx.x] = a.tok[threadIdx.x];
}

// ------------------------------------------------------------------------------------------
// Draft extension (reuse of rejected drafts).  One warp each.
//
// extend: the retained segment is appended to the draft the drafter left, unless the draft would
// grow beyond max_total tokens, in which case the segment is dropped.
__device__ __forceinline__ void extend_draft_body(int* state, int max_total) {  // one warp
    const int lane = threadIdx.x;
    const int m = state[ST_DRAFT_LEN], sl = state[ST_SEG_LEN];
    const bool fits = sl > 0 && m + sl <= max_total;
    const int tok = (fits && lane < sl) ? state[ST_SEG + lane] : 0;
    __syncwarp();
    if (fits && lane < sl) state[ST_DRAFT + m + lane] = tok;
    if (lane == 0) {
        state[ST_BASE_LEN] = m;
        state[ST_SEG_USED] = fits ? 1 : 0;
        if (fits) {
            state[ST_DRAFT_LEN] = m + sl;
        } else if (sl > 0) {
            state[ST_SEG_LEN] = 0;
            state[ST_SEG_LIFE] = 0;
        }
    }
}
__global__ void extend_draft_kernel(int* state, int max_total, int in_run) {
    if (in_run && state[ST_BUDGET] == 0) return;
    extend_draft_body(state, max_total);
}

// update, after the accept scan of a verify step: lane i tests x_{i+1} == y_{i+1} beyond the reject
// point; the longest run of agreeing drafts (the earliest among equals) is the candidate.  Runs of
// length t survive t - 1 rounds of r &= r >> 1 (bit i of r: a run of the current length starts at
// i).  Then the retention rules: a segment that was appended ages by one step; it is dropped when
// the accepted prefix reached into it or its age passes max_life; a strictly longer candidate
// replaces what is retained.
__device__ __forceinline__ void extension_update_body(int* state, int max_life) {  // one warp
    const int lane = threadIdx.x;
    const int dl = state[ST_DRAFT_LEN], a = state[ST_ACCEPT_LEN];
    const int x = state[ST_DRAFT + lane], y = state[ST_Y + lane];
    const bool agree = lane < dl && lane > a && x == y;
    unsigned r = __ballot_sync(0xffffffffu, agree);
    int len = 0, first = 0;
    if (r) {
        len = 1;
        for (unsigned nr = r & (r >> 1); nr; nr = r & (r >> 1)) {
            r = nr;
            ++len;
        }
        first = __ffs((int)r) - 1;
    }
    int sl = state[ST_SEG_LEN], life = state[ST_SEG_LIFE];
    const int used = state[ST_SEG_USED], base = state[ST_BASE_LEN];
    if (used) ++life;
    if (sl > 0 && ((used && a > base) || life > max_life)) {
        sl = 0;
        life = 0;
    }
    const bool replace = len > sl;
    const int tok = (replace && lane < len) ? state[ST_DRAFT + first + lane] : 0;
    __syncwarp();
    if (replace) {
        if (lane < len) state[ST_SEG + lane] = tok;
        sl = len;
        life = 0;
    }
    if (lane == 0) {
        state[ST_SEG_LEN] = sl;
        state[ST_SEG_LIFE] = life;
        state[ST_SEG_USED] = 0;
    }
}
__global__ void extension_update_kernel(int* state, int max_life, int in_run) {
    if (in_run && state[ST_BUDGET] == 0) return;
    extension_update_body(state, max_life);
}

// ------------------------------------------------------------------------------------------
// Greedy tokens and accept scan.  Row j's token is the best of the per-block candidates
// (largest logit, lowest id among equals); a = number of leading drafts equal to the model's
// prediction; emitted = x_1..x_a, y_{a+1}.  One block of 32 * rows threads: warp j reduces row j.
// `row0`: the sequence's first row among the launch's rows (0 unless the step was batched); `launch_state`:
// the state block the launch ran on when it is not `state` itself, whose error word is carried over.
__device__ __forceinline__ void accept_body(int* state, const float* cand_val, const int* cand_idx, int G, int from_host_y,
                                            int row0, const int* launch_state) {
    __shared__ int y_s[kMaxRows + 1];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int dl = state[ST_DRAFT_LEN];
    if (launch_state && threadIdx.x == 0 && launch_state[ST_ERR]) state[ST_ERR] = launch_state[ST_ERR];
    if (warp <= dl) {
        int bi;
        if (from_host_y) {
            bi = state[ST_Y + warp];
        } else {
            float bv = -CUDART_INF_F;
            bi = 0x7fffffff;
            for (int c = lane; c < G; c += 32) {
                const float v = cand_val[(size_t)c * kMaxRows + row0 + warp];
                const int i = cand_idx[(size_t)c * kMaxRows + row0 + warp];
                if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
            }
            for (int off = 16; off; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
                if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
            }
            if (bi == 0x7fffffff) bi = 0;
        }
        if (lane == 0) { y_s[warp] = bi; state[ST_Y + warp] = bi; }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int a = 0;
        if (state[ST_TREE_ON]) {
            // strict acceptance on a tree: step to the lowest-numbered child that carries the model's
            // prediction at the current row, until no child does
            int cur = 0;
            for (;;) {
                int nxt = -1;
                for (int c = 1; c <= dl && nxt < 0; ++c)
                    if (state[ST_PARENT + c] == cur && state[ST_DRAFT + c - 1] == y_s[cur]) nxt = c;
                if (nxt < 0) break;
                state[ST_PATH + a] = nxt;
                state[ST_EMITTED + a] = state[ST_DRAFT + nxt - 1];
                ++a;
                cur = nxt;
            }
            state[ST_EMITTED + a] = y_s[cur];
            state[ST_PATH_LEN] = a;
        } else {
            while (a < dl && state[ST_DRAFT + a] == y_s[a]) ++a;
            for (int i = 0; i < a; ++i) state[ST_EMITTED + i] = state[ST_DRAFT + i];
            state[ST_EMITTED + a] = y_s[a];
        }
        state[ST_ACCEPT_LEN] = a;
        state[ST_N_EMITTED] = a + 1;
        state[ST_VERIFIED] = 1;
    }
}
__global__ void accept_kernel(int* state, const float* cand_val, const int* cand_idx, int G, int from_host_y, int row0,
                              const int* launch_state, int in_run) {
    if (in_run && state[ST_BUDGET] == 0) return;
    accept_body(state, cand_val, cand_idx, G, from_host_y, row0, launch_state);
}

// Batched verify: the token rows of up to kMaxBatch sequences (each its pending token, then its draft, token 0
// past the draft's length) are laid out one after another in the state block the shared launch reads.
struct BatchGatherArg {
    const int* state[kMaxBatch];
    int r0[kMaxBatch], M[kMaxBatch];
    int n;
};
__global__ void batch_gather_kernel(int* launch_state, BatchGatherArg a) {
    const int t = threadIdx.x;
    for (int b = 0; b < a.n; ++b) {
        if (t < a.M[b]) {
            const int* st = a.state[b];
            const int tok = (t == 0) ? st[ST_PENDING] : (t <= st[ST_DRAFT_LEN] ? st[ST_DRAFT + t - 1] : 0);
            const int row = a.r0[b] + t;
            if (row == 0) launch_state[ST_PENDING] = tok;
            else launch_state[ST_DRAFT + row - 1] = tok;
        }
    }
    if (t == 0) {
        launch_state[ST_DRAFT_LEN] = a.r0[a.n - 1] + a.M[a.n - 1] - 1;
        launch_state[ST_TREE_ON] = 0;
        launch_state[ST_ERR] = 0;
    }
}

// Commit: append the emitted tokens (cut to max_emit when > 0) to the history, advance the KV
// length by their number, make the last one the pending token.  KV rows past the new length
// are left as they are and overwritten by later steps.
__device__ __forceinline__ void commit_body(int* state, int* hist, int max_emit, int force_accept, int force_token, int in_run) {
    if (threadIdx.x != 0) return;
    if (in_run) {  // the run's token budget cuts its last step and ends it
        const int budget = state[ST_BUDGET];
        if (budget == 0) return;
        if (budget > 0) {
            const int n0 = state[ST_N_EMITTED];
            max_emit = budget;
            state[ST_BUDGET] = budget - (n0 < budget ? n0 : budget);
        }
    }
    int n = state[ST_N_EMITTED];
    if (force_accept >= 0) {
        n = force_accept + 1;
        for (int i = 0; i < force_accept; ++i) state[ST_EMITTED + i] = state[ST_DRAFT + i];
        state[ST_EMITTED + force_accept] = force_token;
        state[ST_ACCEPT_LEN] = force_accept;
    }
    if (max_emit > 0 && n > max_emit) n = max_emit;
    const int hl = state[ST_HIST_LEN];
    for (int i = 0; i < n; ++i) hist[hl + i] = state[ST_EMITTED + i];
    state[ST_N_EMITTED] = n;
    state[ST_HIST_LEN] = hl + n;
    state[ST_KV_LEN] += n;
    state[ST_PENDING] = state[ST_EMITTED + n - 1];
    state[ST_DRAFT_LEN] = 0;
    state[ST_VERIFIED] = 0;
    state[ST_TREE_ON] = 0;
}
__global__ void commit_kernel(int* state, int* hist, int max_emit, int force_accept, int force_token, int in_run) {
    commit_body(state, hist, max_emit, force_accept, force_token, in_run);
}

// Everything between two forward kernels (of a run of enqueued steps, or of sdv_step), in one launch of 1024 threads: the accept
// scan of the step just verified, [the update of the retained segment,] its commit under the run's token
// budget, and, unless the run ends here, the draft of the next step [and its extension].  The stages
// meet at block barriers: what one writes to the state block and the history, the next reads.
__global__ void __launch_bounds__(1024) step_tail_kernel(int* state, int* hist, const int* db, const float* cand_val,
                                                         const int* cand_idx, int G, int n, int n_min, int k, int search_history,
                                                         int ext_max_total, int ext_max_life, int draft_next, int in_run) {
    if (in_run && state[ST_BUDGET] == 0) return;   // enqueued behind the end of the run
    accept_body(state, cand_val, cand_idx, G, 0, 0, nullptr);
    __syncthreads();
    if (ext_max_total > 0) {
        if (threadIdx.x < 32) extension_update_body(state, ext_max_life);
        __syncthreads();
    }
    commit_body(state, hist, 0, -1, 0, in_run);
    __syncthreads();
    if (!draft_next || (in_run && state[ST_BUDGET] == 0)) return;
    ngram_draft_body(state, hist, db, n, n_min, k, search_history);
    if (ext_max_total > 0) {
        __syncthreads();
        if (threadIdx.x < 32) extend_draft_body(state, ext_max_total);
    }
}

// After the last prefill tile: the greedy token of its last row becomes the pending token.
__global__ void prefill_final_kernel(int* state, int* hist, const float* cand_val, const int* cand_idx, int G,
                                     int row) {
    const int lane = threadIdx.x;
    float bv = -CUDART_INF_F;
    int bi = 0x7fffffff;
    for (int c = lane; c < G; c += 32) {
        const float v = cand_val[(size_t)c * kMaxRows + row];
        const int i = cand_idx[(size_t)c * kMaxRows + row];
        if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
    }
    for (int off = 16; off; off >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
        if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) {
        if (bi == 0x7fffffff) bi = 0;
        const int hl = state[ST_HIST_LEN];
        hist[hl] = bi;
        state[ST_HIST_LEN] = hl + 1;
        state[ST_PENDING] = bi;
        state[ST_DRAFT_LEN] = 0;
        state[ST_Y] = bi;
    }
}

__global__ void set_state_kernel(int* state, int kv_len, int hist_len, int n_ctx, int pending_from_hist,
                                 const int* hist) {
    if (threadIdx.x != 0) return;
    state[ST_KV_LEN] = kv_len;
    state[ST_HIST_LEN] = hist_len;
    state[ST_N_CTX] = n_ctx;
    if (pending_from_hist && hist_len > 0) state[ST_PENDING] = hist[hist_len - 1];
    state[ST_DRAFT_LEN] = 0;
    state[ST_VERIFIED] = 0;
    state[ST_TREE_ON] = 0;
    state[ST_SEG_LEN] = 0;   // a new request starts without a retained segment
    state[ST_SEG_LIFE] = 0;
    state[ST_SEG_USED] = 0;
    state[ST_BASE_LEN] = 0;
}

// A bounded wait on a word nothing ever sets: exercises the give-up path of the device waits.
__global__ void timeout_probe_kernel(int* state, const int* never_set, unsigned long long limit_ns) {
    const uint64_t t0 = global_timer_ns();
    bool expired = false;
    while (ld_acquire_gpu(never_set) != 0x5eed) {
        if (global_timer_ns() - t0 > limit_ns) {
            expired = true;
            break;
        }
    }
    if (expired) atomicExch(state + ST_ERR, 2);
}

}  // namespace sdv
