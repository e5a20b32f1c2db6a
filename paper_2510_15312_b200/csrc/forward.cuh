// The persistent forward kernel: one launch runs the decoder over M <= 32 token rows
// (a verify step over [T, x_1..x_k], or one tile of a prefill chunk).
//
// One thread block per SM, 12 warps:
//   warp 11      weight streamer: walks the block's static share of every GEMM in launch order
//                and keeps a ring of 32 KB shared-memory stages full with bulk asynchronous copies.
//                It never waits for activations or grid barriers, only for free ring slots, so HBM
//                traffic continues across operation boundaries.
//   warp 10      one elected lane issues the tensor-core instructions (tcgen05.mma, M = 128 weight
//                rows x N = 16 or 32 token rows x K = 16 per instruction): the streamed stage is the A
//                operand, the token rows, resident in shared memory for the whole operation, the
//                B operand; accumulators live in tensor memory (two buffers of two 128-row
//                accumulators, so the next pass starts while the previous one is read out).
//   warps 0..7   read the accumulators back (tcgen05.ld) and run the fused epilogues: warps 0..3 the
//                first accumulator of a pass, warps 4..7 the second (or, for passes of up to 128
//                rows, alternate pairs of token columns of the one accumulator).
//   warps 0..9   build the token operand at the start of an operation (RMSNorm scale, merge of the
//                split-KV partial results, ...); warps 0..10 run the attention step.
// A layer is four operations separated by a bounded grid barrier: QKV projection; attention;
// output projection (+ residual); gate|up with SwiGLU followed, inside the same block and without
// a barrier, by the slice of the down projection (+ residual) that consumes this block's SwiGLU
// columns.
#pragma once
#include <math_constants.h>

#include "layout.cuh"
#include "ptx.cuh"

namespace sdv {

enum PhaseKind { PH_EMBED = 0, PH_QKV, PH_ATTN, PH_O, PH_GUD, PH_LM, PH_RAW };
constexpr int kPhasesPerLayer = 4;

// Phase numbering of a launch: 0 = embedding; 1 + 4*layer + {0..3} = QKV, attention, output
// projection, gate|up + down; 1 + 4*n_layers = LM head; 2 + 4*n_layers = stand-alone GEMM.
__host__ __device__ __forceinline__ int decode_phase(int ph, int n_layers, int& layer) {
    layer = 0;
    if (ph == 0) return PH_EMBED;
    if (ph == 1 + kPhasesPerLayer * n_layers) return PH_LM;
    if (ph == 2 + kPhasesPerLayer * n_layers) return PH_RAW;
    layer = (ph - 1) / kPhasesPerLayer;
    return PH_QKV + (ph - 1) % kPhasesPerLayer;
}
// The one or two streamed operations of a phase, in streaming order.
__device__ __forceinline__ int phase_ops(int kind, int (&ops)[2]) {
    switch (kind) {
        case PH_QKV: ops[0] = OP_QKV; return 1;
        case PH_O: ops[0] = OP_O; return 1;
        case PH_GUD: ops[0] = OP_GU; ops[1] = OP_DOWN; return 2;
        case PH_LM: ops[0] = OP_LM; return 1;
        case PH_RAW: ops[0] = OP_RAW; return 1;
        default: return 0;
    }
}
__device__ __forceinline__ const uint8_t* op_weights(const FwdParams& P, int op, int layer) {
    if (op == OP_LM) return P.wlm + P.op[OP_LM].w_off;
    if (op == OP_RAW) return P.wraw + P.op[OP_RAW].w_off;
    return P.wlayers + (unsigned long long)layer * P.layer_stride + P.op[op].w_off;
}

struct Misc {
    uint64_t full[kMaxStages], empty[kMaxStages];
    uint64_t tmem_full[2], tmem_empty[2];
    uint64_t act_ready;   // the SwiGLU operand of this block is complete (one arrival per epilogue warp)
    uint64_t done_bar;    // last tensor-core instruction of the launch has completed
    uint32_t tmem_base;
    unsigned long long* prof_ptr;  // this block's profile words of the running phase (or null)
    int abort_flag;
    int skip;  // block-uniform copy of abort_flag, refreshed inside every grid barrier
    float sumsq[kMaxRows];  // sums of squares of the residual rows (this block's operand columns)
    float best_v[kEpilogueWarps][kMaxRows];
    int best_i[kEpilogueWarps][kMaxRows];
    Part part[OP_COUNT];  // this block's share of every operation
    FwdParams P;          // block-local copy of the launch parameters
};
static_assert(sizeof(Misc) <= kMiscSmemBytes, "misc shared memory");

// ------------------------------------------------------------------------------------------
// Grid barrier: every block adds one to a counter (release) and waits (bounded, acquire) until all
// have.  Called by all worker threads.  Returns, identically for all of them, whether some bounded
// wait in this block has been abandoned (the remaining phases then do no work).
__device__ __forceinline__ bool grid_barrier(const FwdParams& P, unsigned target, Misc* misc, int wtid) {
    named_bar_sync(1, kWorkerThreads);
    if (wtid == 0) {
        red_release_add_u32(P.bar, 1u);  // no return value to wait for: polling starts at once
        uint64_t t0 = 0;  // the global timer is slow to read: only once the wait has lasted a while
        uint32_t spins = 0;
        while ((int)(ld_acquire_gpu_u32(P.bar) - target) < 0) {  // wrap-safe: the difference, read as signed
            if ((++spins & 63u) == 0) {
                if (*(volatile int*)&misc->abort_flag) break;
                const uint64_t now = global_timer_ns();
                if (t0 == 0) t0 = now;
                if (now - t0 > P.wait_limit_ns) {
                    *(volatile int*)&misc->abort_flag = 1;
                    break;
                }
            }
        }
        *(volatile int*)&misc->skip = *(volatile int*)&misc->abort_flag;
    }
    named_bar_sync(1, kWorkerThreads);
    return *(volatile int*)&misc->skip != 0;
}

// ------------------------------------------------------------------------------------------
// Weight streamer (one thread).
__device__ __forceinline__ void producer_loop(const FwdParams& P, uint8_t* smem, Misc* misc) {
    const uint64_t policy = l2_policy_evict_first();
    const uint32_t nstage = (uint32_t)P.nstage;
    uint32_t slot = 0, par = 0, issued = 0;  // ring position; parity of the current trip round the ring
    bool ok = true;
    for (int ph = P.ph_begin; ph < P.ph_end && ok; ++ph) {
        int layer, ops[2];
        const int kind = decode_phase(ph, P.n_layers, layer);
        const int nops = phase_ops(kind, ops);
        for (int oi = 0; oi < nops && ok; ++oi) {
            const Part& pt = misc->part[ops[oi]];
            if (pt.ntiles == 0 || pt.nk == 0) continue;
            const uint8_t* src = op_weights(P, ops[oi], layer) + pt.off;
            const int nst = pt.nst, SK = pt.SK, nk = pt.nk;
            for (int p = 0; p < pt.npass && ok; ++p) {
                const uint32_t pbytes = (uint32_t)pass_count(pt, p) * kStepBytes;
                int kleft = nk;
                for (int st = 0; st < nst; ++st, kleft -= SK) {
                    const uint32_t bytes = pbytes * (uint32_t)min(SK, kleft);
                    // the slot's previous contents must have been consumed (first trip: free at once)
                    if (!mbar_wait_bounded(&misc->empty[slot], par ^ 1u, &misc->abort_flag, P.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                    mbar_arrive_expect_tx(&misc->full[slot], bytes);
                    bulk_g2s(smem + slot * kStageBytes, src, bytes, &misc->full[slot], policy);
                    src += bytes;
                    ++issued;
                    if (++slot == nstage) { slot = 0; par ^= 1u; }
                }
            }
        }
    }
    if (!ok) {
        // Abandoned: wait (bounded) for the copies still in flight before the block may exit.
        for (uint32_t back = 0; back < nstage && back < issued; ++back) {
            if (slot == 0) { slot = nstage; par ^= 1u; }
            --slot;
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(&misc->full[slot], par)) {
                if (global_timer_ns() - t0 > P.wait_limit_ns) break;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Token operand of a GEMM, resident in shared memory for the whole operation, in a layout the
// tensor core reads (K-major, no swizzle): for every 8 columns the M token rows, 16 bytes each:
//     [8-column group][row 0..M-1][8 bf16].
// An 8-row core matrix is 128 contiguous bytes, row groups are 128 bytes apart and the two halves
// of a column step M * 16 bytes.  The instruction reads 16 or 32 rows: the ones past M belong to the
// next column groups (or lie behind the operand, still inside shared memory) and only feed
// accumulator columns nobody reads.
__device__ __forceinline__ uint32_t operand_off(int k8, int row, int M) {
    return (uint32_t)((k8 * M + row) * 16);
}

// Operand = residual rows scaled by the RMSNorm weight (the per-row factor rsqrt(mean + eps)
// commutes with the GEMM and is applied by the consumer of the result), or, for the stand-alone
// GEMM, the caller's fp32 rows as they are.  Warp w converts rows w, w + 11, ...; all loads of a
// batch are issued before the first use.  Leaves the rows' sums of squares over this block's
// columns in misc->sumsq; QKV blocks of row partition 0 also add them to the global sums the
// attention step reads.
__device__ __forceinline__ void build_norm_operand(const FwdParams& P, int kind, int layer, const Part& pt, uint8_t* U,
                                                Misc* misc, int wtid) {
    constexpr int UB = 12;  // 4-column units per lane and batch; a warp instruction reads 512 contiguous bytes
    const int warp = wtid >> 5, lane = wtid & 31;
    const int M = P.M;
    const int k4_0 = pt.k0 * 4, nk4 = pt.nk * 4;
    const bool raw = (kind == PH_RAW);
    const int stride = raw ? P.raw_K : P.d;
    const float* xbase = raw ? P.raw_x : P.h;
    const float* wn = raw ? nullptr
                          : P.norm_w + (size_t)(kind == PH_QKV ? layer * 2 : (kind == PH_GUD ? layer * 2 + 1 : P.n_layers * 2)) * P.d;
    for (int row = warp; row < M; row += kBuilderWarps) {
        const float4* src = reinterpret_cast<const float4*>(xbase + (size_t)row * stride) + k4_0;
        const float4* wsrc = wn ? reinterpret_cast<const float4*>(wn) + k4_0 : nullptr;
        const float4* wld = wsrc ? wsrc : src;  // without norm weights the loaded value is not used
        float ss = 0.f;
        for (int base = lane; base < nk4; base += 32 * UB) {
            float4 a[UB], w[UB];
            // every unit loads (past the end: the row's last unit again, not used), so that the loads are one
            // straight run of instructions instead of a branch per unit
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int k4 = min(base + u * 32, nk4 - 1);
                a[u] = ld_cg_f4_inorder(src + k4);
                w[u] = ld_nc_f4_inorder(wld + k4);
            }
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int k4 = base + u * 32;
                if (k4 < nk4) {
                    const float4 x = a[u];
                    const float4 g = wsrc ? w[u] : make_float4(1.f, 1.f, 1.f, 1.f);
                    ss += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
                    const uint2 out = make_uint2(pack_bf16(x.x * g.x, x.y * g.y), pack_bf16(x.z * g.z, x.w * g.w));
                    *reinterpret_cast<uint2*>(U + operand_off(k4 >> 1, row, M) + (k4 & 1) * 8) = out;
                }
            }
        }
#pragma unroll
        for (int off = 16; off; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        if (lane == 0) {
            misc->sumsq[row] = ss;
            if (kind == PH_QKV && pt.pr == 0) atomicAdd(P.sumsq + (layer & 1) * kMaxRows + row, ss);
        }
    }
}

__device__ __forceinline__ void attn_split(const FwdParams& P, int& S, int& kps);

// Operand of the output projection = attention output of this block's columns: the split-KV
// partial results (un-normalised sums with their running maximum and sum) are merged on the way.
// Four lanes share one (row, 8 columns) item, each taking every fourth partial result.
__device__ __forceinline__ void build_merged_operand(const FwdParams& P, const Part& pt, uint8_t* U, int wtid) {
    constexpr int TPL = (kMaxSplits + 1 + 3) / 4;  // partial results per lane at most
    int S, kps;
    attn_split(P, S, kps);
    const int S1 = S + 1;
    const int M = P.M, hd = P.hd;
    const int k8_0 = pt.k0 * 2, nk8 = pt.nk * 2;
    const int nitems = M * nk8, sub = wtid & 3;
    for (int it0 = 0; it0 < nitems; it0 += kBuilderWarps * 32 / 4) {
        const int item = it0 + (wtid >> 2);
        const bool live = item < nitems;
        const int j = live ? item / nk8 : 0, k8l = live ? item % nk8 : 0;
        const int col = (k8_0 + k8l) * 8, hq = col / hd, c = col % hd;
        const size_t base = ((size_t)hq * (kMaxSplits + 1)) * kMaxRows + j;
        float m[TPL], l[TPL];
        float4 a[TPL], b[TPL];
        // every slot loads (beyond the last partial result: the last one again, given no weight below), so that
        // the loads are one straight run of instructions instead of a branch per slot
#pragma unroll
        for (int t = 0; t < TPL; ++t) {
            const int s = sub + 4 * t;
            const size_t row = base + (size_t)min(s, S) * kMaxRows;
            const float2 ml = ld_cg_f2_inorder(P.part_ml + row * 2);
            const float* op = P.part_o + row * hd + c;
            a[t] = ld_cg_f4_inorder(op);
            b[t] = ld_cg_f4_inorder(op + 4);
            const bool use = live && s < S1;
            m[t] = use ? ml.x : -CUDART_INF_F;
            l[t] = use ? ml.y : 0.f;
        }
        float mmax = m[0];
#pragma unroll
        for (int t = 1; t < TPL; ++t) mmax = fmaxf(mmax, m[t]);
        mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, 1));
        mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, 2));
        const float ref = (mmax == -CUDART_INF_F) ? 0.f : mmax;
        float v[9];
#pragma unroll
        for (int e = 0; e < 9; ++e) v[e] = 0.f;
#pragma unroll
        for (int t = 0; t < TPL; ++t) {
            const float w = exp2f(m[t] - ref);  // 0 for partial results that saw no key
            v[0] += w * a[t].x; v[1] += w * a[t].y; v[2] += w * a[t].z; v[3] += w * a[t].w;
            v[4] += w * b[t].x; v[5] += w * b[t].y; v[6] += w * b[t].z; v[7] += w * b[t].w;
            v[8] += w * l[t];
        }
#pragma unroll
        for (int e = 0; e < 9; ++e) {
            v[e] += __shfl_xor_sync(0xffffffffu, v[e], 1);
            v[e] += __shfl_xor_sync(0xffffffffu, v[e], 2);
        }
        if (live && sub == 0) {
            const float inv = 1.f / v[8];
            const uint4 out = make_uint4(pack_bf16(v[0] * inv, v[1] * inv), pack_bf16(v[2] * inv, v[3] * inv),
                                         pack_bf16(v[4] * inv, v[5] * inv), pack_bf16(v[6] * inv, v[7] * inv));
            *reinterpret_cast<uint4*>(U + operand_off(k8l, j, M)) = out;
        }
    }
}

// ------------------------------------------------------------------------------------------
// Tensor-core issue.  The whole warp walks the loop so that ring positions and operand descriptors
// stay warp-uniform values; one elected lane issues the instructions.  Pipeline positions: (slot, par) is the ring position (slot
// index and parity of the current trip round the ring), `q` counts accumulator passes; all advance
// over the whole launch, identically in every role.  The issuing thread is bound by its own
// instruction latency, so the loop keeps ready-made descriptors and advances them by additions.
struct PipePos {
    uint32_t slot, par, q, act_uses;
    uint32_t w_full, w_acc;  // cycles the tensor-core thread waited for weights / for a free accumulator (profile)
};

__device__ __forceinline__ void mma_op(const FwdParams& P, const Part& pt, uint8_t* smem, const uint8_t* B, Misc* misc,
                                       PipePos& pos, bool& dead, bool& synced) {
    const uint32_t nstage = (uint32_t)P.nstage;
    const uint32_t idesc = umma_idesc_bf16_m128((uint32_t)P.NB);
    const uint64_t wait_limit = P.wait_limit_ns;
    const uint32_t lbo_b = (uint32_t)P.M * 16u;
    const uint64_t bstep = (uint64_t)((2u * lbo_b) >> 4);       // one column step, in descriptor address units
    const uint64_t bdesc0 = umma_smem_desc(smem_u32(B), lbo_b, 128u);
    const uint32_t ring0 = smem_u32(smem);
    const uint32_t tmem0 = misc->tmem_base;
    const int nst = pt.nst, SK = pt.SK, nk = pt.nk;
    for (int p = 0; p < pt.npass; ++p, ++pos.q) {
        const int pcount = pass_count(pt, p);
        const uint32_t buf = pos.q & 1u;
        const long long tq0 = clock64();
        if (!dead && !mbar_wait_bounded(&misc->tmem_empty[buf], ((pos.q >> 1) & 1u) ^ 1u, &misc->abort_flag, wait_limit))
            dead = true;
        pos.w_acc += (uint32_t)(clock64() - tq0);
        const uint32_t d_tmem = tmem0 + buf * 64u;
        const bool two = pcount > 8;  // rows 128.. of the pass go to the buffer's second accumulator
        const uint32_t lbo_a = (uint32_t)(2 * pcount) * 128u;
        const uint64_t astep = (uint64_t)((2u * lbo_a) >> 4);
        const uint64_t adesc0 = umma_smem_desc(ring0, lbo_a, 128u);
        uint64_t bdesc = bdesc0;
        int kleft = nk;
        for (int st = 0; st < nst; ++st, kleft -= SK) {
            const uint32_t slot = pos.slot, par = pos.par;
            if (++pos.slot == nstage) { pos.slot = 0; pos.par ^= 1u; }
            const int nks = min(SK, kleft);
            if (!synced) {
                // everything above ran while the other warps were still building the token operand
                named_bar_sync(1, kWorkerThreads);
                synced = true;
            }
            if (dead) continue;
            const long long tw0 = clock64();
            if (!mbar_wait_bounded(&misc->full[slot], par, &misc->abort_flag, wait_limit)) {
                dead = true;
                continue;
            }
            pos.w_full += (uint32_t)(clock64() - tw0);
            tc_fence_after();
            uint64_t adesc = adesc0 + (uint64_t)((slot * (uint32_t)kStageBytes) >> 4);
            if (elect_one()) {
                if (st == 0) {
                    umma_bf16_first(d_tmem, adesc, bdesc, idesc);
                    if (two) umma_bf16_first(d_tmem + 32u, adesc + 128u, bdesc, idesc);
                } else {
                    umma_bf16_acc(d_tmem, adesc, bdesc, idesc);
                    if (two) umma_bf16_acc(d_tmem + 32u, adesc + 128u, bdesc, idesc);
                }
#pragma unroll 3
                for (int ks = 1; ks < nks; ++ks) {
                    adesc += astep;
                    bdesc += bstep;
                    umma_bf16_acc(d_tmem, adesc, bdesc, idesc);
                    if (two) umma_bf16_acc(d_tmem + 32u, adesc + 128u, bdesc, idesc);
                }
                bdesc += bstep;
                umma_commit(&misc->empty[slot]);  // the slot is free once these instructions have read it
            } else {
                bdesc += (uint64_t)nks * bstep;
            }
            __syncwarp();
        }
        if (!dead && elect_one()) umma_commit(&misc->tmem_full[buf]);
        __syncwarp();
    }
}

// ------------------------------------------------------------------------------------------
// Epilogues (warps 0..7).  Thread t = 32 * (warp & 3) + lane owns row t of its 128-row accumulator,
// i.e. one weight row (output feature), for the token columns its warp group takes.
// SwiGLU on one accumulator row per thread.  Rows 0..7 of a 16-row tile are gate rows, rows 8..15 the
// matching up rows, so the two values of an output sit 8 lanes apart.  Token columns are taken in
// pairs: the gate lane evaluates the even column of a pair, the up lane the odd one; one shuffle per
// pair hands each lane the partner's value it needs.  All pairs are independent and written without
// branches, so that their shuffles, exponentials and divisions overlap.  SEL >= 0: only pairs j with
// (j & 1) == SEL (the other group of epilogue warps takes the rest).
template <int NBT, int SEL>
__device__ __forceinline__ void swiglu_pairs(const float (&v)[NBT], const float (&rstd)[NBT], int t, bool valid, int M,
                                             uint8_t* dst) {
    constexpr int STEP = SEL < 0 ? 1 : 2, J0 = SEL < 0 ? 0 : SEL, NP = (NBT / 2 - J0 + STEP - 1) / STEP;
    const bool is_up = (t & 8) != 0;
    float got[NP], out[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const int j = J0 + i * STEP;
        got[i] = __shfl_xor_sync(0xffffffffu, is_up ? v[2 * j] : v[2 * j + 1], 8);
    }
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const int j = J0 + i * STEP;
        const float mine = is_up ? v[2 * j + 1] : v[2 * j], r = is_up ? rstd[2 * j + 1] : rstd[2 * j];
        const float x = (is_up ? got[i] : mine) * r, y = (is_up ? mine : got[i]) * r;
        out[i] = __fdividef(x, 1.f + __expf(-x)) * y;
    }
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const int n = 2 * (J0 + i * STEP) + (is_up ? 1 : 0);
        if (valid && n < M) *reinterpret_cast<__nv_bfloat16*>(dst + n * 16) = __float2bfloat16(out[i]);
    }
}

// LM: the operation is the LM head (bv / bi carry the running best logit per token row); the other operations
// are compiled without that state, which would otherwise occupy 2 x NBT registers through every phase.
template <int NBT, bool LM>  // NBT: token columns read, 16 or 32
__device__ __forceinline__ void epilogue_op(const FwdParams& P, int kind, int op, int layer, const Part& pt, uint8_t* act, Misc* misc,
                                            PipePos& pos, bool& dead, int warp, int lane, float (&bv)[LM ? NBT : 1],
                                            int (&bi)[LM ? NBT : 1]) {
    const int M = P.M;
    const int quarter = warp & 3, myhalf = warp >> 2;  // this warp's 32 accumulator lanes; which of the two accumulators
    const int t = quarter * 32 + lane;
    const uint64_t wait_limit = P.wait_limit_ns;
    const uint32_t tmem_lane = misc->tmem_base + ((uint32_t)(quarter * 32) << 16);
    const int npass = pt.npass, tile0 = pt.tile0;
    float rstd[NBT];
    if (op == OP_GU || LM) {
        const float inv_d = 1.f / (float)P.d, eps = P.eps;
#pragma unroll
        for (int n = 0; n < NBT; ++n) rstd[n] = (n < M) ? rsqrtf(misc->sumsq[n] * inv_d + eps) : 0.f;
    }
    float* out = P.h;
    int stride = P.d;
    bool add = true;  // residual add (O, down)
    if (op == OP_QKV) { out = P.qkv_acc; stride = P.n_qkv; add = P.op[OP_QKV].P_k > 1; }
    else if (op == OP_RAW) { out = P.raw_out; stride = P.raw_N; add = P.op[OP_RAW].P_k > 1; }
    const int store_logits = P.store_logits;
    for (int p = 0; p < npass; ++p, ++pos.q) {
        const int pcount = pass_count(pt, p), pstart = pass_start(pt, p);
        const uint32_t buf = pos.q & 1u;
        if (!dead && !mbar_wait_bounded(&misc->tmem_full[buf], (pos.q >> 1) & 1u, &misc->abort_flag, wait_limit)) dead = true;
        dead = __any_sync(0xffffffffu, dead);
        if (dead) continue;
        tc_fence_after();
        if (misc->prof_ptr && t == 0 && p == npass - 1) misc->prof_ptr[10] = global_timer_ns();
        const int nhalf = pcount > 8 ? 2 : 1;  // a pass of more than 8 tiles fills both 128-row accumulators of the buffer
        // two accumulators: warps 0..3 read the first, 4..7 the second; one accumulator: both groups read
        // it and share its token columns (pairs of columns alternate between the groups)
        const int nsel = (nhalf == 2) ? -1 : myhalf;
        {
            const int half = (nhalf == 2) ? myhalf : 0;
            float v[NBT];
            {
                const uint32_t taddr = tmem_lane + buf * 64u + (uint32_t)half * 32u;
                float lo[16];
                tmem_ld16(taddr, lo);
#pragma unroll
                for (int n = 0; n < 16; ++n) v[n] = lo[n];
                if (NBT == 32) {
                    float hi[16];
                    tmem_ld16(taddr + 16u, hi);
#pragma unroll
                    for (int n = 0; n < 16; ++n) v[(NBT == 32 ? 16 : 0) + n] = hi[n];
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&misc->tmem_empty[buf]);  // this warp's part of the accumulators may be overwritten
            const int tt = half * 128 + t;         // row within the pass
            const bool valid = tt < 16 * pcount;
            const int row = (tile0 + pstart) * 16 + tt;  // weight row = output feature
            if (!LM && op == OP_GU) {
                // rows 0..7 of a tile are gate rows, 8..15 the matching up rows, 8 lanes apart: the gate
                // lane evaluates the even token columns, the up lane the odd ones
                const int col = (pstart + (tt >> 4)) * 8 + (tt & 7);  // SwiGLU column within this block's slice
                uint8_t* dst = act + operand_off(col >> 3, 0, M) + (col & 7) * 2;
                if (nsel < 0) swiglu_pairs<NBT, -1>(v, rstd, t, valid, M, dst);
                else if (nsel == 0) swiglu_pairs<NBT, 0>(v, rstd, t, valid, M, dst);
                else swiglu_pairs<NBT, 1>(v, rstd, t, valid, M, dst);
            } else if (LM) {
#pragma unroll
                for (int n = 0; n < NBT; ++n) {
                    if (valid && n < M && (nsel < 0 || ((n >> 1) & 1) == nsel)) {
                        const float x = v[n] * rstd[n];
                        if (store_logits) __stcg(P.logits + (size_t)n * P.V + row, x);
                        // rows come in ascending order per thread, so ">" keeps the lowest id among equals
                        if (x > bv[LM ? n : 0]) { bv[LM ? n : 0] = x; bi[LM ? n : 0] = row; }
                    }
                }
            } else if (valid) {
                float* d2 = out + row;
                if (add) {
#pragma unroll
                    for (int n = 0; n < NBT; ++n, d2 += stride)
                        if (n < M && (nsel < 0 || ((n >> 1) & 1) == nsel)) red_add_f32(d2, v[n]);
                } else {
#pragma unroll
                    for (int n = 0; n < NBT; ++n, d2 += stride)
                        if (n < M && (nsel < 0 || ((n >> 1) & 1) == nsel)) __stcg(d2, v[n]);
                }
            }
        }
    }
    if (!LM && op == OP_GU) {
        // this warp's SwiGLU columns are written: hand them to the tensor-core thread
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&misc->act_ready);
    }
}

// Best logit per token row over the block: lanes, then the four epilogue warps.
template <int NBT>
__device__ __forceinline__ void argmax_finish(const FwdParams& P, Misc* misc, int warp, int lane, float (&bv)[NBT], int (&bi)[NBT],
                                              bool dead) {
#pragma unroll
    for (int n = 0; n < NBT; ++n) {
        float v = bv[n];
        int i = bi[n];
#pragma unroll
        for (int off = 1; off <= 16; off <<= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, v, off);
            const int oi = __shfl_xor_sync(0xffffffffu, i, off);
            if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
        }
        if (lane == 0) {
            misc->best_v[warp][n] = v;
            misc->best_i[warp][n] = i;
        }
    }
    named_bar_sync(2, kEpilogueWarps * 32);
    const int t = warp * 32 + lane;
    if (t < NBT && t < P.M && !dead) {
        float v = misc->best_v[0][t];
        int i = misc->best_i[0][t];
        for (int w = 1; w < kEpilogueWarps; ++w) {
            const float ov = misc->best_v[w][t];
            const int oi = misc->best_i[w][t];
            if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
        }
        P.cand_val[(size_t)blockIdx.x * kMaxRows + t] = v;
        P.cand_idx[(size_t)blockIdx.x * kMaxRows + t] = i;
    }
}

template <int NBT>
__device__ __forceinline__ void epilogue_phase(const FwdParams& P, int kind, int layer, uint8_t* act, Misc* misc, PipePos& pos,
                                            bool& dead, int warp, int lane) {
    if (kind == PH_LM) {
        float bv[NBT];
        int bi[NBT];
#pragma unroll
        for (int n = 0; n < NBT; ++n) { bv[n] = -CUDART_INF_F; bi[n] = 0x7fffffff; }
        const Part& pt = misc->part[OP_LM];
        if (pt.ntiles > 0 && pt.nk > 0) epilogue_op<NBT, true>(P, kind, OP_LM, layer, pt, act, misc, pos, dead, warp, lane, bv, bi);
        argmax_finish<NBT>(P, misc, warp, lane, bv, bi, dead);
        return;
    }
    float none_v[1];
    int none_i[1];
    int ops[2];
    const int nops = phase_ops(kind, ops);
    for (int oi = 0; oi < nops; ++oi) {
        const Part& pt = misc->part[ops[oi]];
        if (pt.ntiles == 0 || pt.nk == 0) continue;
        epilogue_op<NBT, false>(P, kind, ops[oi], layer, pt, act, misc, pos, dead, warp, lane, none_v, none_i);
    }
}

// ------------------------------------------------------------------------------------------
// Split-KV attention.  The committed cache [0, L) is cut into S key ranges of kps keys (a multiple
// of 64, at most kMaxSplits ranges); the query heads of a KV head are cut into QG groups of up to
// gh heads, a group's rows (heads x M) filling at most four 16-row tiles (the host picks gh so
// that the longest chain of 16-key steps a warp walks is shortest).
// Unit (kv head, head group, s < S) attends the group's rows to range s; unit (kv head, head group,
// S) covers the M new rows: it finishes their K/V projection (norm scale, bias, rotary), appends
// them to the cache (group 0 only) and attends to them under the causal mask (row j sees new keys
// 0..j).  Every unit leaves an un-normalised partial result with its running maximum and sum; the
// output projection merges them while it builds its operand.
//
// Keys come in blocks of 64, copied asynchronously into two shared-memory buffers by all worker
// warps.  Warp (row tile, key group) owns one row tile and every KG-th group of 16 keys of a block
// (KG = 4 with up to two row tiles, 3 with three, 2 with four): scores (Q K^T on tensor cores), online softmax with quad
// shuffles in the log2 domain and P V all stay in its registers; the key groups of a row tile meet
// in shared memory at the end.
// The heads per group are chosen on the host per launch; the key ranges follow from it: as many
// as there are blocks to take a (KV head, head group, range) unit each, at most kMaxSplits.
__device__ __forceinline__ void attn_split(const FwdParams& P, int& S, int& kps) {
    S = P.att_S;      // worked out once per launch (attn_split_compute): the divisions are not repeated per phase
    kps = P.att_kps;
}
__device__ __forceinline__ void attn_split_compute(const FwdParams& P, int& S, int& kps) {
    if (P.L <= 0) { S = 0; kps = 0; return; }
    const int QG = (P.g + P.att_gh - 1) / P.att_gh;
    int cap = P.G / (P.n_kv * QG) - 1;
    if (cap > kMaxSplits) cap = kMaxSplits;
    if (cap < 1) cap = 1;
    kps = ((P.L + cap - 1) / cap + 63) / 64 * 64;
    S = (P.L + kps - 1) / kps;
}

// MODE 0: the new rows are a chain; 1: a tree (positions and visibility from the state block); 2: the chain of
// sequence `b` of a batched step (its rows, length and KV cache from P.seq[b]).
template <int HD, int MODE>
__device__ __noinline__ void attention_unit(const FwdParams& P, int layer, int hk, int qg, int gh, int s, int S, int kps, uint8_t* att,
                                            int wtid, unsigned long long* prof, int b) {
    constexpr bool TREE = MODE == 1, BATCH = MODE == 2;
    constexpr int HD2 = HD / 2;
    constexpr int KSTEPS = HD / 16;
    constexpr int UNITS = HD / 8;    // 16-byte units per K/V row
    constexpr int NT_O = HD / 8;     // 8-column tiles of the output
    constexpr int KB = 64;           // keys per block
    constexpr int NBUF = 2;
    constexpr int QBYTES = 64 * HD * 2;
    constexpr int KVBYTES = KB * HD * 2;  // one K (or V) block
    static_assert(QBYTES + NBUF * 2 * KVBYTES <= kAttnSmemBytes, "attention tiles");
    // exchange area of the key-group merge: (KG - 1) * MT <= 6 tiles of (output + statistics)
    static_assert(6 * (NT_O + 1) * 32 * 16 <= NBUF * 2 * KVBYTES, "exchange area of the key-group merge");
    const int warp = wtid >> 5, lane = wtid & 31;
    const int M = BATCH ? P.seq[b].M : P.M, L = BATCH ? P.seq[b].L : P.L;
    const int r0 = BATCH ? P.seq[b].r0 : 0;      // first row of this sequence in the launch's buffers
    __nv_bfloat16* const kcache = BATCH ? P.seq[b].kcache : P.kcache;
    __nv_bfloat16* const vcache = BATCH ? P.seq[b].vcache : P.vcache;
    const int nheads = min(gh, P.g - qg * gh);   // the last group may hold fewer heads
    const int R = nheads * M;                    // R <= 64
    const int MT = (R + 15) >> 4, RP = MT * 16;
    const int KG = MT <= 2 ? 4 : (MT == 3 ? 3 : 2);  // key groups: 16-key chunks of a block handled side by side
    const bool active = warp < MT * KG;
    const int mt = active ? warp % MT : 0, kgp = active ? warp / MT : 0;
    const int head0 = hk * P.g + qg * gh;     // first query head of this unit
    const bool is_new = (s == S);
    uint8_t* Qs = att;
    uint8_t* KVs = att + QBYTES;
    const float* sumsq = P.sumsq + (layer & 1) * kMaxRows;
    const float* bias = P.bias ? P.bias + (size_t)layer * P.n_qkv : nullptr;
    const int Nq = P.n_q * HD, Nkv = P.n_kv * HD;

    int t_begin = 0, nkeys = M;
    if (!is_new) {
        t_begin = s * kps;
        const int t_end = min(L, t_begin + kps);
        nkeys = max(0, t_end - t_begin);
    }
    const int nblk = (nkeys + KB - 1) / KB;
    const size_t cache_row0 = ((size_t)layer * P.n_kv + hk) * P.max_seq;

    // cached keys and values of one block: 16-byte asynchronous copies, rows past the range zero-filled
    auto load_block = [&](int blk) {
        if (blk < nblk) {
            uint8_t* Ks = KVs + (blk % NBUF) * 2 * KVBYTES;
            uint8_t* Vs = Ks + KVBYTES;
            for (int u = wtid; u < KB * UNITS; u += kWorkerThreads) {
                const int key = u / UNITS, q16 = u % UNITS, kk = blk * KB + key;
                const bool valid = kk < nkeys;
                const size_t off = (cache_row0 + t_begin + (valid ? kk : 0)) * HD + q16 * 8;
                const uint32_t so = (q16 >> 3) * (KB * 128) + swz_unit(key, q16 & 7);
                cp_async_16_zfill(Ks + so, kcache + off, valid);
                cp_async_16_zfill(Vs + so, vcache + off, valid);
            }
        }
        cp_async_commit();  // possibly empty: keeps the group count uniform
    };
    if (prof && wtid == 0) prof[2] = global_timer_ns();
    if (!is_new) {
#pragma unroll
        for (int b = 0; b < NBUF; ++b) load_block(b);
    }

    // ---- query tile: normalise, add bias, rotate, round to bf16; 4 rotary pairs per item
    {
        constexpr int QI = 2;  // items per thread and batch: all loads are issued before the first use
        const int items = RP * (HD2 / 4);
        for (int base = wtid; base < items; base += QI * kWorkerThreads) {
            float4 qa[QI], qb[QI], c0[QI], c1[QI];
            float ssq[QI];
            int rr[QI], ii[QI];
#pragma unroll
            for (int t = 0; t < QI; ++t) {
                const int idx = base + t * kWorkerThreads;
                rr[t] = idx / (HD2 / 4);
                ii[t] = (idx % (HD2 / 4)) * 4;
                ssq[t] = 0.f;
                qa[t] = qb[t] = c0[t] = c1[t] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (idx < items && rr[t] < R) {
                    const int hl = rr[t] / M, j = rr[t] % M, col = (head0 + hl) * HD + ii[t];
                    ssq[t] = __ldcg(sumsq + r0 + j);
                    qa[t] = ld_cg_f4_inorder(P.qkv_acc + (size_t)(r0 + j) * P.n_qkv + col);
                    qb[t] = ld_cg_f4_inorder(P.qkv_acc + (size_t)(r0 + j) * P.n_qkv + col + HD2);
                    const int pj = TREE ? __ldcg(P.state + ST_DEPTH + j) : j;  // tree drafts: a row's position is its depth
                    const float4* rp = reinterpret_cast<const float4*>(P.rope + (size_t)(L + pj) * HD2 + ii[t]);
                    c0[t] = ld_nc_f4_inorder(rp);
                    c1[t] = ld_nc_f4_inorder(rp + 1);
                }
            }
#pragma unroll
            for (int t = 0; t < QI; ++t) {
                const int idx = base + t * kWorkerThreads;
                if (idx >= items) continue;
                const int r = rr[t], i = ii[t];
                uint2 lo = make_uint2(0, 0), hi = make_uint2(0, 0);
                if (r < R) {
                    const float rs = rsqrtf(ssq[t] / (float)P.d + P.eps);
                    float a[4] = {qa[t].x * rs, qa[t].y * rs, qa[t].z * rs, qa[t].w * rs};
                    float b[4] = {qb[t].x * rs, qb[t].y * rs, qb[t].z * rs, qb[t].w * rs};
                    if (bias) {
                        const int col = (head0 + r / M) * HD + i;
#pragma unroll
                        for (int e = 0; e < 4; ++e) { a[e] += bias[col + e]; b[e] += bias[col + HD2 + e]; }
                    }
                    const float cs[4] = {c0[t].x, c0[t].z, c1[t].x, c1[t].z}, sn[4] = {c0[t].y, c0[t].w, c1[t].y, c1[t].w};
                    float x0[4], x1[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) { x0[e] = a[e] * cs[e] - b[e] * sn[e]; x1[e] = b[e] * cs[e] + a[e] * sn[e]; }
                    lo = make_uint2(pack_bf16(x0[0], x0[1]), pack_bf16(x0[2], x0[3]));
                    hi = make_uint2(pack_bf16(x1[0], x1[1]), pack_bf16(x1[2], x1[3]));
                }
                const int cA = i, cB = i + HD2;
                *reinterpret_cast<uint2*>(Qs + (cA >> 6) * (RP * 128) + swz_off(r, cA & 63)) = lo;
                *reinterpret_cast<uint2*>(Qs + (cB >> 6) * (RP * 128) + swz_off(r, cB & 63)) = hi;
            }
        }
    }
    // the new rows' own keys and values fit one block (M <= 32 <= KB)
    if (is_new) {
        uint8_t* Ks = KVs;
        uint8_t* Vs = Ks + KVBYTES;
        // K and V rows of the new tokens: finish the projection, rotate K, append to the cache
        for (int u = wtid; u < KB * UNITS; u += kWorkerThreads) {
            const int key = u / UNITS, q16 = u % UNITS, kk = key;
            uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
            if (kk < nkeys) {
                const float rs = rsqrtf(__ldcg(sumsq + r0 + kk) / (float)P.d + P.eps);
                const float* accrow = P.qkv_acc + (size_t)(r0 + kk) * P.n_qkv;
                const int colb = q16 * 8, ib = colb % HD2;  // 8 columns share one half of the rotary pairing
                const float* pa = accrow + Nq + hk * HD + ib;
                const float4 a0 = ldcg_f4(pa), a1 = ldcg_f4(pa + 4), b0 = ldcg_f4(pa + HD2), b1 = ldcg_f4(pa + HD2 + 4);
                const float* pv = accrow + Nq + Nkv + hk * HD + colb;
                const float4 v0 = ldcg_f4(pv), v1 = ldcg_f4(pv + 4);
                const int pk = TREE ? __ldcg(P.state + ST_DEPTH + kk) : kk;
                const float4* rp = reinterpret_cast<const float4*>(P.rope + (size_t)(L + pk) * HD2 + ib);
                const float4 r0 = __ldg(rp), r1 = __ldg(rp + 1), r2 = __ldg(rp + 2), r3 = __ldg(rp + 3);
                float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                float v[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                const float cs[8] = {r0.x, r0.z, r1.x, r1.z, r2.x, r2.z, r3.x, r3.z};
                const float sn[8] = {r0.y, r0.w, r1.y, r1.w, r2.y, r2.w, r3.y, r3.w};
                float kvals[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    a[e] *= rs; b[e] *= rs; v[e] *= rs;
                    if (bias) {
                        a[e] += bias[Nq + hk * HD + ib + e];
                        b[e] += bias[Nq + hk * HD + ib + HD2 + e];
                        v[e] += bias[Nq + Nkv + hk * HD + colb + e];
                    }
                    kvals[e] = (colb < HD2) ? (a[e] * cs[e] - b[e] * sn[e]) : (b[e] * cs[e] + a[e] * sn[e]);
                }
                kv4 = make_uint4(pack_bf16(kvals[0], kvals[1]), pack_bf16(kvals[2], kvals[3]),
                                 pack_bf16(kvals[4], kvals[5]), pack_bf16(kvals[6], kvals[7]));
                vv4 = make_uint4(pack_bf16(v[0], v[1]), pack_bf16(v[2], v[3]), pack_bf16(v[4], v[5]),
                                 pack_bf16(v[6], v[7]));
                if (qg == 0) {  // every head group computes the rows, one appends them
                    const size_t off = (cache_row0 + L + kk) * HD + q16 * 8;
                    *reinterpret_cast<uint4*>(kcache + off) = kv4;
                    *reinterpret_cast<uint4*>(vcache + off) = vv4;
                }
            }
            const uint32_t so = (q16 >> 3) * (KB * 128) + swz_unit(key, q16 & 7);
            *reinterpret_cast<uint4*>(Ks + so) = kv4;
            *reinterpret_cast<uint4*>(Vs + so) = vv4;
        }
    }
    if (prof && wtid == 0) prof[3] = global_timer_ns();

    const int g = lane >> 2, q2 = (lane & 3) * 2;
    const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
    const int j_lo = r_lo % M, j_hi = r_hi % M;
    // new keys a row may see: rows 0..j of a chain, its own path from the root in a tree
    const bool tree_mask = TREE && is_new;
    const unsigned see_lo = tree_mask ? (unsigned)__ldcg(P.state + ST_ANC + j_lo) : 0u;
    const unsigned see_hi = tree_mask ? (unsigned)__ldcg(P.state + ST_ANC + j_hi) : 0u;
    float o[NT_O][4];
#pragma unroll
    for (int n = 0; n < NT_O; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m_lo = -CUDART_INF_F, m_hi = -CUDART_INF_F, l_lo = 0.f, l_hi = 0.f;
    const uint32_t qb = smem_u32(Qs);

    for (int blk = 0; blk < nblk; ++blk) {
        if (!is_new) cp_async_wait<NBUF - 1>();
        named_bar_sync(1, kWorkerThreads);  // the block (and, first time, the Q tile) is in place
        if (prof && wtid == 0 && blk == 0) prof[4] = global_timer_ns();
        if (active) {
            const uint32_t kb = smem_u32(KVs + (blk % NBUF) * 2 * KVBYTES), vb = kb + KVBYTES;
            for (int c = kgp; c < KB / 16; c += KG) {
                if (blk * KB + c * 16 >= nkeys) break;
                // ---- scores of 16 rows x 16 keys
                float sc[2][4];
#pragma unroll
                for (int n = 0; n < 2; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
                    ldsm_x4(qb + (ks >> 2) * (RP * 128) + swz_unit(mt * 16 + (lane & 15), (ks & 3) * 2 + (lane >> 4)), a0, a1, a2, a3);
                    const int row = c * 16 + (lane & 7) + ((lane >> 4) << 3);
                    ldsm_x4(kb + (ks >> 2) * (KB * 128) + swz_unit(row, (ks & 3) * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
                    mma_bf16_16816(sc[0], a0, a1, a2, a3, b0, b1);
                    mma_bf16_16816(sc[1], a0, a1, a2, a3, b2, b3);
                }
                float mx_lo = -CUDART_INF_F, mx_hi = -CUDART_INF_F;
#pragma unroll
                for (int n = 0; n < 2; ++n)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int key = blk * KB + c * 16 + n * 8 + q2 + (e & 1);
                        const bool hi = e >= 2;
                        const int row = hi ? r_hi : r_lo, j = hi ? j_hi : j_lo;
                        bool ok = key < nkeys && row < R && (!is_new || key <= j);
                        if (TREE && tree_mask) ok = key < nkeys && row < R && (((hi ? see_hi : see_lo) >> (key & 31)) & 1u);
                        const float v = ok ? sc[n][e] * P.scale_log2e : -CUDART_INF_F;
                        sc[n][e] = v;
                        if (hi) mx_hi = fmaxf(mx_hi, v); else mx_lo = fmaxf(mx_lo, v);
                    }
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
                mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
                mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
                // ---- online softmax: new maximum, rescale, probabilities
                const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
                const float use_lo = (mn_lo == -CUDART_INF_F) ? 0.f : mn_lo, use_hi = (mn_hi == -CUDART_INF_F) ? 0.f : mn_hi;
                const float c_lo = exp2f(m_lo - use_lo), c_hi = exp2f(m_hi - use_hi);
                m_lo = mn_lo;
                m_hi = mn_hi;
                float p[2][4];
#pragma unroll
                for (int n = 0; n < 2; ++n) {
                    p[n][0] = exp2f(sc[n][0] - use_lo);
                    p[n][1] = exp2f(sc[n][1] - use_lo);
                    p[n][2] = exp2f(sc[n][2] - use_hi);
                    p[n][3] = exp2f(sc[n][3] - use_hi);
                }
                l_lo = l_lo * c_lo + p[0][0] + p[0][1] + p[1][0] + p[1][1];
                l_hi = l_hi * c_hi + p[0][2] + p[0][3] + p[1][2] + p[1][3];
#pragma unroll
                for (int n = 0; n < NT_O; ++n) { o[n][0] *= c_lo; o[n][1] *= c_lo; o[n][2] *= c_hi; o[n][3] *= c_hi; }
                // ---- O += P V: the score accumulators are, pairwise packed, the A operand of the next product
                const uint32_t a0 = pack_bf16(p[0][0], p[0][1]), a1 = pack_bf16(p[0][2], p[0][3]);
                const uint32_t a2 = pack_bf16(p[1][0], p[1][1]), a3 = pack_bf16(p[1][2], p[1][3]);
#pragma unroll
                for (int cg = 0; cg < NT_O / 2; ++cg) {
                    uint32_t b0, b1, b2, b3;
                    const int key = c * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                    const int cu = cg * 2 + (lane >> 4);
                    ldsm_x4_trans(vb + (cu >> 3) * (KB * 128) + swz_unit(key, cu & 7), b0, b1, b2, b3);
                    mma_bf16_16816(o[2 * cg], a0, a1, a2, a3, b0, b1);
                    mma_bf16_16816(o[2 * cg + 1], a0, a1, a2, a3, b2, b3);
                }
            }
        }
        named_bar_sync(1, kWorkerThreads);  // the block has been consumed
        if (!is_new) load_block(blk + NBUF);
    }
    if (!is_new) cp_async_wait<0>();
    if (prof && wtid == 0) prof[5] = global_timer_ns();

    // ---- row sums over the quad; the key groups of a row tile meet in shared memory
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    {
        float4* ex_o = reinterpret_cast<float4*>(KVs);          // [key group - 1][row tile][output tile][lane]
        float4* ex_ml = ex_o + 6 * NT_O * 32;                   // [key group - 1][row tile][lane]
        if (active && kgp > 0) {
            float4* dst = ex_o + ((kgp - 1) * MT + mt) * NT_O * 32;
#pragma unroll
            for (int n = 0; n < NT_O; ++n) dst[n * 32 + lane] = make_float4(o[n][0], o[n][1], o[n][2], o[n][3]);
            ex_ml[((kgp - 1) * MT + mt) * 32 + lane] = make_float4(m_lo, m_hi, l_lo, l_hi);
        }
        named_bar_sync(1, kWorkerThreads);
        if (active && kgp == 0) {
            for (int og = 0; og < KG - 1; ++og) {
                const float4 ml = ex_ml[(og * MT + mt) * 32 + lane];
                const float mn_lo = fmaxf(m_lo, ml.x), mn_hi = fmaxf(m_hi, ml.y);
                const float use_lo = (mn_lo == -CUDART_INF_F) ? 0.f : mn_lo, use_hi = (mn_hi == -CUDART_INF_F) ? 0.f : mn_hi;
                const float e0_lo = exp2f(m_lo - use_lo), e1_lo = exp2f(ml.x - use_lo);
                const float e0_hi = exp2f(m_hi - use_hi), e1_hi = exp2f(ml.y - use_hi);
                m_lo = mn_lo;
                m_hi = mn_hi;
                l_lo = l_lo * e0_lo + ml.z * e1_lo;
                l_hi = l_hi * e0_hi + ml.w * e1_hi;
                const float4* src = ex_o + (og * MT + mt) * NT_O * 32;
#pragma unroll
                for (int n = 0; n < NT_O; ++n) {
                    const float4 t = src[n * 32 + lane];
                    o[n][0] = o[n][0] * e0_lo + t.x * e1_lo;
                    o[n][1] = o[n][1] * e0_lo + t.y * e1_lo;
                    o[n][2] = o[n][2] * e0_hi + t.z * e1_hi;
                    o[n][3] = o[n][3] * e0_hi + t.w * e1_hi;
                }
            }
        }
    }

    // ---- un-normalised partial result of this key range
    if (active && kgp == 0) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? r_hi : r_lo;
            if (r >= R) continue;
            const int hq = head0 + r / M, j = r % M;
            const size_t row = ((size_t)hq * (kMaxSplits + 1) + s) * kMaxRows + r0 + j;
            float* po = P.part_o + row * HD + q2;
#pragma unroll
            for (int n = 0; n < NT_O; ++n)
                __stcg(reinterpret_cast<float2*>(po + n * 8), make_float2(o[n][half * 2], o[n][half * 2 + 1]));
            if ((lane & 3) == 0)
                __stcg(reinterpret_cast<float2*>(P.part_ml + row * 2), make_float2(half ? m_hi : m_lo, half ? l_hi : l_lo));
        }
    }
}

__device__ void attention_phase(const FwdParams& P, int layer, uint8_t* att, int wtid, unsigned long long* prof) {
    int S, kps;
    attn_split(P, S, kps);
    const int S1 = S + 1;
    const int gh = P.att_gh, QG = P.att_QG;
    const int per_seq = P.att_per_seq;
    const int nunits = per_seq * (P.nseq > 0 ? P.nseq : 1);
    for (int unit = blockIdx.x; unit < nunits; unit += P.G) {
        int b = P.att_b0, hk = P.att_hk0, qg = P.att_qg0, s = P.att_s0;
        if (unit != (int)blockIdx.x) {  // further units of this block (more units than blocks: batched steps)
            const int u = unit % per_seq, rem = u % (QG * S1);
            b = unit / per_seq;
            hk = u / (QG * S1);
            qg = rem / S1;
            s = rem % S1;
        }
        if (P.nseq > 0) {
            // every sequence takes the key ranges of the longest one; a range past its own length holds no key
            if (P.hd == 128) attention_unit<128, 2>(P, layer, hk, qg, gh, s, S, kps, att, wtid, prof, b);
            else attention_unit<64, 2>(P, layer, hk, qg, gh, s, S, kps, att, wtid, prof, b);
        } else if (P.tree) {
            if (P.hd == 128) attention_unit<128, 1>(P, layer, hk, qg, gh, s, S, kps, att, wtid, prof, 0);
            else attention_unit<64, 1>(P, layer, hk, qg, gh, s, S, kps, att, wtid, prof, 0);
        } else {
            if (P.hd == 128) attention_unit<128, 0>(P, layer, hk, qg, gh, s, S, kps, att, wtid, prof, 0);
            else attention_unit<64, 0>(P, layer, hk, qg, gh, s, S, kps, att, wtid, prof, 0);
        }
        named_bar_sync(1, kWorkerThreads);  // the unit's shared-memory tiles are free again
        if (prof && wtid == 0) { prof[6] = global_timer_ns(); prof[7] = (unsigned long long)(s == S); }
    }
}
// ------------------------------------------------------------------------------------------
__device__ void embed_phase(const FwdParams& P, int wtid) {
    // residual rows from the embedding table; rows beyond M are cleared
    const int units = kMaxRows * (P.d / 8);
    for (int u = blockIdx.x * kWorkerThreads + wtid; u < units; u += P.G * kWorkerThreads) {
        const int row = u / (P.d / 8), c8 = u % (P.d / 8);
        float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
        if (row < P.M) {
            int tok;
            if (P.mode == 1) tok = P.hist[P.L + row];
            else if (row == 0) tok = P.state[ST_PENDING];
            else tok = (row <= P.state[ST_DRAFT_LEN]) ? P.state[ST_DRAFT + row - 1] : 0;
            tok = min(max(tok, 0), P.V - 1);
            const uint4 raw = __ldg(reinterpret_cast<const uint4*>(P.emb + (size_t)tok * P.d + c8 * 8));
            const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&raw);
            const float2 f0 = __bfloat1622float2(pb[0]), f1 = __bfloat1622float2(pb[1]);
            const float2 f2 = __bfloat1622float2(pb[2]), f3 = __bfloat1622float2(pb[3]);
            lo = make_float4(f0.x, f0.y, f1.x, f1.y);
            hi = make_float4(f2.x, f2.y, f3.x, f3.y);
        }
        float* dst = P.h + (size_t)row * P.d + c8 * 8;
        __stcg(reinterpret_cast<float4*>(dst), lo);
        __stcg(reinterpret_cast<float4*>(dst + 4), hi);
    }
}
__device__ void zero_qkv_acc(const FwdParams& P, int sumsq_buf, int wtid) {
    const int n4 = kMaxRows * P.n_qkv / 4;
    for (int i = blockIdx.x * kWorkerThreads + wtid; i < n4; i += P.G * kWorkerThreads)
        __stcg(reinterpret_cast<float4*>(P.qkv_acc) + i, make_float4(0.f, 0.f, 0.f, 0.f));
    if (blockIdx.x == 0 && wtid < kMaxRows) __stcg(P.sumsq + sumsq_buf * kMaxRows + wtid, 0.f);
}


// ------------------------------------------------------------------------------------------
// One GEMM phase as seen by the worker warps: build the token operand, then the tensor-core
// thread walks the block's stages while the epilogue warps drain the accumulators.
__device__ __forceinline__ void advance_pos(PipePos& pos, const Part& pt, uint32_t nstage) {
    const uint32_t at = pos.slot + (uint32_t)(pt.npass * pt.nst);
    pos.slot = at % nstage;
    pos.par ^= (at / nstage) & 1u;
    pos.q += (uint32_t)pt.npass;
}

__device__ __forceinline__ void gemm_phase(const FwdParams& P, int kind, int layer, uint8_t* smem, Misc* misc, PipePos& pos, int wtid,
                                        unsigned long long* prof) {
    const int warp = wtid >> 5, lane = wtid & 31;
    uint8_t* U = smem + P.u_off;
    uint8_t* act = smem + P.act_off;
    int ops[2];
    const int nops = phase_ops(kind, ops);
    const Part& p0 = misc->part[ops[0]];
    const bool have0 = p0.ntiles > 0 && p0.nk > 0;
    bool dead = *(volatile int*)&misc->abort_flag != 0;
    if (wtid == 0) misc->prof_ptr = prof;

    if (warp == kMmaWarp) {
        // the tensor-core warp builds nothing: it prepares its descriptors and meets the others at the
        // operand barrier just before its first instruction
        PipePos mp = pos;
        mp.w_full = mp.w_acc = 0;
        const long long tc0 = clock64();
        bool synced = false;
        for (int oi = 0; oi < nops; ++oi) {
            const Part& pt = misc->part[ops[oi]];
            if (pt.ntiles == 0 || pt.nk == 0) continue;
            if (ops[oi] == OP_DOWN) {
                if (prof && lane == 0) prof[5] = global_timer_ns();
                if (!dead && !mbar_wait_bounded(&misc->act_ready, mp.act_uses & 1u, &misc->abort_flag, P.wait_limit_ns))
                    dead = true;
                dead = __any_sync(0xffffffffu, dead);
                tc_fence_after();
                if (prof && lane == 0) prof[6] = global_timer_ns();
            }
            mma_op(P, pt, smem, ops[oi] == OP_DOWN ? act : U, misc, mp, dead, synced);
        }
        if (!synced) named_bar_sync(1, kWorkerThreads);
        if (prof && lane == 0) {
            prof[3] = global_timer_ns();
            prof[7] = mp.w_full;
            prof[8] = mp.w_acc;
            prof[9] = (unsigned long long)(clock64() - tc0);  // cycles of the whole issue loop
        }
    } else {
        if (have0 && !dead) {
            if (kind == PH_O) build_merged_operand(P, p0, U, wtid);
            else build_norm_operand(P, kind, layer, p0, U, misc, wtid);
            fence_proxy_async_smem();
        }
        if (kind == PH_O && warp >= 4) {
            // clear the accumulators the next QKV projection adds into (idle warps)
            const int n4 = kMaxRows * P.n_qkv / 4, nth = (kBuilderWarps - 4) * 32;
            for (int i = blockIdx.x * nth + (wtid - 4 * 32); i < n4; i += P.G * nth)
                __stcg(reinterpret_cast<float4*>(P.qkv_acc) + i, make_float4(0.f, 0.f, 0.f, 0.f));
            if (blockIdx.x == 0 && wtid < 4 * 32 + kMaxRows)
                __stcg(P.sumsq + ((layer + 1) & 1) * kMaxRows + (wtid - 4 * 32), 0.f);
        }
        named_bar_sync(1, kWorkerThreads);  // the operand is complete and visible to the tensor core
        if (prof && wtid == 0) prof[2] = global_timer_ns();
    }
    if (warp < kEpilogueWarps) {
        PipePos ep = pos;
        if (P.NB == 32) epilogue_phase<32>(P, kind, layer, act, misc, ep, dead, warp, lane);
        else epilogue_phase<16>(P, kind, layer, act, misc, ep, dead, warp, lane);
        if (prof && wtid == 0) prof[4] = global_timer_ns();
    }
    // pipeline positions advance identically for every role
    for (int oi = 0; oi < nops; ++oi) {
        const Part& pt = misc->part[ops[oi]];
        if (pt.ntiles == 0 || pt.nk == 0) continue;
        advance_pos(pos, pt, (uint32_t)P.nstage);
        if (ops[oi] == OP_GU) ++pos.act_uses;
    }
}

// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 1) sdv_forward_kernel(const __grid_constant__ FwdParams Pg) {
    static_assert(sizeof(FwdParams) % 4 == 0, "parameter block is copied word by word");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Misc* misc = reinterpret_cast<Misc*>(smem + Pg.misc_off);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (Pg.l_from_state && Pg.state[ST_BUDGET] == 0) {
        // a step enqueued behind the end of its run: nothing to do, but the barrier counter moves as the host assumed
        if (tid == 0 && Pg.ph_end - Pg.ph_begin > 1) red_release_add_u32(Pg.bar, (unsigned)(Pg.ph_end - Pg.ph_begin - 1));
        return;
    }
    {
        const int* src = reinterpret_cast<const int*>(&Pg);
        int* dst = reinterpret_cast<int*>(&misc->P);
        for (int i = tid; i < (int)(sizeof(FwdParams) / 4); i += kThreads) dst[i] = src[i];
    }
    const FwdParams& P = misc->P;
    if (tid >= 32 && tid < 32 + OP_COUNT) misc->part[tid - 32] = get_part(Pg.op[tid - 32], Pg.op[OP_GU], blockIdx.x, Pg.G);

    if (tid == 0) {
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(&misc->full[s], 1);
            mbar_init(&misc->empty[s], 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&misc->tmem_full[b], 1);
            mbar_init(&misc->tmem_empty[b], kEpilogueWarps);
        }
        mbar_init(&misc->act_ready, kEpilogueWarps);
        mbar_init(&misc->done_bar, 1);
        misc->abort_flag = 0;
        misc->skip = 0;
        mbar_fence_init();
    }
    if (warp == kMmaWarp) tmem_alloc(&misc->tmem_base, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    // the first reader of L and of the key ranges (the attention phase) comes after a grid barrier, which orders
    // these writes before it
    if (tid == 0) {
        if (Pg.l_from_state) misc->P.L = Pg.state[ST_KV_LEN];
        attn_split_compute(misc->P, misc->P.att_S, misc->P.att_kps);
        // the block's first attention unit: the same for every layer, so its index arithmetic is done here
        FwdParams& Q = misc->P;
        const int S1 = Q.att_S + 1;
        Q.att_QG = (Q.g + Q.att_gh - 1) / Q.att_gh;
        Q.att_per_seq = Q.n_kv * Q.att_QG * S1;
        const int unit = blockIdx.x, u = unit % Q.att_per_seq, rem = u % (Q.att_QG * S1);
        Q.att_b0 = unit / Q.att_per_seq;
        Q.att_hk0 = u / (Q.att_QG * S1);
        Q.att_qg0 = rem / S1;
        Q.att_s0 = rem % S1;
    }

    if (warp == kProducerWarp) {
        if (lane == 0) producer_loop(P, smem, misc);
        return;
    }

    const int wtid = tid;  // 0 .. kWorkerThreads-1
    PipePos pos;
    pos.slot = pos.par = pos.q = pos.act_uses = pos.w_full = pos.w_acc = 0;
    int nbar = 0;
    bool skip = false;
    for (int ph = P.ph_begin; ph < P.ph_end; ++ph) {
        int layer;
        const int kind = decode_phase(ph, P.n_layers, layer);
        unsigned long long* pp = P.prof ? P.prof + ((size_t)(ph - P.ph_begin) * P.G + blockIdx.x) * kProfWords : nullptr;
        if (pp && wtid == 0) pp[0] = global_timer_ns();
        // after an abandoned wait the remaining phases do no work but still meet at every barrier
        if (skip) {
        } else if (kind == PH_EMBED) {
            embed_phase(P, wtid);
            zero_qkv_acc(P, 0, wtid);
        } else if (kind == PH_ATTN) {
            attention_phase(P, layer, smem + P.u_off, wtid, pp);
        } else {
            gemm_phase(P, kind, layer, smem, misc, pos, wtid, pp);
        }
        if (pp) {
            named_bar_sync(1, kWorkerThreads);
            if (wtid == 0) pp[1] = global_timer_ns();
        }
        if (ph + 1 < P.ph_end) {
            ++nbar;
            skip = grid_barrier(P, P.bar_base + (unsigned)(nbar * P.G), misc, wtid);
        }
    }
    // all tensor-core work must have completed before tensor memory is returned
    if (warp == kMmaWarp && lane == 0) {
        umma_commit(&misc->done_bar);
        mbar_wait_bounded(&misc->done_bar, 0, &misc->abort_flag, P.wait_limit_ns);
    }
    tc_fence_before();
    named_bar_sync(1, kWorkerThreads);
    tc_fence_after();
    if (warp == kMmaWarp) tmem_dealloc(misc->tmem_base, kTmemCols);
    if (*(volatile int*)&misc->abort_flag) {
        if (wtid == 0) atomicExch(P.state + ST_ERR, 1);
    }
}

}  // namespace sdv
