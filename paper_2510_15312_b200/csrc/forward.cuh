// The persistent forward kernel: one launch runs the decoder over M <= 8*NT token rows
// (a verify step over [T, x_1..x_k], or one tile of a prefill chunk).
//
// One thread block per SM, 12 warps:
//   warp 11      weight streamer: walks the block's static share of every GEMM in launch order
//                and keeps a ring of 16 KB shared-memory stages full with bulk asynchronous copies.
//                It never waits for activations or grid barriers, only for free ring slots, so HBM
//                traffic continues across operation boundaries.
//   warps 8..10  activation loaders: fill each stage's bf16 operand chunks ([rows x 64] each) from
//                L2, two chunks in flight per warp, applying the RMSNorm scale where one is due.
//   warps 0..7   MMA warps in an RW x KW grid: warp (rw, kw) multiplies row tile rw of the stage by
//                operand chunk kw (weights are the MMA "A" operand, token rows the 8-wide "B"
//                operand); epilogues are fused per operation.
// Operations are separated by a bounded grid barrier; attention and the split-KV merge use all 11
// non-producer warps.
#pragma once
#include <math_constants.h>

#include "layout.cuh"
#include "ptx.cuh"

namespace sdv {

enum PhaseKind { PH_EMBED = 0, PH_QKV, PH_ATTN, PH_COMB, PH_O, PH_GU, PH_DOWN, PH_LM, PH_RAW };
constexpr int kPhasesPerLayer = 6;

// Phase numbering of a launch: 0 = embedding; 1 + 6*layer + {0..5} = QKV, attention, split merge,
// output projection, gate|up, down; 1 + 6*n_layers = LM head; 2 + 6*n_layers = stand-alone GEMM.
__host__ __device__ __forceinline__ int decode_phase(int ph, int n_layers, int& layer) {
    layer = 0;
    if (ph == 0) return PH_EMBED;
    if (ph == 1 + kPhasesPerLayer * n_layers) return PH_LM;
    if (ph == 2 + kPhasesPerLayer * n_layers) return PH_RAW;
    layer = (ph - 1) / kPhasesPerLayer;
    return PH_QKV + (ph - 1) % kPhasesPerLayer;
}
__device__ __forceinline__ int phase_op(int kind) {
    switch (kind) {
        case PH_QKV: return OP_QKV;
        case PH_O: return OP_O;
        case PH_GU: return OP_GU;
        case PH_DOWN: return OP_DOWN;
        case PH_LM: return OP_LM;
        case PH_RAW: return OP_RAW;
        default: return -1;
    }
}
__device__ __forceinline__ const uint8_t* op_weights(const FwdParams& P, int kind, int layer) {
    if (kind == PH_LM) return P.wlm + P.op[OP_LM].w_off;
    if (kind == PH_RAW) return P.wraw + P.op[OP_RAW].w_off;
    return P.wlayers + (unsigned long long)layer * P.layer_stride + P.op[phase_op(kind)].w_off;
}

template <int NT>
struct SmemLayout {
    static constexpr int MP = 8 * NT;
    static constexpr int A_CHUNK = MP * 128;
    static constexpr int A_STAGE = kMaxKW * A_CHUNK;
    static constexpr int NSTAGE =
        (kSmemBudget - 1024 - kAttnSmemBytes - kMiscSmemBytes) / (kStageWeightBytes + A_STAGE);
    static constexpr int W_OFF = 0;
    static constexpr int A_OFF = NSTAGE * kStageWeightBytes;
    static constexpr int ATT_OFF = A_OFF + NSTAGE * A_STAGE;
    static constexpr int MISC_OFF = ATT_OFF + kAttnSmemBytes;
    static constexpr int TOTAL = MISC_OFF + kMiscSmemBytes + 1024;  // + slack for 1024-byte alignment
};

struct Misc {
    uint64_t full_w[16], full_a[16], empty[16];
    uint64_t rstd_bar;
    int abort_flag;
    int skip;  // block-uniform copy of abort_flag, refreshed inside every grid barrier
    float ss_part[4][kMaxRows];
    float best_v[kConsumerWarps][kMaxRows];
    int best_i[kConsumerWarps][kMaxRows];
    Part part[OP_COUNT];  // this block's share of every operation
    FwdParams P;  // block-local copy of the launch parameters (cheap to reach from out-of-line code)
};
static_assert(sizeof(Misc) <= kMiscSmemBytes, "misc shared memory");

// ------------------------------------------------------------------------------------------
// Grid barrier: every block adds one to a counter and waits (bounded) until all have.
// Called by all worker threads.  Returns, identically for all of them, whether some bounded
// wait in this block has been abandoned (the remaining phases then do no work).
__device__ __forceinline__ bool grid_barrier(const FwdParams& P, int target, Misc* misc, int wtid) {
    named_bar_sync(1, kWorkerThreads);
    if (wtid == 0) {
        __threadfence();
        red_add_s32(P.bar, 1);  // no return value to wait for: polling starts at once
        const uint64_t t0 = global_timer_ns();
        uint32_t spins = 0;
        while ((int)(ld_acquire_gpu(P.bar) - target) < 0) {
            if ((++spins & 63u) == 0) {
                if (*(volatile int*)&misc->abort_flag) break;
                if (global_timer_ns() - t0 > P.wait_limit_ns) {
                    *(volatile int*)&misc->abort_flag = 1;
                    break;
                }
            }
        }
        __threadfence();
        *(volatile int*)&misc->skip = *(volatile int*)&misc->abort_flag;
    }
    named_bar_sync(1, kWorkerThreads);
    return *(volatile int*)&misc->skip != 0;
}

// ------------------------------------------------------------------------------------------
// Weight streamer (one thread).
template <int NT>
__device__ __noinline__ void producer_loop(const FwdParams& P, uint8_t* smem, Misc* misc) {
    using SL = SmemLayout<NT>;
    const uint64_t policy = l2_policy_evict_first();
    uint32_t it = 0;
    const uint32_t ahead = (P.ahead >= 1 && P.ahead <= SL::NSTAGE) ? (uint32_t)P.ahead : (uint32_t)SL::NSTAGE;
    bool ok = true;
    for (int ph = P.ph_begin; ph < P.ph_end && ok; ++ph) {
        int layer;
        const int kind = decode_phase(ph, P.n_layers, layer);
        const int op = phase_op(kind);
        if (op < 0) continue;
        const Part& pt = misc->part[op];
        if (pt.ntiles == 0) continue;
        const int KW = 1 << pt.lkw;
        const uint8_t* src = op_weights(P, kind, layer) + pt.off;
        const int npass = pt.npass, nst = pt.nst;
        for (int p = 0; p < npass && ok; ++p) {
            const int pcount = pass_count(pt, p);
            for (int st = 0; st < nst; ++st, ++it) {
                const int kcnt = min(KW, pt.nchunks - st * KW);
                const uint32_t bytes = (uint32_t)(pcount * kcnt) * kTileBytes;
                const uint32_t slot = it % SL::NSTAGE;
                // run at most `ahead` stages in front of the MMA warps: stage it - ahead must be consumed
                if (it >= ahead) {
                    const uint32_t j = it - ahead;
                    if (!mbar_wait_bounded(&misc->empty[j % SL::NSTAGE], (j / SL::NSTAGE) & 1, &misc->abort_flag,
                                           P.wait_limit_ns)) {
                        ok = false;
                        break;
                    }
                }
                mbar_arrive_expect_tx(&misc->full_w[slot], bytes);
                bulk_g2s(smem + SL::W_OFF + slot * kStageWeightBytes, src, bytes, &misc->full_w[slot], policy);
                src += bytes;
            }
        }
    }
    if (!ok) {
        // Abandoned: wait (bounded) for the copies still in flight before the block may exit.
        const uint32_t issued = it;
        for (uint32_t back = 0; back < (uint32_t)SL::NSTAGE && back < issued; ++back) {
            const uint32_t j = issued - 1 - back;
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(&misc->full_w[j % SL::NSTAGE], (j / SL::NSTAGE) & 1)) {
                if (global_timer_ns() - t0 > P.wait_limit_ns) break;
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Activation loaders.  The operand chunks ([rows x 64] bf16 each) of a phase are dealt round-robin
// to the three loader warps.
//  - Ready-made operands (SwiGLU output, merged attention output) are already stored chunk by
//    chunk in the shared-memory image: one lane issues a bulk asynchronous copy per chunk straight
//    into the stage's slot, as far ahead as free slots allow.
//  - Operands that still need the RMSNorm scale: the chunk's fp32 residual rows and norm weights
//    are first staged in shared memory by 16-byte asynchronous copies (up to three chunks in flight
//    per warp, no registers held), then scaled, rounded to bf16 and stored into the slot.  The
//    row sums of squares fall out of the first pass.
constexpr int kRedBytes = 16384;  // staged-epilogue buffer at the start of the attention region
constexpr int kStageBufBytes = (kAttnSmemBytes - kRedBytes) / kLoaderWarps / 256 * 256;

__device__ __forceinline__ uint32_t chunk_arrivals(int c, int nchunks, int KW) {
    uint32_t cnt = kMaxKW / KW;
    if (c == nchunks - 1) cnt *= (uint32_t)(KW - ((nchunks - 1) & (KW - 1)));  // the last chunk covers a ragged stage
    return cnt;
}

template <int NT>
__device__ __noinline__ void loader_copy(const FwdParams& P, int kind, const OpDesc& od, const Part& pt, uint8_t* smem,
                                         Misc* misc, uint32_t it, uint32_t ci, int lw, int lane,
                                         unsigned long long* prof) {
    // The chunks of a stage are adjacent both in the operand buffer and in the stage's slot: one
    // bulk copy per stage, issued by one lane as far ahead as free slots allow.
    using SL = SmemLayout<NT>;
    const int KW = 1 << pt.lkw;
    const int npass = pt.npass, nst = pt.nst;
    const uint8_t* src_op = (kind == PH_O) ? P.attn_op : P.act;
    const uint32_t it0 = it;
    if (prof && lw == 0 && lane == 0) prof[6] = global_timer_ns();
    if (lw == 0 && lane == 0) {
        bool dead = *(volatile int*)&misc->abort_flag != 0;
        uint32_t sidx = it0;
        for (int p = 0; p < npass && !dead; ++p) {
            for (int st = 0; st < nst; ++st, ++sidx) {
                const uint32_t slot = sidx % SL::NSTAGE, use = sidx / SL::NSTAGE;
                if (use > 0 &&
                    !mbar_wait_bounded(&misc->empty[slot], (use - 1) & 1, &misc->abort_flag, P.wait_limit_ns)) {
                    dead = true;
                    break;
                }
                const int kcnt = min(KW, pt.nchunks - st * KW);
                const uint32_t bytes = (uint32_t)kcnt * SL::A_CHUNK;
                mbar_arrive_cnt(&misc->full_a[slot], kMaxKW - 1);
                mbar_arrive_expect_tx(&misc->full_a[slot], bytes);
                bulk_g2s_plain(smem + SL::A_OFF + slot * SL::A_STAGE,
                               src_op + (size_t)(pt.chunk0 + st * KW) * SL::A_CHUNK, bytes, &misc->full_a[slot]);
                if (prof && sidx == it0) prof[7] = global_timer_ns();
            }
        }
    }
    __syncwarp();
    if (prof && lw == 0 && lane == 0) prof[5] = global_timer_ns();
}

// A bounded wait that ran out marks the warp "dead": it stops touching the pipeline but still
// walks the control flow to the end.
template <int NT>
__device__ __noinline__ void loader_norm(const FwdParams& P, int kind, int layer, const OpDesc& od, const Part& pt,
                                         uint8_t* smem, Misc* misc, uint32_t it, uint32_t ci, int lw, int lane,
                                         unsigned long long* prof) {
    using SL = SmemLayout<NT>;
    const int KW = 1 << pt.lkw, lkw = pt.lkw;
    const int npass = pt.npass, nst = pt.nst;
    const int nchunks = pt.nchunks;
    const int M = P.M, d = P.d;
    const float* wn = P.norm_w + (size_t)(kind == PH_QKV ? layer * 2 : (kind == PH_GU ? layer * 2 + 1 : P.n_layers * 2)) * d;
    const float* hbase = P.h;
    float ss[2 * NT];
#pragma unroll
    for (int i = 0; i < 2 * NT; ++i) ss[i] = 0.f;
    bool dead = *(volatile int*)&misc->abort_flag != 0;
    const uint32_t it0 = it, ci0 = ci;
    const int total = npass * nchunks;  // chunk visits of this phase, pass-major
    const int x0 = (int)((lw + kLoaderWarps - (ci0 % kLoaderWarps)) % kLoaderWarps);
    const int nmine = (x0 < total) ? (total - x0 + kLoaderWarps - 1) / kLoaderWarps : 0;
    const int entry = (M + 1) * 256;  // M rows of 64 floats, then the 64 norm weights
    int D = kStageBufBytes / entry;
    if (D > 3) D = 3;
    if (D < 1) D = 1;
    uint8_t* stage = smem + SL::ATT_OFF + kRedBytes + lw * kStageBufBytes;
    if (prof && lw == 0 && lane == 0) prof[6] = global_timer_ns();

    int ic = x0;  // chunk index (within the partition) of the next visit to issue, kept below nchunks
    while (ic >= nchunks) ic -= nchunks;
    auto issue = [&](int k) {
        if (k < nmine) {
            const int chunk = pt.chunk0 + ic;
            ic += kLoaderWarps;
            while (ic >= nchunks) ic -= nchunks;
            uint8_t* dst = stage + (k % D) * entry;
            const int units = (M + 1) * 16;
            for (int u = lane; u < units; u += 32) {
                const int row = u >> 4, part = u & 15;
                const float* src = (row < M ? hbase + (size_t)row * d : wn) + chunk * 64 + part * 4;
                cp_async_16(dst + u * 16, src);
            }
        }
        cp_async_commit();  // possibly empty: keeps the group count uniform
    };
    auto publish = [&]() {
        // this warp's share of the per-row sums of squares (its first-pass chunks)
#pragma unroll
        for (int i = 0; i < 2 * NT; ++i) {
            float v = ss[i];
            v += __shfl_xor_sync(0xffffffffu, v, 1);
            v += __shfl_xor_sync(0xffffffffu, v, 2);
            v += __shfl_xor_sync(0xffffffffu, v, 4);
            const int tok = (lane + 32 * i) >> 3;
            if ((lane & 7) == 0) {
                if (kind == PH_QKV) {
                    // the attention step normalises q, k, v; only one row partition reports
                    if (pt.pr == 0 && tok < M && !dead) atomicAdd(P.sumsq + (layer & 1) * kMaxRows + tok, v);
                } else {
                    misc->ss_part[lw][tok] = v;
                }
            }
        }
        if (kind != PH_QKV) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&misc->rstd_bar);
        }
    };

    bool published = false;
    if (x0 >= nchunks) { publish(); published = true; }  // no first-pass chunk falls to this warp
    for (int k = 0; k < D; ++k) issue(k);
    int p_ = 0, c_ = x0;
    for (int k = 0; k < nmine; ++k, c_ += kLoaderWarps) {
        const int x = x0 + k * kLoaderWarps;
        while (c_ >= nchunks) { c_ -= nchunks; ++p_; }
        if (D == 3) cp_async_wait<2>(); else if (D == 2) cp_async_wait<1>(); else cp_async_wait<0>();
        __syncwarp();
        const uint32_t sidx = it0 + (uint32_t)(p_ * nst + (c_ >> lkw));
        const uint32_t slot = sidx % SL::NSTAGE, use = sidx / SL::NSTAGE;
        if (!dead && use > 0) {
            const bool got = mbar_wait_bounded(&misc->empty[slot], (use - 1) & 1, &misc->abort_flag, P.wait_limit_ns);
            if (!__all_sync(0xffffffffu, got)) dead = true;
        }
        if (!dead) {
            const uint8_t* src = stage + (k % D) * entry;
            uint8_t* dst = smem + SL::A_OFF + slot * SL::A_STAGE + (c_ & (KW - 1)) * SL::A_CHUNK;
            const int q = lane & 7;
            const float4 w0 = *reinterpret_cast<const float4*>(src + M * 256 + q * 32);
            const float4 w1 = *reinterpret_cast<const float4*>(src + M * 256 + q * 32 + 16);
#pragma unroll
            for (int i = 0; i < 2 * NT; ++i) {
                const int tok = (lane + 32 * i) >> 3;
                uint4 out = make_uint4(0, 0, 0, 0);
                if (tok < M) {
                    const float4 a = *reinterpret_cast<const float4*>(src + tok * 256 + q * 32);
                    const float4 b = *reinterpret_cast<const float4*>(src + tok * 256 + q * 32 + 16);
                    if (p_ == 0)
                        ss[i] += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w + b.x * b.x + b.y * b.y + b.z * b.z +
                                 b.w * b.w;
                    out.x = pack_bf16(a.x * w0.x, a.y * w0.y);
                    out.y = pack_bf16(a.z * w0.z, a.w * w0.w);
                    out.z = pack_bf16(b.x * w1.x, b.y * w1.y);
                    out.w = pack_bf16(b.z * w1.z, b.w * w1.w);
                }
                *reinterpret_cast<uint4*>(dst + swz_unit(tok, q)) = out;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_cnt(&misc->full_a[slot], chunk_arrivals(c_, nchunks, KW));
            if (prof && k == 0 && lw == 0 && lane == 0) prof[7] = global_timer_ns();
        }
        __syncwarp();   // every lane is done with the staging entry before it is refilled
        issue(k + D);
        if (!published && x + kLoaderWarps >= nchunks) { publish(); published = true; }
    }
    cp_async_wait<0>();
    if (!published) publish();
    if (prof && lw == 0 && lane == 0) prof[5] = global_timer_ns();
}

// ------------------------------------------------------------------------------------------
// MMA warps.
template <int NT>
__device__ __noinline__ void consumer_phase(const FwdParams& P, int kind, int layer, const OpDesc& od, const Part& pt, uint8_t* smem,
                               Misc* misc, uint32_t it, uint32_t norm_uses, int warp, int lane,
                               unsigned long long* prof) {
    using SL = SmemLayout<NT>;
    constexpr int MP = SL::MP;
    const int RW = od.RW, KW = 1 << pt.lkw;
    const int rw = warp & (RW - 1), kw = warp >> (3 - pt.lkw);
    const int npass = pt.npass, nst = pt.nst;
    const int g = lane >> 2, q2 = (lane & 3) * 2;
    const bool need_rstd = (kind == PH_GU || kind == PH_LM);
    const bool staged = (kind == PH_QKV || kind == PH_O || kind == PH_DOWN || kind == PH_RAW);
    float rstd[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) rstd[nt][0] = rstd[nt][1] = 0.f;
    bool have_rstd = false;
    bool dead = *(volatile int*)&misc->abort_flag != 0;
    // running arg-max for the LM head: token slots (nt, e)
    float bv[NT][2];
    int bi[NT][2];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
        bv[nt][0] = bv[nt][1] = -CUDART_INF_F;
        bi[nt][0] = bi[nt][1] = 0x7fffffff;
    }
    float* red = reinterpret_cast<float*>(smem + SL::ATT_OFF);  // [8 warps][MP][16] partial tiles (staged epilogue)
    uint64_t wait_w = 0, wait_a = 0, mma_cycles = 0, mma_stages = 0;

    for (int p = 0; p < npass; ++p) {
        const int pcount = pass_count(pt, p);
        const int tile_base = pt.tile0 + pass_start(pt, p);
        const int tile = tile_base + rw;
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;

        for (int st = 0; st < nst; ++st, ++it) {
            const uint32_t slot = it % SL::NSTAGE, par = (it / SL::NSTAGE) & 1;
            if (!dead) {
                const uint64_t tw0 = prof ? global_timer_ns() : 0;
                bool got = mbar_wait_bounded(&misc->full_w[slot], par, &misc->abort_flag, P.wait_limit_ns);
                const uint64_t tw1 = prof ? global_timer_ns() : 0;
                got = got && mbar_wait_bounded(&misc->full_a[slot], par, &misc->abort_flag, P.wait_limit_ns);
                if (prof && warp == 0 && lane == 0) {
                    const uint64_t tw2 = global_timer_ns();
                    wait_w += tw1 - tw0;
                    wait_a += tw2 - tw1;
                }
                if (!__all_sync(0xffffffffu, got)) dead = true;
            }
            if (dead) continue;
            if (prof && p == 0 && st == 0 && warp == 0 && lane == 0) prof[2] = global_timer_ns();
            const long long c0 = prof ? clock64() : 0;
            const int kcnt = min(KW, pt.nchunks - st * KW);
            if (rw < pcount && kw < kcnt) {
                const uint32_t wbase =
                    smem_u32(smem + SL::W_OFF + slot * kStageWeightBytes + (kw * pcount + rw) * kTileBytes);
                const uint32_t abase = smem_u32(smem + SL::A_OFF + slot * SL::A_STAGE + kw * SL::A_CHUNK);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t a0, a1, a2, a3;
                    ldsm_x4(wbase + swz_unit(lane & 15, ks * 2 + (lane >> 4)), a0, a1, a2, a3);
#pragma unroll
                    for (int np = 0; np < NT / 2; ++np) {
                        uint32_t b0, b1, b2, b3;
                        const int row = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                        ldsm_x4(abase + swz_unit(row, ks * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
                        mma_bf16_16816(acc[2 * np], a0, a1, a2, a3, b0, b1);
                        mma_bf16_16816(acc[2 * np + 1], a0, a1, a2, a3, b2, b3);
                    }
                    if (NT & 1) {
                        uint32_t b0, b1;
                        const int row = (NT - 1) * 8 + (lane & 7);
                        ldsm_x2(abase + swz_unit(row, ks * 2 + ((lane >> 3) & 1)), b0, b1);
                        mma_bf16_16816(acc[NT - 1], a0, a1, a2, a3, b0, b1);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&misc->empty[slot]);
            if (prof) { mma_cycles += (uint64_t)(clock64() - c0); ++mma_stages; }
        }

        if (prof && p == npass - 1 && warp == 0 && lane == 0) prof[3] = global_timer_ns();
        if (need_rstd && !have_rstd && !dead) {
            const bool got = mbar_wait_bounded(&misc->rstd_bar, norm_uses & 1, &misc->abort_flag, P.wait_limit_ns);
            if (!__all_sync(0xffffffffu, got)) dead = true;
        }
        if (need_rstd && !have_rstd && !dead) {
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int n = nt * 8 + q2 + e;
                    float s = 0.f;
#pragma unroll
                    for (int w = 0; w < kLoaderWarps; ++w) s += misc->ss_part[w][n];
                    rstd[nt][e] = rsqrtf(s / (float)P.d + P.eps);
                }
            have_rstd = true;
        }

        // ---------------- epilogues
        if (staged) {
            // partial tiles meet in shared memory: the KW column splits are summed there and each
            // thread then owns 4 adjacent output rows of one token (one 16-byte global operation)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int n = nt * 8 + q2 + e;
                    red[(warp * MP + n) * 16 + g] = acc[nt][e];
                    red[(warp * MP + n) * 16 + g + 8] = acc[nt][2 + e];
                }
            named_bar_sync(2, kConsumerWarps * 32);
            if (!dead) {
                float* out;
                int stride;
                if (kind == PH_QKV) { out = P.qkv_acc; stride = P.n_qkv; }
                else if (kind == PH_RAW) { out = P.raw_out; stride = P.raw_N; }
                else { out = P.h; stride = P.d; }
                const int M = P.M, ngroups = pcount * 4 * M;
                for (int idx = warp * 32 + lane; idx < ngroups; idx += kConsumerWarps * 32) {
                    const int rwi = idx / (4 * M), rem = idx % (4 * M), n = rem >> 2, r4 = rem & 3;
                    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int kwi = 0; kwi < KW; ++kwi) {
                        const float4 t =
                            *reinterpret_cast<const float4*>(red + ((kwi * RW + rwi) * MP + n) * 16 + r4 * 4);
                        v.x += t.x; v.y += t.y; v.z += t.z; v.w += t.w;
                    }
                    float* dst = out + (size_t)n * stride + (tile_base + rwi) * 16 + r4 * 4;
                    if (od.P_k > 1) {
                        red_add_v4_f32(dst, v);
                    } else if (kind == PH_QKV || kind == PH_RAW) {
                        __stcg(reinterpret_cast<float4*>(dst), v);  // sole owner of a zeroed buffer
                    } else {
                        const float4 o = ldcg_f4(dst);  // sole owner: residual add in place
                        __stcg(reinterpret_cast<float4*>(dst), make_float4(o.x + v.x, o.y + v.y, o.z + v.z, o.w + v.w));
                    }
                }
            }
            named_bar_sync(2, kConsumerWarps * 32);
            continue;
        }
        if (warp >= pcount || dead) continue;  // RW = 8 here: one tile per warp

        if (kind == PH_GU) {
            const int fi = tile * 8 + g;  // rows 0..7 of the tile are gate rows, 8..15 the matching up rows
            uint8_t* dst = P.act + (size_t)(fi >> 6) * SL::A_CHUNK;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int n = nt * 8 + q2 + e;
                    float v = 0.f;
                    if (n < P.M) {
                        const float x = acc[nt][e] * rstd[nt][e], y = acc[nt][2 + e] * rstd[nt][e];
                        v = x / (1.f + expf(-x)) * y;
                    }
                    *reinterpret_cast<__nv_bfloat16*>(dst + swz_off(n, fi & 63)) = __float2bfloat16(v);
                }
        } else if (kind == PH_LM) {
            const int r0 = tile * 16 + g;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int n = nt * 8 + q2 + e;
                    const float v0 = acc[nt][e] * rstd[nt][e], v1 = acc[nt][2 + e] * rstd[nt][e];
                    if (P.store_logits && n < P.M) {
                        __stcg(P.logits + (size_t)n * P.V + r0, v0);
                        __stcg(P.logits + (size_t)n * P.V + r0 + 8, v1);
                    }
                    // rows come in ascending order per thread, so ">" keeps the lowest id among equals
                    if (v0 > bv[nt][e]) { bv[nt][e] = v0; bi[nt][e] = r0; }
                    if (v1 > bv[nt][e]) { bv[nt][e] = v1; bi[nt][e] = r0 + 8; }
                }
        }
    }
    if (prof && warp == 0 && lane == 0) {
        prof[4] = global_timer_ns();
        prof[8] = wait_w;
        prof[9] = wait_a;
        prof[10] = mma_cycles;  // SM clock cycles between the waits' end and the slot's release, all stages
        prof[11] = mma_stages;
    }

    if (kind == PH_LM) {
        // best over the 8 row groups of the warp, then over the 8 warps
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                float v = bv[nt][e];
                int i = bi[nt][e];
#pragma unroll
                for (int off = 4; off <= 16; off <<= 1) {
                    const float ov = __shfl_xor_sync(0xffffffffu, v, off);
                    const int oi = __shfl_xor_sync(0xffffffffu, i, off);
                    if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
                }
                if (g == 0) {
                    misc->best_v[warp][nt * 8 + q2 + e] = v;
                    misc->best_i[warp][nt * 8 + q2 + e] = i;
                }
            }
        named_bar_sync(2, kConsumerWarps * 32);
        const int t = warp * 32 + lane;
        if (t < MP && !dead) {
            float v = misc->best_v[0][t];
            int i = misc->best_i[0][t];
            for (int w = 1; w < kConsumerWarps; ++w) {
                const float ov = misc->best_v[w][t];
                const int oi = misc->best_i[w][t];
                if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
            }
            P.cand_val[(size_t)blockIdx.x * kMaxRows + t] = v;
            P.cand_idx[(size_t)blockIdx.x * kMaxRows + t] = i;
        }
    }
}

// ------------------------------------------------------------------------------------------
// Split-KV attention.  The committed cache [0, L) is cut into S key ranges of kps keys (a multiple
// of 64, as many ranges as there are blocks to take them); unit (kv head, s < S) attends all
// query rows of the head group to range s; unit (kv head, S) covers the M new rows: it finishes
// their K/V projection (norm scale, bias, rotary), appends them to the cache and attends to them
// under the causal mask (row j sees new keys 0..j).  Partial results are merged afterwards.
//
// Inside a unit the R = (query heads per KV head) x M rows form MT tiles of 16 rows and the keys
// come in blocks of KB (64 while the row tile leaves room, else 32).  A block takes three short
// steps, each spread over all 11 worker warps as independent tasks so that no warp runs a long
// dependent chain:
//   A  scores: task (row tile, 16 keys) = Q K^T on tensor cores, scaled and masked, kept in
//      registers; per-row maxima of the 16 keys go to shared memory;
//   B  same tasks: block maximum per row from the partial maxima, probabilities exp2(s - m),
//      written as bf16 over the K block (no longer needed), partial row sums to shared memory;
//   C  output: task (row tile, 16 head columns) = rescale the running output, add P V.
// Running maximum, sum and rescale factor per row live in shared memory.
__device__ __forceinline__ void attn_split(const FwdParams& P, int& S, int& kps) {
    if (P.L <= 0) { S = 0; kps = 0; return; }
    int cap = P.G / P.n_kv - 1;
    if (cap > kMaxSplits) cap = kMaxSplits;
    if (cap < 1) cap = 1;
    kps = ((P.L + cap - 1) / cap + 63) / 64 * 64;
    S = (P.L + kps - 1) / kps;
}

constexpr int kAttnStatsOff = 49152;  // row statistics behind the Q | K | V tiles

template <int HD, bool BIG>  // BIG: more than 64 query rows (4 row tiles)
__device__ __noinline__ void attention_unit(const FwdParams& P, int layer, int hk, int s, int S, int kps, uint8_t* att, int wtid,
                                            unsigned long long* prof) {
    constexpr int HD2 = HD / 2;
    constexpr int KSTEPS = HD / 16;
    constexpr int UNITS = HD / 8;   // 16-byte units per K/V row
    constexpr int CG = HD / 16;     // 16-column groups of the output
    constexpr int NWARPS = kWorkerThreads / 32;
    constexpr int TA_MAX = 2;                                // score tasks per warp (at most 16 tasks)
    constexpr int TC_MAX = ((BIG ? 8 : 4) * CG + NWARPS - 1) / NWARPS;  // output tasks per warp
    constexpr int KB = BIG ? 32 : 64, lng = BIG ? 1 : 2, NG = 1 << lng;  // keys per block; 16-key groups
    const int warp = wtid >> 5, lane = wtid & 31;
    const int M = P.M, L = P.L, R = P.g * M;
    const int MT = (R + 15) >> 4, RP = MT * 16;
    const bool is_new = (s == S);
    uint8_t* Qs = att;
    uint8_t* Ks = att + RP * HD * 2;
    uint8_t* Vs = Ks + KB * HD * 2;
    // probabilities: over the keys once the scores are done (head_dim 128, where the tiles fill the
    // region), else in the free space behind the tiles
    uint8_t* Pb = (HD == 128) ? Ks : att + 32768;
    float* st_m = reinterpret_cast<float*>(att + kAttnStatsOff);  // [2][128] running maximum, by block parity
    float* st_l = st_m + 256;                                     // [128] running sum
    float* st_corr = st_l + 128;                                  // [128] rescale factor of this block
    float* st_pmax = st_corr + 128;                               // [RP][NG] per-task maxima
    float* st_psum = st_pmax + 256;                               // [RP][NG] per-task sums
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
        for (int u = wtid; u < KB * UNITS; u += kWorkerThreads) {
            const int key = u / UNITS, q16 = u % UNITS, kk = blk * KB + key;
            const bool valid = kk < nkeys;
            const size_t off = (cache_row0 + t_begin + (valid ? kk : 0)) * HD + q16 * 8;
            const uint32_t so = (q16 >> 3) * (KB * 128) + swz_unit(key, q16 & 7);
            cp_async_16_zfill(Ks + so, P.kcache + off, valid);
            cp_async_16_zfill(Vs + so, P.vcache + off, valid);
        }
        cp_async_commit();
    };
    if (prof && wtid == 0) prof[2] = global_timer_ns();
    if (!is_new && nblk > 0) load_block(0);
    if (wtid < 128) {
        st_m[wtid] = -CUDART_INF_F;
        st_l[wtid] = 0.f;
    }

    // ---- query tile: normalise, add bias, rotate, round to bf16; 4 rotary pairs per item
    {
        const int items = RP * (HD2 / 4);
        for (int base = wtid; base < items; base += 2 * kWorkerThreads) {
            float4 qa[2], qb[2], c0[2], c1[2];
            float ssq[2];
            int rr[2], ii[2];
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int idx = base + t * kWorkerThreads;
                rr[t] = idx / (HD2 / 4);
                ii[t] = (idx % (HD2 / 4)) * 4;
                ssq[t] = 0.f;
                qa[t] = qb[t] = c0[t] = c1[t] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (idx < items && rr[t] < R) {
                    const int hl = rr[t] / M, j = rr[t] % M, col = (hk * P.g + hl) * HD + ii[t];
                    ssq[t] = __ldcg(sumsq + j);
                    qa[t] = ldcg_f4(P.qkv_acc + (size_t)j * P.n_qkv + col);
                    qb[t] = ldcg_f4(P.qkv_acc + (size_t)j * P.n_qkv + col + HD2);
                    const float4* rp = reinterpret_cast<const float4*>(P.rope + (size_t)(L + j) * HD2 + ii[t]);
                    c0[t] = __ldg(rp);
                    c1[t] = __ldg(rp + 1);
                }
            }
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int idx = base + t * kWorkerThreads;
                if (idx >= items) continue;
                const int r = rr[t], i = ii[t];
                uint2 lo = make_uint2(0, 0), hi = make_uint2(0, 0);
                if (r < R) {
                    const float rs = rsqrtf(ssq[t] / (float)P.d + P.eps);
                    float a[4] = {qa[t].x * rs, qa[t].y * rs, qa[t].z * rs, qa[t].w * rs};
                    float b[4] = {qb[t].x * rs, qb[t].y * rs, qb[t].z * rs, qb[t].w * rs};
                    if (bias) {
                        const int col = (hk * P.g + r / M) * HD + i;
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
        // K and V rows of the new tokens: finish the projection, rotate K, append to the cache
        for (int u = wtid; u < KB * UNITS; u += kWorkerThreads) {
            const int key = u / UNITS, q16 = u % UNITS, kk = key;
            uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
            if (kk < nkeys) {
                const float rs = rsqrtf(__ldcg(sumsq + kk) / (float)P.d + P.eps);
                const float* accrow = P.qkv_acc + (size_t)kk * P.n_qkv;
                const int colb = q16 * 8, ib = colb % HD2;  // 8 columns share one half of the rotary pairing
                const float* pa = accrow + Nq + hk * HD + ib;
                const float4 a0 = ldcg_f4(pa), a1 = ldcg_f4(pa + 4), b0 = ldcg_f4(pa + HD2), b1 = ldcg_f4(pa + HD2 + 4);
                const float* pv = accrow + Nq + Nkv + hk * HD + colb;
                const float4 v0 = ldcg_f4(pv), v1 = ldcg_f4(pv + 4);
                const float4* rp = reinterpret_cast<const float4*>(P.rope + (size_t)(L + kk) * HD2 + ib);
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
                const size_t off = (cache_row0 + L + kk) * HD + q16 * 8;
                *reinterpret_cast<uint4*>(P.kcache + off) = kv4;
                *reinterpret_cast<uint4*>(P.vcache + off) = vv4;
            }
            const uint32_t so = (q16 >> 3) * (KB * 128) + swz_unit(key, q16 & 7);
            *reinterpret_cast<uint4*>(Ks + so) = kv4;
            *reinterpret_cast<uint4*>(Vs + so) = vv4;
        }
    }
    if (prof && wtid == 0) prof[3] = global_timer_ns();

    const int g = lane >> 2, q2 = (lane & 3) * 2;
    const int ntaskA = MT << lng, ntaskC = MT * CG;
    // byte offset of 16-byte unit `unit` of row r in the probability tile (swizzled against bank conflicts)
    auto p_unit = [&](uint32_t r, uint32_t unit) -> uint32_t {
        return KB == 64 ? swz_unit(r, unit) : r * 64u + (((unit ^ (r >> 1)) & 3u) << 4);
    };
    float o[TC_MAX][2][4];
#pragma unroll
    for (int t = 0; t < TC_MAX; ++t)
#pragma unroll
        for (int n = 0; n < 2; ++n) o[t][n][0] = o[t][n][1] = o[t][n][2] = o[t][n][3] = 0.f;

    for (int blk = 0; blk < nblk; ++blk) {
        const int par = blk & 1;
        if (!is_new) {
            if (blk > 0) load_block(blk);
            cp_async_wait<0>();
        }
        named_bar_sync(1, kWorkerThreads);  // K/V block (and, first time, the Q tile and the row statistics) are in place
        if (prof && wtid == 0 && blk == 0) prof[4] = global_timer_ns();

        // ---- A: scores of (row tile, 16 keys), kept in registers
        float sc[TA_MAX][2][4];
        const uint32_t qb = smem_u32(Qs), kb = smem_u32(Ks), vb = smem_u32(Vs), pb = smem_u32(Pb);
#pragma unroll
        for (int ti = 0; ti < TA_MAX; ++ti) {
            const int task = warp + ti * NWARPS;
            if (task >= ntaskA) continue;
            const int mt = task >> lng, kg = task & (NG - 1);
#pragma unroll
            for (int n = 0; n < 2; ++n) sc[ti][n][0] = sc[ti][n][1] = sc[ti][n][2] = sc[ti][n][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
                ldsm_x4(qb + (ks >> 2) * (RP * 128) + swz_unit(mt * 16 + (lane & 15), (ks & 3) * 2 + (lane >> 4)), a0, a1, a2,
                        a3);
                const int row = kg * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldsm_x4(kb + (ks >> 2) * (KB * 128) + swz_unit(row, (ks & 3) * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
                mma_bf16_16816(sc[ti][0], a0, a1, a2, a3, b0, b1);
                mma_bf16_16816(sc[ti][1], a0, a1, a2, a3, b2, b3);
            }
            const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
            const int j_lo = r_lo % M, j_hi = r_hi % M;
            float mx_lo = -CUDART_INF_F, mx_hi = -CUDART_INF_F;
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = blk * KB + kg * 16 + n * 8 + q2 + (e & 1);
                    const bool hi = e >= 2;
                    const int row = hi ? r_hi : r_lo, j = hi ? j_hi : j_lo;
                    const bool ok = key < nkeys && row < R && (!is_new || key <= j);
                    const float v = ok ? sc[ti][n][e] * P.scale_log2e : -CUDART_INF_F;
                    sc[ti][n][e] = v;
                    if (hi) mx_hi = fmaxf(mx_hi, v); else mx_lo = fmaxf(mx_lo, v);
                }
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
            if ((lane & 3) == 0) {
                st_pmax[(r_lo << lng) + kg] = mx_lo;
                st_pmax[(r_hi << lng) + kg] = mx_hi;
            }
        }
        named_bar_sync(1, kWorkerThreads);  // partial maxima are visible; the K block has been read

        // ---- B: probabilities
#pragma unroll
        for (int ti = 0; ti < TA_MAX; ++ti) {
            const int task = warp + ti * NWARPS;
            if (task >= ntaskA) continue;
            const int mt = task >> lng, kg = task & (NG - 1);
            const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
            float mb_lo = st_pmax[r_lo << lng], mb_hi = st_pmax[r_hi << lng];
            for (int i = 1; i < NG; ++i) {
                mb_lo = fmaxf(mb_lo, st_pmax[(r_lo << lng) + i]);
                mb_hi = fmaxf(mb_hi, st_pmax[(r_hi << lng) + i]);
            }
            const float mo_lo = st_m[par * 128 + r_lo], mo_hi = st_m[par * 128 + r_hi];
            const float mn_lo = fmaxf(mo_lo, mb_lo), mn_hi = fmaxf(mo_hi, mb_hi);
            const float use_lo = (mn_lo == -CUDART_INF_F) ? 0.f : mn_lo, use_hi = (mn_hi == -CUDART_INF_F) ? 0.f : mn_hi;
            float sum_lo = 0.f, sum_hi = 0.f;
#pragma unroll
            for (int n = 0; n < 2; ++n) {
                const float p0 = exp2f(sc[ti][n][0] - use_lo), p1 = exp2f(sc[ti][n][1] - use_lo);
                const float p2 = exp2f(sc[ti][n][2] - use_hi), p3 = exp2f(sc[ti][n][3] - use_hi);
                sum_lo += p0 + p1;
                sum_hi += p2 + p3;
                const uint32_t unit = (uint32_t)(kg * 2 + n);
                *reinterpret_cast<uint32_t*>(Pb + p_unit(r_lo, unit) + q2 * 2) = pack_bf16(p0, p1);
                *reinterpret_cast<uint32_t*>(Pb + p_unit(r_hi, unit) + q2 * 2) = pack_bf16(p2, p3);
            }
            sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 1);
            sum_lo += __shfl_xor_sync(0xffffffffu, sum_lo, 2);
            sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 1);
            sum_hi += __shfl_xor_sync(0xffffffffu, sum_hi, 2);
            if ((lane & 3) == 0) {
                st_psum[(r_lo << lng) + kg] = sum_lo;
                st_psum[(r_hi << lng) + kg] = sum_hi;
                if (kg == 0) {
                    st_corr[r_lo] = exp2f(mo_lo - use_lo);
                    st_corr[r_hi] = exp2f(mo_hi - use_hi);
                    st_m[(par ^ 1) * 128 + r_lo] = mn_lo;
                    st_m[(par ^ 1) * 128 + r_hi] = mn_hi;
                }
            }
        }
        named_bar_sync(1, kWorkerThreads);  // probabilities, sums and rescale factors are visible

        // ---- C: O = O * corr + P V for (row tile, 16 columns)
#pragma unroll
        for (int tj = 0; tj < TC_MAX; ++tj) {
            const int task = warp + tj * NWARPS;
            if (task >= ntaskC) continue;
            const int mt = task / CG, cg = task % CG;
            const int r_lo = mt * 16 + g, r_hi = r_lo + 8;
            const float c_lo = st_corr[r_lo], c_hi = st_corr[r_hi];
#pragma unroll
            for (int n = 0; n < 2; ++n) { o[tj][n][0] *= c_lo; o[tj][n][1] *= c_lo; o[tj][n][2] *= c_hi; o[tj][n][3] *= c_hi; }
            for (int k2 = 0; k2 < NG; ++k2) {
                uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
                ldsm_x4(pb + p_unit(mt * 16 + (lane & 15), k2 * 2 + (lane >> 4)), a0, a1, a2, a3);
                const int key = k2 * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                const int cu = cg * 2 + (lane >> 4);
                ldsm_x4_trans(vb + (cu >> 3) * (KB * 128) + swz_unit(key, cu & 7), b0, b1, b2, b3);
                mma_bf16_16816(o[tj][0], a0, a1, a2, a3, b0, b1);
                mma_bf16_16816(o[tj][1], a0, a1, a2, a3, b2, b3);
            }
            if (cg == 0 && (lane & 3) == 0) {
                float s_lo = 0.f, s_hi = 0.f;
                for (int i = 0; i < NG; ++i) {
                    s_lo += st_psum[(r_lo << lng) + i];
                    s_hi += st_psum[(r_hi << lng) + i];
                }
                st_l[r_lo] = st_l[r_lo] * c_lo + s_lo;
                st_l[r_hi] = st_l[r_hi] * c_hi + s_hi;
            }
        }
        named_bar_sync(1, kWorkerThreads);  // the block has been consumed; row statistics are up to date
    }

    // ---- un-normalised partial result of this key range
    if (prof && wtid == 0) prof[5] = global_timer_ns();
#pragma unroll
    for (int tj = 0; tj < TC_MAX; ++tj) {
        const int task = warp + tj * NWARPS;
        if (task >= ntaskC) continue;
        const int mt = task / CG, cg = task % CG;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = mt * 16 + g + half * 8;
            if (r >= R) continue;
            const int hq = hk * P.g + r / M, j = r % M;
            const size_t row = ((size_t)hq * (kMaxSplits + 1) + s) * kMaxRows + j;
            float* po = P.part_o + row * HD + cg * 16 + q2;
            __stcg(reinterpret_cast<float2*>(po), make_float2(o[tj][0][half * 2], o[tj][0][half * 2 + 1]));
            __stcg(reinterpret_cast<float2*>(po + 8), make_float2(o[tj][1][half * 2], o[tj][1][half * 2 + 1]));
        }
    }
    if (wtid < R) {
        const int hq = hk * P.g + wtid / M, j = wtid % M;
        const size_t row = ((size_t)hq * (kMaxSplits + 1) + s) * kMaxRows + j;
        __stcg(reinterpret_cast<float2*>(P.part_ml + row * 2), make_float2(st_m[(nblk & 1) * 128 + wtid], st_l[wtid]));
    }
}

__device__ void attention_phase(const FwdParams& P, int layer, uint8_t* att, int wtid, unsigned long long* prof) {
    int S, kps;
    attn_split(P, S, kps);
    const int S1 = S + 1;
    const int nunits = P.n_kv * S1;
    for (int unit = blockIdx.x; unit < nunits; unit += P.G) {
        const int hk = unit / S1, s = unit % S1;
        const bool big = P.g * P.M > 64;
        if (P.hd == 128) {
            if (big) attention_unit<128, true>(P, layer, hk, s, S, kps, att, wtid, prof);
            else attention_unit<128, false>(P, layer, hk, s, S, kps, att, wtid, prof);
        } else {
            if (big) attention_unit<64, true>(P, layer, hk, s, S, kps, att, wtid, prof);
            else attention_unit<64, false>(P, layer, hk, s, S, kps, att, wtid, prof);
        }
        named_bar_sync(1, kWorkerThreads);  // the unit's shared-memory tiles are free again
        if (prof && wtid == 0) { prof[6] = global_timer_ns(); prof[7] = (unsigned long long)(s == S); }
    }
}

// Merge of the split-KV partial results into the output projection's bf16 operand.  One warp per
// (query head, row, 8 columns); lanes run over the splits.
template <int NT>
__device__ __noinline__ void combine_phase(const FwdParams& P, int wtid) {
    constexpr int A_CHUNK = SmemLayout<NT>::A_CHUNK;
    int S, kps;
    attn_split(P, S, kps);
    const int S1 = S + 1;
    const int warp = wtid >> 5, lane = wtid & 31;
    const int U8 = P.hd / 8, nwarps = kWorkerThreads / 32;
    const int items = P.n_q * P.M * U8;
    for (int item = blockIdx.x * nwarps + warp; item < items; item += P.G * nwarps) {
        const int hq = item / (P.M * U8), j = (item / U8) % P.M, c8 = item % U8;
        const size_t base = ((size_t)hq * (kMaxSplits + 1)) * kMaxRows + j;
        float m[2], l[2];
        float4 a[2], b[2];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int s = lane + 32 * t;
            m[t] = -CUDART_INF_F; l[t] = 0.f;
            a[t] = b[t] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (s < S1) {
                const size_t row = base + (size_t)s * kMaxRows;
                const float2 ml = __ldcg(reinterpret_cast<const float2*>(P.part_ml + row * 2));
                m[t] = ml.x; l[t] = ml.y;
                const float* op = P.part_o + row * P.hd + c8 * 8;
                a[t] = ldcg_f4(op);
                b[t] = ldcg_f4(op + 4);
            }
        }
        float mmax = fmaxf(m[0], m[1]);
#pragma unroll
        for (int off = 16; off; off >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, off));
        const float w0 = exp2f(m[0] - mmax), w1 = exp2f(m[1] - mmax);  // 0 for splits that saw no key
        float v[9];
        v[0] = w0 * a[0].x + w1 * a[1].x; v[1] = w0 * a[0].y + w1 * a[1].y; v[2] = w0 * a[0].z + w1 * a[1].z;
        v[3] = w0 * a[0].w + w1 * a[1].w; v[4] = w0 * b[0].x + w1 * b[1].x; v[5] = w0 * b[0].y + w1 * b[1].y;
        v[6] = w0 * b[0].z + w1 * b[1].z; v[7] = w0 * b[0].w + w1 * b[1].w; v[8] = w0 * l[0] + w1 * l[1];
#pragma unroll
        for (int e = 0; e < 9; ++e)
#pragma unroll
            for (int off = 16; off; off >>= 1) v[e] += __shfl_xor_sync(0xffffffffu, v[e], off);
        if (lane == 0) {
            const float inv = 1.f / v[8];
            const int col = hq * P.hd + c8 * 8;
            const uint4 out = make_uint4(pack_bf16(v[0] * inv, v[1] * inv), pack_bf16(v[2] * inv, v[3] * inv),
                                         pack_bf16(v[4] * inv, v[5] * inv), pack_bf16(v[6] * inv, v[7] * inv));
            *reinterpret_cast<uint4*>(P.attn_op + (size_t)(col >> 6) * A_CHUNK + swz_unit(j, (col & 63) >> 3)) = out;
        }
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
template <int NT>
__global__ void __launch_bounds__(kThreads, 1) sdv_forward_kernel(const __grid_constant__ FwdParams Pg) {
    using SL = SmemLayout<NT>;
    static_assert(SL::NSTAGE >= 4 && SL::NSTAGE <= 16, "ring depth");
    static_assert(kConsumerWarps * SL::MP * 16 * 4 <= kRedBytes, "staged epilogue buffer");
    static_assert(sizeof(FwdParams) % 4 == 0, "parameter block is copied word by word");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Misc* misc = reinterpret_cast<Misc*>(smem + SL::MISC_OFF);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    {
        const int* src = reinterpret_cast<const int*>(&Pg);
        int* dst = reinterpret_cast<int*>(&misc->P);
        for (int i = tid; i < (int)(sizeof(FwdParams) / 4); i += kThreads) dst[i] = src[i];
    }
    const FwdParams& P = misc->P;
    if (tid >= 32 && tid < 32 + OP_COUNT) misc->part[tid - 32] = get_part(Pg.op[tid - 32], blockIdx.x, Pg.G);

    if (tid == 0) {
        for (int s = 0; s < SL::NSTAGE; ++s) {
            mbar_init(&misc->full_w[s], 1);
            mbar_init(&misc->full_a[s], kMaxKW);
            mbar_init(&misc->empty[s], kConsumerWarps);
        }
        mbar_init(&misc->rstd_bar, kLoaderWarps);
        misc->abort_flag = 0;
        misc->skip = 0;
        mbar_fence_init();
    }
    __syncthreads();

    if (warp == kConsumerWarps + kLoaderWarps) {
        if (lane == 0) producer_loop<NT>(P, smem, misc);
        return;
    }

    const int wtid = tid;  // 0 .. kWorkerThreads-1
    uint32_t it = 0, ci = 0, norm_uses = 0;
    int nbar = 0;
    bool skip = false;
    for (int ph = P.ph_begin; ph < P.ph_end; ++ph) {
        int layer;
        const int kind = decode_phase(ph, P.n_layers, layer);
        if (P.prof && wtid == 0) P.prof[((size_t)(ph - P.ph_begin) * P.G + blockIdx.x) * kProfWords] = global_timer_ns();
        // after an abandoned wait the remaining phases do no work but still meet at every barrier
        if (skip) {
        } else if (kind == PH_EMBED) {
            embed_phase(P, wtid);
            zero_qkv_acc(P, 0, wtid);
        } else if (kind == PH_ATTN) {
            attention_phase(P, layer, smem + SL::ATT_OFF, wtid,
                            P.prof ? P.prof + ((size_t)(ph - P.ph_begin) * P.G + blockIdx.x) * kProfWords : nullptr);
        } else if (kind == PH_COMB) {
            combine_phase<NT>(P, wtid);
        } else {
            if (kind == PH_O) zero_qkv_acc(P, (layer + 1) & 1, wtid);
            const OpDesc& od = P.op[phase_op(kind)];
            const Part& pt = misc->part[phase_op(kind)];
            if (pt.ntiles > 0) {
                unsigned long long* pp =
                    P.prof ? P.prof + ((size_t)(ph - P.ph_begin) * P.G + blockIdx.x) * kProfWords : nullptr;
                if (warp < kConsumerWarps) {
                    consumer_phase<NT>(P, kind, layer, od, pt, smem, misc, it, norm_uses, warp, lane, pp);
                } else {
                    const bool norm = (kind == PH_QKV || kind == PH_GU || kind == PH_LM);
                    if (norm) loader_norm<NT>(P, kind, layer, od, pt, smem, misc, it, ci, warp - kConsumerWarps, lane, pp);
                    else loader_copy<NT>(P, kind, od, pt, smem, misc, it, ci, warp - kConsumerWarps, lane, pp);
                }
                // pipeline positions advance identically for every role
                it += (uint32_t)(pt.npass * pt.nst);
                ci += (uint32_t)(pt.npass * pt.nchunks);
                if (kind == PH_GU || kind == PH_LM) ++norm_uses;
            }
        }
        if (P.prof) {
            named_bar_sync(1, kWorkerThreads);
            if (wtid == 0) P.prof[((size_t)(ph - P.ph_begin) * P.G + blockIdx.x) * kProfWords + 1] = global_timer_ns();
        }
        if (ph + 1 < P.ph_end) {
            ++nbar;
            skip = grid_barrier(P, P.bar_base + nbar * P.G, misc, wtid);
        }
    }
    if (*(volatile int*)&misc->abort_flag) {
        if (wtid == 0) atomicExch(P.state + ST_ERR, 1);
    }
}

}  // namespace sdv
