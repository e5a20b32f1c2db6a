// The persistent forward kernel: one launch runs the decoder over M <= 8*NT token rows
// (a verify step over [T, x_1..x_k], or one tile of a prefill chunk).
//
// One thread block per SM, 12 warps:
//   warp 11      weight streamer: walks the block's static share of every GEMM in launch order
//                and keeps a ring of 16 KB shared-memory stages full with bulk asynchronous copies.
//                It never waits for activations or grid barriers, only for free ring slots, so HBM
//                traffic continues across operation boundaries.
//   warps 8..10  activation loaders: fill each stage's [rows x 64] bf16 operand from L2, applying
//                the producing step's deferred work (RMSNorm scale, split-KV combine).
//   warps 0..7   MMA warps: one 16-row weight tile each per stage (weights are the MMA "A" operand,
//                token rows the 8-wide "B" operand), epilogues fused per operation.
// Operations are separated by a bounded grid barrier; attention uses all 11 non-producer warps.
#pragma once
#include <math_constants.h>

#include "layout.cuh"
#include "ptx.cuh"

namespace sdv {

enum PhaseKind { PH_EMBED = 0, PH_QKV, PH_ATTN, PH_O, PH_GU, PH_DOWN, PH_LM, PH_RAW };

// Phase numbering of a launch: 0 = embedding; 1 + 5*layer + {0..4} = QKV, attention, output
// projection, gate|up, down; 1 + 5*n_layers = LM head; 2 + 5*n_layers = the stand-alone GEMM.
__device__ __forceinline__ int decode_phase(int ph, int n_layers, int& layer) {
    layer = 0;
    if (ph == 0) return PH_EMBED;
    if (ph == 1 + 5 * n_layers) return PH_LM;
    if (ph == 2 + 5 * n_layers) return PH_RAW;
    layer = (ph - 1) / 5;
    return PH_QKV + (ph - 1) % 5;
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
    static constexpr int A_STAGE = MP * 128;
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
};
static_assert(sizeof(Misc) <= kMiscSmemBytes, "misc shared memory");

// ------------------------------------------------------------------------------------------
// Grid barrier: every block adds one to a counter and waits (bounded) until all have.
// Called by all worker threads.  Returns, identically for all of them, whether some bounded
// wait in this block has been abandoned (the remaining phases then do no work).
__device__ __forceinline__ bool grid_barrier(const FwdParams& P, int target, Misc* misc, int wtid) {
    __threadfence();  // every thread's own stores and reductions are performed before it reports in
    named_bar_sync(1, kWorkerThreads);
    if (wtid == 0) {
        __threadfence();
        atomicAdd(P.bar, 1);
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
__device__ void producer_loop(const FwdParams& P, uint8_t* smem, Misc* misc) {
    using SL = SmemLayout<NT>;
    const int cta = blockIdx.x;
    const uint64_t policy = l2_policy_evict_first();
    uint32_t it = 0;
    bool ok = true;
    for (int ph = P.ph_begin; ph < P.ph_end && ok; ++ph) {
        int layer;
        const int kind = decode_phase(ph, P.n_layers, layer);
        const int op = phase_op(kind);
        if (op < 0) continue;
        const Part pt = get_part(P.op[op], cta, P.G);
        if (pt.ntiles == 0) continue;
        const uint8_t* src = op_weights(P, kind, layer) + pt.off;
        const int npass = part_passes(pt);
        for (int p = 0; p < npass && ok; ++p) {
            const uint32_t bytes = (uint32_t)even_count(pt.ntiles, npass, p) * kTileBytes;
            for (int c = 0; c < pt.nchunks; ++c, ++it) {
                const uint32_t slot = it % SL::NSTAGE, use = it / SL::NSTAGE;
                if (use > 0 && !mbar_wait_bounded(&misc->empty[slot], (use - 1) & 1, &misc->abort_flag,
                                                  P.wait_limit_ns)) {
                    ok = false;
                    break;
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
// Activation loaders.  Loader warp w fills the operand of every stage with index = w mod 3.
template <int NT>
__device__ __forceinline__ void load_norm_chunk(const FwdParams& P, const float* wn, int col0, uint8_t* dst, int lane,
                                                float (&ss)[2 * NT], bool accumulate) {
#pragma unroll
    for (int i = 0; i < 2 * NT; ++i) {
        const int u = lane + 32 * i, tok = u >> 3, q = u & 7;
        uint4 out = make_uint4(0, 0, 0, 0);
        if (tok < P.M) {
            const float* hp = P.h + (size_t)tok * P.d + col0 + q * 8;
            const float4 a = ldcg_f4(hp), b = ldcg_f4(hp + 4);
            const float4 wa = __ldg(reinterpret_cast<const float4*>(wn + col0 + q * 8));
            const float4 wb = __ldg(reinterpret_cast<const float4*>(wn + col0 + q * 8 + 4));
            if (accumulate)
                ss[i] += a.x * a.x + a.y * a.y + a.z * a.z + a.w * a.w + b.x * b.x + b.y * b.y + b.z * b.z + b.w * b.w;
            out.x = pack_bf16(a.x * wa.x, a.y * wa.y);
            out.y = pack_bf16(a.z * wa.z, a.w * wa.w);
            out.z = pack_bf16(b.x * wb.x, b.y * wb.y);
            out.w = pack_bf16(b.z * wb.z, b.w * wb.w);
        }
        *reinterpret_cast<uint4*>(dst + swz_unit(tok, q)) = out;
    }
}

template <int NT>
__device__ __forceinline__ void load_copy_chunk(const uint8_t* src, uint8_t* dst, int lane) {
#pragma unroll
    for (int i = 0; i < 2 * NT; ++i) {
        const int u = lane + 32 * i;
        *reinterpret_cast<uint4*>(dst + u * 16) = ldcg_u4(src + u * 16);
    }
}

__device__ __forceinline__ int attn_splits(int L) {
    if (L <= 0) return 0;
    const int s = (L + kSplitTargetKeys - 1) / kSplitTargetKeys;
    return s < kMaxSplits ? s : kMaxSplits;
}
__device__ __forceinline__ int attn_keys_per_split(int L, int S) {
    const int k = (L + S - 1) / S;
    return (k + kAttnBlockKeys - 1) / kAttnBlockKeys * kAttnBlockKeys;
}

// Operand of the output projection: merge the split-KV partial results of one head's columns.
template <int NT>
__device__ __forceinline__ void load_combine_chunk(const FwdParams& P, int col0, uint8_t* dst, int lane) {
    const int hq = col0 / P.hd, co = col0 % P.hd;
    const int S1 = attn_splits(P.L) + 1;
#pragma unroll 1
    for (int i = 0; i < 2 * NT; ++i) {
        const int u = lane + 32 * i, tok = u >> 3, q = u & 7;
        uint4 out = make_uint4(0, 0, 0, 0);
        if (tok < P.M) {
            const size_t base = ((size_t)hq * (kMaxSplits + 1)) * kMaxRows + tok;
            float mmax = -CUDART_INF_F;
            for (int s = 0; s < S1; ++s)
                mmax = fmaxf(mmax, __ldcg(P.part_ml + (base + (size_t)s * kMaxRows) * 2));
            float den = 0.f, acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            for (int s = 0; s < S1; ++s) {
                const size_t row = base + (size_t)s * kMaxRows;
                const float2 ml = __ldcg(reinterpret_cast<const float2*>(P.part_ml + row * 2));
                const float wgt = exp2f(ml.x - mmax);  // 0 for a split that saw no key (m = -inf)
                den += wgt * ml.y;
                const float* op = P.part_o + row * P.hd + co + q * 8;
                const float4 a = ldcg_f4(op), b = ldcg_f4(op + 4);
                acc[0] += wgt * a.x; acc[1] += wgt * a.y; acc[2] += wgt * a.z; acc[3] += wgt * a.w;
                acc[4] += wgt * b.x; acc[5] += wgt * b.y; acc[6] += wgt * b.z; acc[7] += wgt * b.w;
            }
            const float inv = 1.f / den;
            out.x = pack_bf16(acc[0] * inv, acc[1] * inv);
            out.y = pack_bf16(acc[2] * inv, acc[3] * inv);
            out.z = pack_bf16(acc[4] * inv, acc[5] * inv);
            out.w = pack_bf16(acc[6] * inv, acc[7] * inv);
        }
        *reinterpret_cast<uint4*>(dst + swz_unit(tok, q)) = out;
    }
}

// A bounded wait that ran out marks the warp "dead": it stops touching the pipeline but still
// walks the control flow, so that every named barrier is reached by all of its threads.
template <int NT>
__device__ void loader_phase(const FwdParams& P, int kind, int layer, const Part& pt, uint8_t* smem, Misc* misc,
                             uint32_t& it, int lw, int lane) {
    using SL = SmemLayout<NT>;
    const int npass = part_passes(pt);
    const bool is_norm = (kind == PH_QKV || kind == PH_GU || kind == PH_LM);
    const float* wn = nullptr;
    if (kind == PH_QKV) wn = P.norm_w + (size_t)(layer * 2 + 0) * P.d;
    if (kind == PH_GU) wn = P.norm_w + (size_t)(layer * 2 + 1) * P.d;
    if (kind == PH_LM) wn = P.norm_w + (size_t)(P.n_layers * 2) * P.d;
    float ss[2 * NT];
#pragma unroll
    for (int i = 0; i < 2 * NT; ++i) ss[i] = 0.f;
    bool dead = *(volatile int*)&misc->abort_flag != 0;
    for (int p = 0; p < npass; ++p) {
        for (int c = 0; c < pt.nchunks; ++c, ++it) {
            if ((int)(it % kLoaderWarps) != lw) continue;
            const uint32_t slot = it % SL::NSTAGE, use = it / SL::NSTAGE;
            if (!dead && use > 0) {
                const bool got = mbar_wait_bounded(&misc->empty[slot], (use - 1) & 1, &misc->abort_flag, P.wait_limit_ns);
                if (!__all_sync(0xffffffffu, got)) dead = true;
            }
            if (dead) continue;
            uint8_t* dst = smem + SL::A_OFF + slot * SL::A_STAGE;
            const int chunk = pt.chunk0 + c;
            if (is_norm) {
                load_norm_chunk<NT>(P, wn, chunk * 64, dst, lane, ss, p == 0);
            } else if (kind == PH_O) {
                load_combine_chunk<NT>(P, chunk * 64, dst, lane);
            } else {
                load_copy_chunk<NT>(P.act + (size_t)chunk * SL::A_STAGE, dst, lane);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&misc->full_a[slot]);
        }
        if (p == 0 && is_norm) {
            // per-row sums of squares of the columns this warp handled
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
                        if (pt.pr == 0 && tok < P.M && !dead) atomicAdd(P.sumsq + (layer & 1) * kMaxRows + tok, v);
                    } else {
                        misc->ss_part[lw][tok] = v;
                    }
                }
            }
            if (kind != PH_QKV) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&misc->rstd_bar);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// MMA warps.
template <int NT>
__device__ void consumer_phase(const FwdParams& P, int kind, int layer, const Part& pt, uint8_t* smem, Misc* misc,
                               uint32_t& it, uint32_t& norm_uses, int warp, int lane) {
    using SL = SmemLayout<NT>;
    constexpr int MP = SL::MP;
    const int npass = part_passes(pt);
    const int g = lane >> 2, q2 = (lane & 3) * 2;
    const bool need_rstd = (kind == PH_GU || kind == PH_LM);
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

    for (int p = 0; p < npass; ++p) {
        const int pcount = even_count(pt.ntiles, npass, p);
        const int tile = pt.tile0 + even_start(pt.ntiles, npass, p) + warp;
        const bool active = warp < pcount;
        float acc[NT][4];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f;

        for (int c = 0; c < pt.nchunks; ++c, ++it) {
            const uint32_t slot = it % SL::NSTAGE, par = (it / SL::NSTAGE) & 1;
            if (!dead) {
                const bool got = mbar_wait_bounded(&misc->full_w[slot], par, &misc->abort_flag, P.wait_limit_ns) &&
                                 mbar_wait_bounded(&misc->full_a[slot], par, &misc->abort_flag, P.wait_limit_ns);
                if (!__all_sync(0xffffffffu, got)) dead = true;
            }
            if (dead) continue;
            if (active) {
                const uint32_t wbase = smem_u32(smem + SL::W_OFF + slot * kStageWeightBytes + warp * kTileBytes);
                const uint32_t abase = smem_u32(smem + SL::A_OFF + slot * SL::A_STAGE);
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
        }

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
        if (!active || dead) continue;

        // ---------------- epilogues
        if (kind == PH_QKV || kind == PH_O || kind == PH_DOWN || kind == PH_RAW) {
            float* out;
            int stride;
            if (kind == PH_QKV) { out = P.qkv_acc; stride = P.n_qkv; }
            else if (kind == PH_RAW) { out = P.raw_out; stride = P.raw_N; }
            else { out = P.h; stride = P.d; }
            const int r0 = tile * 16 + g;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int n = nt * 8 + q2 + e;
                    if (n < P.M) {
                        red_add_f32(out + (size_t)n * stride + r0, acc[nt][e]);
                        red_add_f32(out + (size_t)n * stride + r0 + 8, acc[nt][2 + e]);
                    }
                }
        } else if (kind == PH_GU) {
            const int fi = tile * 8 + g;  // rows 0..7 of the tile are gate rows, 8..15 the matching up rows
            uint8_t* dst = P.act + (size_t)(fi >> 6) * (MP * 128);
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
    if (need_rstd) ++norm_uses;

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
// Attention over one (KV head, key range) unit for all query rows of the head group.
// Unit s < S covers cache keys [s*kps, min(L, (s+1)*kps)); unit s == S covers the M new rows:
// it finishes their K/V projection (norm scale, bias, rotary), appends them to the cache and
// attends to them under the causal mask (row j sees new keys 0..j).
template <int HD>
__device__ void attention_unit(const FwdParams& P, int layer, int hk, int s, int S, int kps, uint8_t* att, int wtid) {
    constexpr int HD2 = HD / 2;
    constexpr int KSTEPS = HD / 16;
    constexpr int UNITS = HD / 8;  // 16-byte units per K/V row
    const int warp = wtid >> 5, lane = wtid & 31;
    const int M = P.M, L = P.L, R = P.g * M;
    const int MT = (R + 15) >> 4, RP = MT * 16;
    const bool is_new = (s == S);
    uint8_t* Qs = att;
    uint8_t* Ks = att + 32768;
    uint8_t* Vs = att + 32768 + 8192;
    const float* sumsq = P.sumsq + (layer & 1) * kMaxRows;
    const float* bias = P.bias ? P.bias + (size_t)layer * P.n_qkv : nullptr;
    const int Nq = P.n_q * HD, Nkv = P.n_kv * HD;

    // ---- query tile: normalise, add bias, rotate, round to bf16
    for (int idx = wtid; idx < RP * HD2; idx += kWorkerThreads) {
        const int r = idx / HD2, i = idx % HD2;
        float q0 = 0.f, q1 = 0.f;
        if (r < R) {
            const int hl = r / M, j = r % M, col = (hk * P.g + hl) * HD + i;
            const float rs = rsqrtf(__ldcg(sumsq + j) / (float)P.d + P.eps);
            float a = rs * __ldcg(P.qkv_acc + (size_t)j * P.n_qkv + col);
            float b = rs * __ldcg(P.qkv_acc + (size_t)j * P.n_qkv + col + HD2);
            if (bias) { a += bias[col]; b += bias[col + HD2]; }
            const float2 cs = __ldg(P.rope + (size_t)(L + j) * HD2 + i);
            q0 = a * cs.x - b * cs.y;
            q1 = b * cs.x + a * cs.y;
        }
        const int c0 = i, c1 = i + HD2;
        *reinterpret_cast<__nv_bfloat16*>(Qs + (c0 >> 6) * (RP * 128) + swz_off(r, c0 & 63)) = __float2bfloat16(q0);
        *reinterpret_cast<__nv_bfloat16*>(Qs + (c1 >> 6) * (RP * 128) + swz_off(r, c1 & 63)) = __float2bfloat16(q1);
    }

    int t_begin = 0, nkeys = M;
    if (!is_new) {
        t_begin = s * kps;
        const int t_end = min(L, t_begin + kps);
        nkeys = max(0, t_end - t_begin);
    }
    const int nblk = (nkeys + kAttnBlockKeys - 1) / kAttnBlockKeys;
    const size_t cache_row0 = ((size_t)layer * P.n_kv + hk) * P.max_seq;

    const int g = lane >> 2, q2 = (lane & 3) * 2;
    const int r_lo = warp * 16 + g, r_hi = r_lo + 8;
    const int j_lo = r_lo % M, j_hi = r_hi % M;
    float m_lo = -CUDART_INF_F, m_hi = -CUDART_INF_F, l_lo = 0.f, l_hi = 0.f;
    float o[HD / 8][4];
#pragma unroll
    for (int n = 0; n < HD / 8; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

    for (int blk = 0; blk < nblk; ++blk) {
        named_bar_sync(1, kWorkerThreads);  // previous block consumed (and, first time, Q tile written)
        for (int u = wtid; u < kAttnBlockKeys * UNITS; u += kWorkerThreads) {
            const int key = u / UNITS, q16 = u % UNITS, kk = blk * kAttnBlockKeys + key;
            uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
            if (kk < nkeys) {
                if (is_new) {
                    const float rs = rsqrtf(__ldcg(sumsq + kk) / (float)P.d + P.eps);
                    const float* accrow = P.qkv_acc + (size_t)kk * P.n_qkv;
                    float kvals[8], vvals[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const int col = q16 * 8 + e, i = col % HD2;
                        const int ka = Nq + hk * HD + i, kb = ka + HD2, vc = Nq + Nkv + hk * HD + col;
                        float a = rs * __ldcg(accrow + ka), b = rs * __ldcg(accrow + kb), v = rs * __ldcg(accrow + vc);
                        if (bias) { a += bias[ka]; b += bias[kb]; v += bias[vc]; }
                        const float2 cs = __ldg(P.rope + (size_t)(L + kk) * HD2 + i);
                        kvals[e] = (col < HD2) ? (a * cs.x - b * cs.y) : (b * cs.x + a * cs.y);
                        vvals[e] = v;
                    }
                    kv4 = make_uint4(pack_bf16(kvals[0], kvals[1]), pack_bf16(kvals[2], kvals[3]),
                                     pack_bf16(kvals[4], kvals[5]), pack_bf16(kvals[6], kvals[7]));
                    vv4 = make_uint4(pack_bf16(vvals[0], vvals[1]), pack_bf16(vvals[2], vvals[3]),
                                     pack_bf16(vvals[4], vvals[5]), pack_bf16(vvals[6], vvals[7]));
                    const size_t off = (cache_row0 + L + kk) * HD + q16 * 8;
                    *reinterpret_cast<uint4*>(P.kcache + off) = kv4;
                    *reinterpret_cast<uint4*>(P.vcache + off) = vv4;
                } else {
                    const size_t off = (cache_row0 + t_begin + kk) * HD + q16 * 8;
                    kv4 = ldcg_u4(P.kcache + off);
                    vv4 = ldcg_u4(P.vcache + off);
                }
            }
            const uint32_t so = (q16 >> 3) * (kAttnBlockKeys * 128) + swz_unit(key, q16 & 7);
            *reinterpret_cast<uint4*>(Ks + so) = kv4;
            *reinterpret_cast<uint4*>(Vs + so) = vv4;
        }
        named_bar_sync(1, kWorkerThreads);
        if (warp >= MT) continue;

        // ---- S = Q K^T for 16 rows x 32 keys
        float sc[4][4];
#pragma unroll
        for (int n = 0; n < 4; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
        const uint32_t qb = smem_u32(Qs), kb = smem_u32(Ks), vb = smem_u32(Vs);
#pragma unroll
        for (int ks = 0; ks < KSTEPS; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldsm_x4(qb + (ks >> 2) * (RP * 128) + swz_unit(warp * 16 + (lane & 15), (ks & 3) * 2 + (lane >> 4)), a0, a1,
                    a2, a3);
#pragma unroll
            for (int np = 0; np < 2; ++np) {
                uint32_t b0, b1, b2, b3;
                const int row = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldsm_x4(kb + (ks >> 2) * (kAttnBlockKeys * 128) + swz_unit(row, (ks & 3) * 2 + ((lane >> 3) & 1)), b0, b1,
                        b2, b3);
                mma_bf16_16816(sc[2 * np], a0, a1, a2, a3, b0, b1);
                mma_bf16_16816(sc[2 * np + 1], a0, a1, a2, a3, b2, b3);
            }
        }
        // ---- mask, online softmax (log2 domain)
        float mx_lo = -CUDART_INF_F, mx_hi = -CUDART_INF_F;
#pragma unroll
        for (int n = 0; n < 4; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int key = blk * kAttnBlockKeys + n * 8 + q2 + (e & 1);
                const bool hi = e >= 2;
                const int row = hi ? r_hi : r_lo, j = hi ? j_hi : j_lo;
                const bool ok = key < nkeys && row < R && (!is_new || key <= j);
                const float v = ok ? sc[n][e] * P.scale_log2e : -CUDART_INF_F;
                sc[n][e] = v;
                if (hi) mx_hi = fmaxf(mx_hi, v); else mx_lo = fmaxf(mx_lo, v);
            }
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
        mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
        mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
        const float mn_lo = fmaxf(m_lo, mx_lo), mn_hi = fmaxf(m_hi, mx_hi);
        const float use_lo = (mn_lo == -CUDART_INF_F) ? 0.f : mn_lo, use_hi = (mn_hi == -CUDART_INF_F) ? 0.f : mn_hi;
        const float corr_lo = exp2f(m_lo - use_lo), corr_hi = exp2f(m_hi - use_hi);
        m_lo = mn_lo; m_hi = mn_hi;
        l_lo *= corr_lo; l_hi *= corr_hi;
#pragma unroll
        for (int n = 0; n < HD / 8; ++n) { o[n][0] *= corr_lo; o[n][1] *= corr_lo; o[n][2] *= corr_hi; o[n][3] *= corr_hi; }
        uint32_t pa[2][4];
#pragma unroll
        for (int n = 0; n < 4; ++n) {
            const float p0 = exp2f(sc[n][0] - use_lo), p1 = exp2f(sc[n][1] - use_lo);
            const float p2 = exp2f(sc[n][2] - use_hi), p3 = exp2f(sc[n][3] - use_hi);
            l_lo += p0 + p1; l_hi += p2 + p3;
            pa[n >> 1][(n & 1) * 2 + 0] = pack_bf16(p0, p1);
            pa[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        // ---- O += P V
#pragma unroll
        for (int kk2 = 0; kk2 < 2; ++kk2) {
#pragma unroll
            for (int np = 0; np < HD / 16; ++np) {
                uint32_t b0, b1, b2, b3;
                const int key = kk2 * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                const int cu = np * 2 + (lane >> 4);
                ldsm_x4_trans(vb + (cu >> 3) * (kAttnBlockKeys * 128) + swz_unit(key, cu & 7), b0, b1, b2, b3);
                mma_bf16_16816(o[2 * np], pa[kk2][0], pa[kk2][1], pa[kk2][2], pa[kk2][3], b0, b1);
                mma_bf16_16816(o[2 * np + 1], pa[kk2][0], pa[kk2][1], pa[kk2][2], pa[kk2][3], b2, b3);
            }
        }
    }

    // ---- un-normalised partial result of this key range
    if (warp < MT) {
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
        l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
        l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? r_hi : r_lo;
            if (r >= R) continue;
            const int hq = hk * P.g + r / M, j = r % M;
            const size_t row = ((size_t)hq * (kMaxSplits + 1) + s) * kMaxRows + j;
            float* po = P.part_o + row * HD;
#pragma unroll
            for (int n = 0; n < HD / 8; ++n)
                __stcg(reinterpret_cast<float2*>(po + n * 8 + q2), make_float2(o[n][half * 2], o[n][half * 2 + 1]));
            if ((lane & 3) == 0)
                __stcg(reinterpret_cast<float2*>(P.part_ml + row * 2), make_float2(half ? m_hi : m_lo, half ? l_hi : l_lo));
        }
    }
}

__device__ void attention_phase(const FwdParams& P, int layer, uint8_t* att, int wtid) {
    const int S = attn_splits(P.L), S1 = S + 1;
    const int kps = S ? attn_keys_per_split(P.L, S) : 0;
    const int nunits = P.n_kv * S1;
    for (int unit = blockIdx.x; unit < nunits; unit += P.G) {
        const int hk = unit / S1, s = unit % S1;
        if (P.hd == 128) attention_unit<128>(P, layer, hk, s, S, kps, att, wtid);
        else attention_unit<64>(P, layer, hk, s, S, kps, att, wtid);
        named_bar_sync(1, kWorkerThreads);  // the unit's shared-memory tiles are free again
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
__global__ void __launch_bounds__(kThreads, 1) sdv_forward_kernel(const __grid_constant__ FwdParams P) {
    using SL = SmemLayout<NT>;
    static_assert(SL::NSTAGE >= 4 && SL::NSTAGE <= 16, "ring depth");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Misc* misc = reinterpret_cast<Misc*>(smem + SL::MISC_OFF);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < SL::NSTAGE; ++s) {
            mbar_init(&misc->full_w[s], 1);
            mbar_init(&misc->full_a[s], 1);
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
    uint32_t it = 0, norm_uses = 0;
    int nbar = 0;
    bool skip = false;
    for (int ph = P.ph_begin; ph < P.ph_end; ++ph) {
        int layer;
        const int kind = decode_phase(ph, P.n_layers, layer);
        // after an abandoned wait the remaining phases do no work but still meet at every barrier
        if (skip) {
        } else if (kind == PH_EMBED) {
            embed_phase(P, wtid);
            zero_qkv_acc(P, 0, wtid);
        } else if (kind == PH_ATTN) {
            attention_phase(P, layer, smem + SL::ATT_OFF, wtid);
        } else {
            if (kind == PH_O) zero_qkv_acc(P, (layer + 1) & 1, wtid);
            const Part pt = get_part(P.op[phase_op(kind)], blockIdx.x, P.G);
            if (pt.ntiles > 0) {
                if (warp < kConsumerWarps) consumer_phase<NT>(P, kind, layer, pt, smem, misc, it, norm_uses, warp, lane);
                else loader_phase<NT>(P, kind, layer, pt, smem, misc, it, warp - kConsumerWarps, lane);
            }
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
