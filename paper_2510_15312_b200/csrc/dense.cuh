// Dense prefill path: a chunk of the request (tens to hundreds of tokens) through the decoder as
// plain matrix products on the tensor cores.  The verify kernel puts the few token rows on the N
// side of the instruction and streams every weight once per launch; a prefill chunk has enough
// rows to fill the M side instead, so here the tokens are the 128 rows of a tcgen05.mma tile, the
// weights its 128 columns, operands arrive through tensor-map bulk copies (128-byte swizzle) in a
// multi-stage ring and the accumulator lives in tensor memory; a chunk streams each weight matrix
// once (row-major copies kept for this path).  Around the products: RMSNorm rows, rotary embedding +
// KV append, and a causal flash attention of the chunk's queries over cache + chunk (mma.sync tiles).
#pragma once
#include <cuda.h>
#include <math_constants.h>

#include "layout.cuh"
#include "ptx.cuh"

namespace sdv {

constexpr int kDenseBM = 128;      // token rows per tile (the instruction's M)
constexpr int kDenseBN = 128;      // output features per tile (the instruction's N)
constexpr int kDenseBK = 64;       // input features per stage: 64 bf16 = one 128-byte swizzled row
constexpr int kDenseStages = 6;
constexpr int kDenseTileBytes = kDenseBM * kDenseBK * 2;                 // one 128 x 64 operand tile: 16 KB
constexpr int kDenseStageBytes = 2 * kDenseTileBytes;                    // a token tile + a weight tile: 32 KB
constexpr int kDenseSmemBytes = kDenseStages * kDenseStageBytes + 1024 + 256;
constexpr int kDenseThreads = 192;  // warp 0: copies, warp 1: tensor-core issue, warps 2..5: epilogue
constexpr int kDenseMaxRows = 256;  // rows of the activation buffers (one sub-chunk)

enum DenseEpilogue { EPI_STORE = 0, EPI_RESIDUAL = 1, EPI_SWIGLU = 2 };

// Shared-memory operand descriptor, K-major, 128-byte swizzle: rows of 64 bf16 (128 bytes), groups of
// 8 rows 1024 bytes apart; a 16-element K step advances the start address by 32 bytes.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr) {
    uint64_t d = (uint64_t)((saddr >> 4) & 0x3fffu);
    d |= (uint64_t)1 << 16;                         // leading byte offset: unused for swizzled K-major operands
    d |= (uint64_t)(1024u >> 4) << 32;              // stride between 8-row groups
    d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                         // 128-byte swizzle
    return d;
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(smem_u32(smem_dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc));
}

// C[m][n] = sum_k A[m][k] * B[n][k] for one 128 x 128 tile; A = activations (bf16, row-major [rows][K]),
// B = weights (bf16, row-major [N][K]); fp32 accumulation in tensor memory.
//   EPI_STORE:    out_f32[m][n] = C (+ bias[n])
//   EPI_RESIDUAL: out_f32[m][n] += C             (each element belongs to one tile: no atomics)
//   EPI_SWIGLU:   the tile's columns 0..63 are gate features, 64..127 the matching up features:
//                 out_bf16[m][64 * tile + c] = silu(gate) * up
// gridDim.z > 1 splits K (EPI_STORE then needs a zeroed output; not for EPI_SWIGLU).
// Rows >= M and columns >= N are computed on whatever the copies deliver (zeros outside the tensors)
// and never written.  err: set to 1 when a bounded wait runs out.
template <int EPI>
__global__ void __launch_bounds__(kDenseThreads, 1)
dense_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, int M, int N, int K,
                  float* out_f32, int ld_f32, const float* bias, __nv_bfloat16* out_bf16, int ld_bf16, int* err,
                  unsigned long long wait_limit_ns) {
    extern __shared__ uint8_t dense_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(dense_smem_raw) + 1023) & ~(uintptr_t)1023);
    struct Ctl {
        uint64_t full[kDenseStages], empty[kDenseStages], acc_full;
        uint32_t tmem_base;
        int abort_flag;
    };
    Ctl* ctl = reinterpret_cast<Ctl*>(smem + kDenseStages * kDenseStageBytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n0 = blockIdx.x * kDenseBN, m0 = blockIdx.y * kDenseBM;
    // split K: block z of gridDim.z takes an even share of the K/64 stages; partial sums then meet by fp32
    // reductions in L2 (EPI_STORE: into a zeroed buffer, the bias added by share 0)
    const int nkb_all = K / kDenseBK, nz = (int)gridDim.z, z = (int)blockIdx.z;
    const int kb0 = even_start(nkb_all, nz, z), nkb = even_count(nkb_all, nz, z);
    const bool split = nz > 1;
    const int rot = nkb > 0 ? (int)((blockIdx.x * 5 + blockIdx.y * 11) % (unsigned)nkb) : 0;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kDenseStages; ++s) {
            mbar_init(&ctl->full[s], 1);
            mbar_init(&ctl->empty[s], 1);
        }
        mbar_init(&ctl->acc_full, 1);
        ctl->abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) tmem_alloc(&ctl->tmem_base, kDenseBN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = ctl->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t s = 0, par = 0;
            for (int kb = 0; kb < nkb; ++kb) {
                if (!mbar_wait_bounded(&ctl->empty[s], par ^ 1u, &ctl->abort_flag, wait_limit_ns)) break;
                uint8_t* a = smem + s * kDenseStageBytes;
                // blocks start their walk over K at different stages, so that at any moment they ask L2 for
                // different parts of the activations they all share
                const int kx = (kb0 + (kb + rot) % nkb) * kDenseBK;
                mbar_arrive_expect_tx(&ctl->full[s], kDenseStageBytes);
                tma_load_2d(a, &map_a, kx, m0, &ctl->full[s]);
                tma_load_2d(a + kDenseTileBytes, &map_b, kx, n0, &ctl->full[s]);
                if (++s == kDenseStages) { s = 0; par ^= 1u; }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_m128((uint32_t)kDenseBN);
            uint32_t s = 0, par = 0;
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                ok = mbar_wait_bounded(&ctl->full[s], par, &ctl->abort_flag, wait_limit_ns);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a = smem_u32(smem + s * kDenseStageBytes);
                const uint64_t da = umma_desc_sw128(a), db = umma_desc_sw128(a + kDenseTileBytes);
#pragma unroll
                for (int k4 = 0; k4 < kDenseBK / 16; ++k4)
                    umma_bf16(tmem, da + (uint64_t)(2 * k4), db + (uint64_t)(2 * k4), idesc, (uint32_t)(kb | k4));
                umma_commit(&ctl->empty[s]);   // the slot is free once these instructions have read it
                if (++s == kDenseStages) { s = 0; par ^= 1u; }
            }
            if (ok) umma_commit(&ctl->acc_full);
        }
    } else {
        // epilogue: warp w reads accumulator lanes 32 * (w % 4) .. + 31 (lane = token row of the tile), 32 columns
        // at a time, and turns them round through shared memory (the ring is free once the accumulator is
        // complete) so that one warp instruction touches 32 consecutive values of one output row: full 128-byte
        // lines for the stores, the residual read-modify-write and the partial-sum reductions alike
        const int q = warp & 3;
        const int row0 = m0 + q * 32;
        const bool got = mbar_wait_bounded(&ctl->acc_full, 0, &ctl->abort_flag, wait_limit_ns);
        const bool all_got = __all_sync(0xffffffffu, got);
        if (all_got) {
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16);
            float* stage = reinterpret_cast<float*>(smem + q * 8192);   // [32 rows][33]: this warp's turning area
            if (EPI == EPI_SWIGLU) {
                // columns 0..63 gate, 64..127 up: 16 + 16 at a time -> 16 bf16 outputs per row, staged as bf16
                // [32 rows][64 columns (+ 8 pad)] and written as four rows of 128 bytes per instruction
                __nv_bfloat16* st16 = reinterpret_cast<__nv_bfloat16*>(stage);
#pragma unroll 1
                for (int c = 0; c < kDenseBN / 2; c += 16) {
                    float g[16], u[16];
                    tmem_ld16(taddr + (uint32_t)c, g);
                    tmem_ld16(taddr + (uint32_t)(kDenseBN / 2 + c), u);
                    uint32_t pk[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float a0 = __fdividef(g[2 * i], 1.f + __expf(-g[2 * i])) * u[2 * i];
                        const float a1 = __fdividef(g[2 * i + 1], 1.f + __expf(-g[2 * i + 1])) * u[2 * i + 1];
                        pk[i] = pack_bf16(a0, a1);
                    }
                    uint4* d4 = reinterpret_cast<uint4*>(st16 + lane * 72 + c);
                    d4[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    d4[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
                __syncwarp();
#pragma unroll 1
                for (int r = lane >> 3; r < 32; r += 4) {
                    const uint4 v = *reinterpret_cast<const uint4*>(st16 + r * 72 + (lane & 7) * 8);
                    if (row0 + r < M)
                        *reinterpret_cast<uint4*>(out_bf16 + (size_t)(row0 + r) * ld_bf16 + n0 / 2 + (lane & 7) * 8) = v;
                }
            } else if (split) {
                // partial sums of a K share: turned round through shared memory so that one warp instruction adds
                // 32 consecutive values of one output row (full lines for the reductions in L2)
#pragma unroll 1
                for (int c = 0; c < kDenseBN; c += 32) {
                    float v[32];
                    {
                        float lo[16], hi[16];
                        tmem_ld16(taddr + (uint32_t)c, lo);
                        tmem_ld16(taddr + (uint32_t)(c + 16), hi);
#pragma unroll
                        for (int i = 0; i < 16; ++i) { v[i] = lo[i]; v[16 + i] = hi[i]; }
                    }
                    __syncwarp();
#pragma unroll
                    for (int i = 0; i < 32; ++i) stage[lane * 33 + i] = v[i];
                    __syncwarp();
                    const int col = n0 + c + lane;
                    if (col < N) {
                        const float b = (EPI == EPI_STORE && bias && z == 0) ? bias[col] : 0.f;
                        float* dst = out_f32 + (size_t)row0 * ld_f32 + col;
                        const int nr = min(32, M - row0);
                        for (int r = 0; r < nr; ++r) red_add_f32(dst + (size_t)r * ld_f32, stage[r * 33 + lane] + b);
                    }
                }
            } else {
                // one block per output element: plain stores, or read-add-write of the residual, 16 bytes at a time
                const int row = row0 + lane;
                float* dst = out_f32 + (size_t)row * ld_f32 + n0;
#pragma unroll 1
                for (int c = 0; c < kDenseBN; c += 16) {
                    float v[16];
                    tmem_ld16(taddr + (uint32_t)c, v);
                    if (row < M && n0 + c < N) {   // N is a multiple of 16
#pragma unroll
                        for (int i = 0; i < 16; i += 4) {
                            float4 o = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                            if (EPI == EPI_STORE && bias) {
                                o.x += bias[n0 + c + i]; o.y += bias[n0 + c + i + 1]; o.z += bias[n0 + c + i + 2]; o.w += bias[n0 + c + i + 3];
                            }
                            if (EPI == EPI_RESIDUAL) {
                                const float4 old = *reinterpret_cast<const float4*>(dst + c + i);
                                o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                            }
                            *reinterpret_cast<float4*>(dst + c + i) = o;
                        }
                    }
                }
            }
            tc_fence_before();
        }
    }
    __syncthreads();
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem, kDenseBN);
    if (threadIdx.x == 0 && ctl->abort_flag) atomicExch(err, 1);
}

// Residual rows of a sub-chunk from the embedding table: h[r][:] = E[token r].
__global__ void dense_embed_kernel(const int* tokens, const __nv_bfloat16* emb, float* h, int d, int V) {
    const int r = blockIdx.x;
    int tok = tokens[r];
    tok = min(max(tok, 0), V - 1);
    for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
        const uint4 raw = *reinterpret_cast<const uint4*>(emb + (size_t)tok * d + c);
        const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&raw);
        float* dst = h + (size_t)r * d + c;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __bfloat1622float2(pb[i]);
            dst[2 * i] = f.x;
            dst[2 * i + 1] = f.y;
        }
    }
}

// xn[r][:] = bf16(h[r][:] * rsqrt(mean(h[r]^2) + eps) * w): one block per row.
__global__ void dense_rmsnorm_kernel(const float* h, const float* w, __nv_bfloat16* xn, int d, float eps) {
    __shared__ float red[32];
    const float* x = h + (size_t)blockIdx.x * d;
    float ss = 0.f;
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
        const float4 v = *reinterpret_cast<const float4*>(x + c);
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    for (int off = 16; off; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    if (threadIdx.x < 32) {
        ss = threadIdx.x < (blockDim.x >> 5) ? red[threadIdx.x] : 0.f;
        for (int off = 16; off; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        if (threadIdx.x == 0) red[0] = rsqrtf(ss / (float)d + eps);
    }
    __syncthreads();
    const float rs = red[0];
    for (int c = threadIdx.x * 4; c < d; c += blockDim.x * 4) {
        const float4 v = *reinterpret_cast<const float4*>(x + c);
        const float4 g = *reinterpret_cast<const float4*>(w + c);
        *reinterpret_cast<uint2*>(xn + (size_t)blockIdx.x * d + c) =
            make_uint2(pack_bf16(v.x * rs * g.x, v.y * rs * g.y), pack_bf16(v.z * rs * g.z, v.w * rs * g.w));
    }
}

// Rotary embedding of q and k at positions L + r (pairing (i, i + hd/2)); q to the bf16 query matrix,
// k and v appended to the cache at rows L + r.  grid = (rows, q heads + kv heads), hd / 2 threads.
__global__ void dense_rope_append_kernel(const float* qkv, int n_qkv, const float2* rope, __nv_bfloat16* qout, int n_q, int n_kv,
                                         int hd, __nv_bfloat16* kcache, __nv_bfloat16* vcache, size_t layer_off, int max_seq, int L) {
    const int r = blockIdx.x, head = blockIdx.y, i = threadIdx.x, h2 = hd / 2;
    const float2 cs = rope[(size_t)(L + r) * h2 + i];
    const float* row = qkv + (size_t)r * n_qkv;
    if (head < n_q) {
        const float a = row[head * hd + i], b = row[head * hd + i + h2];
        __nv_bfloat16* dst = qout + (size_t)r * (n_q * hd) + head * hd;
        dst[i] = __float2bfloat16(a * cs.x - b * cs.y);
        dst[i + h2] = __float2bfloat16(b * cs.x + a * cs.y);
    } else {
        const int kh = head - n_q;
        const float* kr = row + n_q * hd + kh * hd;
        const float* vr = row + (n_q + n_kv) * hd + kh * hd;
        const float a = kr[i], b = kr[i + h2];
        const size_t off = layer_off + ((size_t)kh * max_seq + L + r) * hd;
        kcache[off + i] = __float2bfloat16(a * cs.x - b * cs.y);
        kcache[off + i + h2] = __float2bfloat16(b * cs.x + a * cs.y);
        vcache[off + i] = __float2bfloat16(vr[i]);
        vcache[off + i + h2] = __float2bfloat16(vr[i + h2]);
    }
}

// Causal attention of a sub-chunk's queries (rows r = 0..M-1 at positions L + r) over cache rows
// 0 .. L + r of their KV head.  One block per (query head, 16-query tile): many small blocks, since
// a sub-chunk has few rows and the keys are the long dimension.  Keys come in blocks of 64 through
// two shared-memory buffers; warp w takes the w-th group of 16 keys of every block: scores, online
// softmax (log2 domain) and P V in its registers (mma.sync m16n8k16), and the four key groups meet in
// shared memory at the end.  Output bf16 [M][n_q * hd].
template <int HD>
__global__ void __launch_bounds__(128) dense_attention_kernel(const __nv_bfloat16* q, const __nv_bfloat16* kcache,
                                                              const __nv_bfloat16* vcache, size_t layer_off, int max_seq, int n_q,
                                                              int g, int M, int L, float scale_log2e, __nv_bfloat16* out) {
    constexpr int KSTEPS = HD / 16, UNITS = HD / 8, NT_O = HD / 8, KB = 64, QR = 16;
    constexpr int QBYTES = QR * HD * 2, KVBYTES = KB * HD * 2;
    static_assert(3 * (NT_O + 1) * 32 * 16 <= 4 * KVBYTES, "exchange area of the key-group merge");
    extern __shared__ uint8_t att_smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(att_smem_raw) + 127) & ~(uintptr_t)127);
    uint8_t* Qs = base;
    uint8_t* KVs = base + QBYTES;   // [2 buffers][K | V]
    const int head = blockIdx.x, r0 = blockIdx.y * QR, kvh = head / g;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, tid = threadIdx.x;
    const size_t cache0 = layer_off + (size_t)kvh * max_seq * HD;
    const int rows = min(QR, M - r0);
    const int nkeys = L + r0 + rows;              // keys any row of this tile may see
    const int nblk = (nkeys + KB - 1) / KB;
    auto load_block = [&](int blk) {
        if (blk < nblk) {
            uint8_t* Ks = KVs + (blk & 1) * 2 * KVBYTES;
            uint8_t* Vs = Ks + KVBYTES;
            for (int u = tid; u < KB * UNITS; u += 128) {
                const int key = u / UNITS, q16 = u % UNITS, kk = blk * KB + key;
                const bool valid = kk < nkeys;
                const size_t off = cache0 + (size_t)(valid ? kk : 0) * HD + q16 * 8;
                const uint32_t so = (q16 >> 3) * (KB * 128) + swz_unit(key, q16 & 7);
                cp_async_16_zfill(Ks + so, kcache + off, valid);
                cp_async_16_zfill(Vs + so, vcache + off, valid);
            }
        }
        cp_async_commit();
    };
    load_block(0);
    load_block(1);
    for (int u = tid; u < QR * UNITS; u += 128) {
        const int r = u / UNITS, q16 = u % UNITS;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < rows) v = *reinterpret_cast<const uint4*>(q + (size_t)(r0 + r) * (n_q * HD) + head * HD + q16 * 8);
        *reinterpret_cast<uint4*>(Qs + (q16 >> 3) * (QR * 128) + swz_unit(r, q16 & 7)) = v;
    }
    const int gq = lane >> 2, q2 = (lane & 3) * 2;
    const int r_lo = gq, r_hi = gq + 8;
    float o[NT_O][4];
#pragma unroll
    for (int n = 0; n < NT_O; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
    float m_lo = -CUDART_INF_F, m_hi = -CUDART_INF_F, l_lo = 0.f, l_hi = 0.f;
    const uint32_t qb = smem_u32(Qs);
    const int lim_lo = L + r0 + r_lo, lim_hi = L + r0 + r_hi;   // last key each row sees
    for (int blk = 0; blk < nblk; ++blk) {
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t kb = smem_u32(KVs + (blk & 1) * 2 * KVBYTES), vb = kb + KVBYTES;
        const int c = warp, key0 = blk * KB + c * 16;
        if (key0 <= L + r0 + QR - 1) {   // some key of this group is visible to some row of the tile
            float sc[2][4];
#pragma unroll
            for (int n = 0; n < 2; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < KSTEPS; ++ks) {
                uint32_t a0, a1, a2, a3, b0, b1, b2, b3;
                ldsm_x4(qb + (ks >> 2) * (QR * 128) + swz_unit(lane & 15, (ks & 3) * 2 + (lane >> 4)), a0, a1, a2, a3);
                const int krow = c * 16 + (lane & 7) + ((lane >> 4) << 3);
                ldsm_x4(kb + (ks >> 2) * (KB * 128) + swz_unit(krow, (ks & 3) * 2 + ((lane >> 3) & 1)), b0, b1, b2, b3);
                mma_bf16_16816(sc[0], a0, a1, a2, a3, b0, b1);
                mma_bf16_16816(sc[1], a0, a1, a2, a3, b2, b3);
            }
            float mx_lo = -CUDART_INF_F, mx_hi = -CUDART_INF_F;
#pragma unroll
            for (int n = 0; n < 2; ++n)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int key = key0 + n * 8 + q2 + (e & 1);
                    const bool hi = e >= 2;
                    const bool ok = key <= (hi ? lim_hi : lim_lo);
                    const float v = ok ? sc[n][e] * scale_log2e : -CUDART_INF_F;
                    sc[n][e] = v;
                    if (hi) mx_hi = fmaxf(mx_hi, v); else mx_lo = fmaxf(mx_lo, v);
                }
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 1));
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(0xffffffffu, mx_lo, 2));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 1));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(0xffffffffu, mx_hi, 2));
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
        __syncthreads();
        load_block(blk + 2);
    }
    cp_async_wait<0>();
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xffffffffu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xffffffffu, l_hi, 2);
    // the key groups of warps 1..3 meet warp 0's in shared memory (the K/V buffers are free now)
    {
        float4* ex_o = reinterpret_cast<float4*>(KVs);   // [warp - 1][output tile][lane]
        float4* ex_ml = ex_o + 3 * NT_O * 32;            // [warp - 1][lane]
        __syncthreads();
        if (warp > 0) {
            float4* dst = ex_o + (warp - 1) * NT_O * 32;
#pragma unroll
            for (int n = 0; n < NT_O; ++n) dst[n * 32 + lane] = make_float4(o[n][0], o[n][1], o[n][2], o[n][3]);
            ex_ml[(warp - 1) * 32 + lane] = make_float4(m_lo, m_hi, l_lo, l_hi);
        }
        __syncthreads();
        if (warp > 0) return;
#pragma unroll 1
        for (int og = 0; og < 3; ++og) {
            const float4 ml = ex_ml[og * 32 + lane];
            const float mn_lo = fmaxf(m_lo, ml.x), mn_hi = fmaxf(m_hi, ml.y);
            const float use_lo = (mn_lo == -CUDART_INF_F) ? 0.f : mn_lo, use_hi = (mn_hi == -CUDART_INF_F) ? 0.f : mn_hi;
            const float e0_lo = exp2f(m_lo - use_lo), e1_lo = exp2f(ml.x - use_lo);
            const float e0_hi = exp2f(m_hi - use_hi), e1_hi = exp2f(ml.y - use_hi);
            m_lo = mn_lo;
            m_hi = mn_hi;
            l_lo = l_lo * e0_lo + ml.z * e1_lo;
            l_hi = l_hi * e0_hi + ml.w * e1_hi;
            const float4* src = ex_o + og * NT_O * 32;
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
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int r = half ? r_hi : r_lo;
        if (r >= rows) continue;
        const float inv = 1.f / (half ? l_hi : l_lo);
        __nv_bfloat16* po = out + (size_t)(r0 + r) * (n_q * HD) + head * HD + q2;
#pragma unroll
        for (int n = 0; n < NT_O; ++n)
            *reinterpret_cast<uint32_t*>(po + n * 8) = pack_bf16(o[n][half * 2] * inv, o[n][half * 2 + 1] * inv);
    }
}

// Weight copy for the dense path.  mode 0: rows copied as they are (dst row = src row).  mode 1:
// gate | up interleaved in blocks of 64: dst rows [128 t, 128 t + 64) = gate rows 64 t.., the next 64
// rows the matching up rows, so that one 128-column tile holds both halves of 64 SwiGLU columns.
__global__ void dense_copy_weights_kernel(uint16_t* dst, const uint16_t* src0, const uint16_t* src1, int rows, int K, int mode) {
    const int K8 = K / 8;
    const long long total = (long long)rows * K8;
    for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < total; u += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(u / K8), k8 = (int)(u % K8);
        const uint16_t* s;
        if (mode == 0) {
            s = src0 + (size_t)r * K;
        } else {
            const int t = r / 128, w = r % 128;
            s = (w < 64) ? src0 + (size_t)(64 * t + w) * K : src1 + (size_t)(64 * t + w - 64) * K;
        }
        *reinterpret_cast<uint4*>(dst + (size_t)r * K + k8 * 8) = *reinterpret_cast<const uint4*>(s + k8 * 8);
    }
}

}  // namespace sdv
