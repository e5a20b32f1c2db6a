"""Seeded generators for model weights and context token arrays.

Weights are drawn in fp32, rounded to bf16 (round-to-nearest-even) and returned
as uint16 bit patterns: those bf16 values *are* the model for every consumer.
Vectors that stay in fp32 on every path (norm scales, biases) are also rounded
to bf16-representable values so either representation holds them exactly.

Every tensor is drawn in row blocks, each from its own Philox stream keyed by
(seed, tensor id, block index), so the result does not depend on the number of
worker threads.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

from .configs import ModelConfig

_ROWS_PER_BLOCK = 2048


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class LayerWeights:
    wq: np.ndarray   # uint16 [n_q*hd, d]
    wk: np.ndarray   # uint16 [n_kv*hd, d]
    wv: np.ndarray   # uint16 [n_kv*hd, d]
    wo: np.ndarray   # uint16 [d, n_q*hd]
    wg: np.ndarray   # uint16 [f, d]
    wu: np.ndarray   # uint16 [f, d]
    wd: np.ndarray   # uint16 [d, f]
    norm1: np.ndarray  # float32 [d]
    norm2: np.ndarray  # float32 [d]
    bq: Optional[np.ndarray] = None  # float32 [n_q*hd]
    bk: Optional[np.ndarray] = None
    bv: Optional[np.ndarray] = None


@dataclass
class ModelWeights:
    cfg: ModelConfig
    emb: np.ndarray                 # uint16 [V, d]
    final_norm: np.ndarray          # float32 [d]
    lm_head: Optional[np.ndarray]   # uint16 [V, d]; None when tied to emb
    layers: List[LayerWeights] = field(default_factory=list)


def _draw_block(seed: int, tensor_id: int, block: int, rows: int, cols: int, std: float) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ tensor_id, block]))
    x = rng.standard_normal((rows, cols), dtype=np.float32)
    x *= np.float32(std)
    return f32_to_bf16_bits(x)


def _draw_matrix(pool, seed, tensor_id, rows, cols, std) -> np.ndarray:
    """Submits the row blocks to the pool and returns the output array at once; the blocks are
    filled in by the workers (the caller waits on pool shutdown before reading)."""
    out = np.empty((rows, cols), dtype=np.uint16)

    def fill(b, r0, r1):
        out[r0:r1] = _draw_block(seed, tensor_id, b, r1 - r0, cols, std)

    for b, r0 in enumerate(range(0, rows, _ROWS_PER_BLOCK)):
        pool.submit(fill, b, r0, min(rows, r0 + _ROWS_PER_BLOCK))
    return out


def _draw_vector(seed, tensor_id, n, mean, std) -> np.ndarray:
    rng = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ tensor_id, 0xFFFF]))
    x = (mean + std * rng.standard_normal(n)).astype(np.float32)
    return bf16_bits_to_f32(f32_to_bf16_bits(x))


def make_weights(cfg: ModelConfig, seed: Optional[int] = None, threads: int = 8) -> ModelWeights:
    """Random-init decoder weights.

    Scales: embeddings and LM head N(0, 1/d) (logits of unit variance);
    Wq, Wk N(0, qk_var/d) (attention scores of variance qk_var); Wv, Wg, Wu
    N(0, 1/d); Wo, Wd N(0, resid_scale^2/(d*K_in)), so every sublayer adds about
    resid_scale/2 of an embedding row's norm to the residual stream; norm scales
    1 + 0.1 N(0,1); biases N(0, 0.02^2).  resid_scale and qk_var are set so that
    the bf16 rounding noise of a 28-layer forward pass stays well inside the
    parity tolerance on logits (larger values make the random network amplify
    that noise) while the layers still contribute about twice the embedding's
    norm to the final hidden state.
    """
    seed = cfg.seed if seed is None else seed
    d, f, hd = cfg.d_model, cfg.d_ffn, cfg.head_dim
    nq, nkv = cfg.n_q_heads * hd, cfg.n_kv_heads * hd
    s_e = 1.0 / math.sqrt(d)
    s_qk = math.sqrt(cfg.qk_var / d)
    s_o = cfg.resid_scale * s_e / math.sqrt(nq)
    s_d = cfg.resid_scale * s_e / math.sqrt(f)
    with ThreadPoolExecutor(max_workers=threads) as pool:
        emb = _draw_matrix(pool, seed, 1, cfg.vocab, d, s_e)
        lm = None if cfg.tied_lm_head else _draw_matrix(pool, seed, 2, cfg.vocab, d, s_e)
        mw = ModelWeights(cfg, emb, _draw_vector(seed, 3, d, 1.0, 0.1), lm)
        for l in range(cfg.n_layers):
            t = 16 * (l + 1)
            lw = LayerWeights(
                wq=_draw_matrix(pool, seed, t + 0, nq, d, s_qk),
                wk=_draw_matrix(pool, seed, t + 1, nkv, d, s_qk),
                wv=_draw_matrix(pool, seed, t + 2, nkv, d, s_e),
                wo=_draw_matrix(pool, seed, t + 3, d, nq, s_o),
                wg=_draw_matrix(pool, seed, t + 4, f, d, s_e),
                wu=_draw_matrix(pool, seed, t + 5, f, d, s_e),
                wd=_draw_matrix(pool, seed, t + 6, d, f, s_d),
                norm1=_draw_vector(seed, t + 7, d, 1.0, 0.1),
                norm2=_draw_vector(seed, t + 8, d, 1.0, 0.1),
            )
            if cfg.qkv_bias:
                lw.bq = _draw_vector(seed, t + 9, nq, 0.0, 0.02)
                lw.bk = _draw_vector(seed, t + 10, nkv, 0.0, 0.02)
                lw.bv = _draw_vector(seed, t + 11, nkv, 0.0, 0.02)
            mw.layers.append(lw)
    return mw


def make_context(cfg: ModelConfig, seed: Optional[int] = None) -> np.ndarray:
    """Context token ids: i.i.d. Zipf(s) over the vocabulary with planted repeats.

    Ranks 1..V get probability proportional to rank^-s (inverse-CDF sampling on
    the normalised cumulative table); a seeded permutation maps rank to token
    id.  The array is cut into `span`-token spans; the chosen spans (never the
    first) are overwritten, in ascending order, by a copy of a uniformly chosen
    earlier span.  A trailing partial span is never a copy source or target.
    """
    seed = cfg.seed if seed is None else seed
    rng = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ 0xC0, 7]))
    ranks = np.arange(1, cfg.vocab + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-cfg.zipf_s))
    cdf /= cdf[-1]
    u = rng.random(cfg.n_ctx)
    r = np.minimum(np.searchsorted(cdf, u, side="left"), cfg.vocab - 1)
    perm = rng.permutation(cfg.vocab)
    ctx = perm[r].astype(np.int32)
    n_spans = cfg.n_ctx // cfg.span
    if n_spans > 1:
        n_rep = cfg.repeat_spans if cfg.repeat_spans >= 0 else int(round(cfg.repeat_frac * n_spans))
        n_rep = min(n_rep, n_spans - 1)
        targets = np.sort(rng.choice(np.arange(1, n_spans), size=n_rep, replace=False))
        for t in targets:
            s = int(rng.integers(0, t))
            ctx[t * cfg.span:(t + 1) * cfg.span] = ctx[s * cfg.span:(s + 1) * cfg.span]
    return ctx
