"""Writes tests/golden/<config>.npz: the oracle's trajectory for one of the large workloads.

Calls only the CPU oracle and the seeded input generators.  Usage:
    python tests/golden/make_golden.py qwen1.5b [--gen N]

Stored per verify step: the state before the step (KV length, pending token), the drafts fed
to it, the oracle's greedy tokens y, accept length, emitted tokens, the top-2 logit margin of
every row, and the logits of every row at a fixed seeded sample of vocabulary ids plus the
row's own 8 best ids.  Drafts alternate between the n-gram drafter's own output and the true
greedy continuation corrupted at a cycling position, so every accept length occurs.
Also stored: K/V rows of the first and last layer at a few sampled positions after prefill.
"""
from __future__ import annotations

import argparse
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import sdv_oracle as O  # noqa: E402
from sdv_inputs import get_config, make_context, make_weights  # noqa: E402

N_SAMPLE = 512
N_TOP = 8


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("config")
    ap.add_argument("--gen", type=int, default=0, help="generated tokens to record (default: the config's)")
    ap.add_argument("--k", type=int, default=0)
    args = ap.parse_args()
    cfg = get_config(args.config)
    gen = args.gen or cfg.gen
    k = args.k or cfg.k
    t0 = time.time()
    w = make_weights(cfg)
    ctx = make_context(cfg)
    print(f"weights {time.time() - t0:.1f}s", flush=True)

    # plain greedy decoding first: the true continuation
    m = O.OracleModel(w)
    greedy = O.greedy_decode(m, ctx, gen, cfg.chunk)
    kv_pos = np.unique(np.linspace(0, cfg.n_ctx - 1, 9).astype(int))
    kv_samples = {}
    for layer in (0, cfg.n_layers - 1):
        kv_samples[f"k{layer}"] = m.kv_view("k")[layer][:, kv_pos].copy()
        kv_samples[f"v{layer}"] = m.kv_view("v")[layer][:, kv_pos].copy()
    print(f"greedy {time.time() - t0:.1f}s", flush=True)

    step_no = [0]

    def drafter(hist, kk):
        s = step_no[0]
        step_no[0] += 1
        if s % 2 == 0:
            return O.ngram_draft(ctx, hist, cfg.ngram_n, cfg.ngram_min, kk)[0].tolist()
        i0 = len(hist) - cfg.n_ctx
        d = [greedy[i0 + i] if i0 + i < gen else 0 for i in range(kk)]
        e = (s // 2) % (kk + 1) + 1          # corrupt position e in 1..kk; e = kk+1 leaves the draft intact
        if e <= kk:
            d[e - 1] = (d[e - 1] + 1) % cfg.vocab
        return d

    m2 = O.OracleModel(w)
    toks, steps = O.spec_decode(m2, ctx, gen, cfg.chunk, k, cfg.ngram_n, cfg.ngram_min, drafter=drafter,
                                keep_logits=True)
    assert toks == greedy, "speculative decoding must reproduce greedy decoding"
    print(f"spec {time.time() - t0:.1f}s, {len(steps)} steps", flush=True)

    rng = np.random.Generator(np.random.Philox(key=[cfg.seed, 0x601D]))
    sample_ids = np.sort(rng.choice(cfg.vocab, size=N_SAMPLE, replace=False)).astype(np.int32)
    S, R = len(steps), k + 1
    out = dict(
        config=np.array(cfg.name), gen=np.array(gen), k=np.array(k), tokens=np.array(toks, dtype=np.int32),
        first_token=np.array(greedy[0], dtype=np.int32), sample_ids=sample_ids, kv_pos=kv_pos.astype(np.int32),
        kv_len_before=np.zeros(S, np.int32), pending=np.zeros(S, np.int32), draft_len=np.zeros(S, np.int32),
        draft=np.zeros((S, k), np.int32), y=np.zeros((S, R), np.int32), accept=np.zeros(S, np.int32),
        n_emitted=np.zeros(S, np.int32), emitted=np.zeros((S, R), np.int32), margin=np.zeros((S, R), np.float32),
        logit_sample=np.zeros((S, R, N_SAMPLE), np.float32), top_ids=np.zeros((S, R, N_TOP), np.int32),
        top_vals=np.zeros((S, R, N_TOP), np.float32), logit_norm=np.zeros((S, R), np.float32),
    )
    for i, s in enumerate(steps):
        dl = len(s.draft)
        out["kv_len_before"][i] = s.kv_len_before
        out["pending"][i] = s.pending
        out["draft_len"][i] = dl
        out["draft"][i, :dl] = s.draft
        out["y"][i, :dl + 1] = s.y
        out["accept"][i] = s.accept
        out["n_emitted"][i] = len(s.emitted)
        out["emitted"][i, :len(s.emitted)] = s.emitted
        out["margin"][i, :dl + 1] = s.margin
        for r in range(dl + 1):
            row = s.logits[r]
            out["logit_sample"][i, r] = row[sample_ids]
            top = np.argsort(-row, kind="stable")[:N_TOP]
            out["top_ids"][i, r] = top
            out["top_vals"][i, r] = row[top]
            out["logit_norm"][i, r] = np.linalg.norm(row)
    out.update(kv_samples)
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), f"{cfg.name}.npz")
    np.savez_compressed(path, **out)
    print(f"wrote {path} ({os.path.getsize(path) / 1e6:.2f} MB) in {time.time() - t0:.1f}s")


if __name__ == "__main__":
    main()
