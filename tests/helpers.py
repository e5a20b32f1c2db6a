"""Shared pieces of the GPU parity tests: running the oracle, and the step-by-step comparison."""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from oracle import sdv_oracle as O

LOGIT_TOL = 0.05      # max |logit difference| allowed against the oracle
COS_TOL = 0.999       # minimum cosine similarity per logits row
MARGIN_TOL = 0.05     # below this top-2 margin of the oracle a different greedy token is legitimate


@dataclass
class RefStep:
    kv_len_before: int
    pending: int
    draft: List[int]
    from_drafter: bool          # the drafts are what the n-gram drafter must produce in this state
    y: List[int]
    accept: int
    emitted: List[int]
    margin: List[float]
    runner_up: List[int]        # oracle's second-best token per row
    near_best: Optional[List[List[int]]] = None   # per row: tokens whose oracle logit lies within MARGIN_TOL of the oracle's best
    logits: Optional[np.ndarray] = None         # [dl+1, V] full rows (live oracle) ...
    sample_ids: Optional[np.ndarray] = None     # ... or values at sampled ids (stored trajectories)
    logit_sample: Optional[np.ndarray] = None
    top_ids: Optional[np.ndarray] = None
    top_vals: Optional[np.ndarray] = None


def steps_from_oracle(steps, from_drafter: bool) -> List[RefStep]:
    out = []
    for s in steps:
        ru = [O.top2(s.logits[r])[1] for r in range(len(s.draft) + 1)]
        out.append(RefStep(s.kv_len_before, s.pending, list(s.draft), from_drafter, list(s.y), s.accept,
                           list(s.emitted), list(s.margin), ru, logits=s.logits,
                           near_best=[np.nonzero(s.logits[r] >= s.logits[r].max() - MARGIN_TOL)[0].tolist()
                                      for r in range(len(s.draft) + 1)]))
    return out


def steps_from_golden(g) -> List[RefStep]:
    out = []
    for i in range(len(g["accept"])):
        dl = int(g["draft_len"][i])
        out.append(RefStep(int(g["kv_len_before"][i]), int(g["pending"][i]), g["draft"][i, :dl].tolist(), i % 2 == 0,
                           g["y"][i, :dl + 1].tolist(), int(g["accept"][i]),
                           g["emitted"][i, :int(g["n_emitted"][i])].tolist(), g["margin"][i, :dl + 1].tolist(),
                           g["top_ids"][i, :dl + 1, 1].tolist(), sample_ids=g["sample_ids"],
                           logit_sample=g["logit_sample"][i, :dl + 1], top_ids=g["top_ids"][i, :dl + 1],
                           top_vals=g["top_vals"][i, :dl + 1],
                           near_best=[[int(t) for t, v in zip(g["top_ids"][i, r], g["top_vals"][i, r])
                                       if v >= g["top_vals"][i, r].max() - MARGIN_TOL] for r in range(dl + 1)]))
    return out


def compare_step(sdv, step: RefStep, k: int, stats: dict, predrafted: bool = False, before_commit=None):
    """Runs draft + verify for one reference step on a context already in the step's state and
    checks everything the step fixes.  Commits the ORACLE's outcome so the states stay aligned.
    predrafted: the device already holds the step's draft (verify runs on it as it is);
    before_commit(y, a): called with the device's predictions and accept length before the commit."""
    dl = len(step.draft)
    assert sdv.kv_len() == step.kv_len_before
    if predrafted:
        y, a = sdv.verify(None)
        rows = dl + 1
    elif step.from_drafter:
        got_draft = sdv.draft(k)
        assert got_draft == step.draft, f"draft differs at L={step.kv_len_before}: {got_draft} vs {step.draft}"
        y, a = sdv.verify(None)
        rows = k + 1
    else:
        y, a = sdv.verify(step.draft)
        rows = dl + 1
    check_verified(sdv, step, y, a, stats, before_commit)
    return rows


def check_verified(sdv, step: RefStep, y, a, stats: dict, before_commit=None):
    """The part of compare_step after the verify call: logits rows, greedy tokens and accept length of the
    context's outstanding verify result against the reference step, then the oracle's outcome is committed."""
    dl = len(step.draft)
    logits = sdv.get_logits(dl + 1)
    assert np.all(np.isfinite(logits))
    for r in range(dl + 1):
        if step.logits is not None:
            ref = step.logits[r]
            got = logits[r]
        else:
            ids = np.concatenate([step.sample_ids, step.top_ids[r]])
            ref = np.concatenate([step.logit_sample[r], step.top_vals[r]])
            got = logits[r][ids]
        err = float(np.abs(got - ref).max())
        cos = float(np.dot(got, ref) / (np.linalg.norm(got) * np.linalg.norm(ref)))
        stats["max_err"] = max(stats.get("max_err", 0.0), err)
        stats["min_cos"] = min(stats.get("min_cos", 1.0), cos)
        assert err <= LOGIT_TOL, f"row {r} at L={step.kv_len_before}: |dlogit| {err}"
        assert cos >= COS_TOL, f"row {r} at L={step.kv_len_before}: cosine {cos}"
    # greedy tokens: identical unless the oracle itself was within MARGIN_TOL of another token
    first_bad = None
    for r in range(dl + 1):
        if int(y[r]) != step.y[r]:
            assert step.margin[r] < MARGIN_TOL, f"row {r}: token {y[r]} vs {step.y[r]}, margin {step.margin[r]}"
            assert int(y[r]) in step.near_best[r], f"row {r}: the oracle's logit of token {y[r]} is not within the margin of its best"
            stats["near_tie_flips"] = stats.get("near_tie_flips", 0) + 1
            if first_bad is None:
                first_bad = r
    if first_bad is None or first_bad > step.accept:
        assert a == step.accept, f"accept length {a} vs {step.accept} at L={step.kv_len_before}"
    stats["steps"] = stats.get("steps", 0) + 1
    stats.setdefault("accepts", []).append(step.accept)
    if before_commit is not None:
        before_commit([int(t) for t in y[:dl + 1]], int(a))
    # teacher forcing: commit what the oracle committed
    sdv.debug_force_commit(len(step.emitted) - 1, step.emitted[-1])
    assert sdv.kv_len() == step.kv_len_before + len(step.emitted)


def compare_prefix_rows(sdv, step: RefStep, kp: int, stats: dict):
    """Verifies only the first kp drafts of a forced-draft step and compares rows 0..kp with the stored
    rows.  Under the linear-chain mask row j sees the cache and new rows 0..j only, so those rows do
    not depend on the drafts behind them: the stored step fixes them for every shorter draft, and
    the accept length is min(a, kp).  This reaches the launch shapes of shorter drafts (other
    instruction widths and attention splits) at full size without another oracle run.  Nothing is
    committed: the next verify overwrites the same KV rows."""
    assert 0 < kp < len(step.draft)
    y, a = sdv.verify(step.draft[:kp])
    logits = sdv.get_logits(kp + 1)
    flipped = None
    for r in range(kp + 1):
        if step.logits is not None:
            ref, got = step.logits[r], logits[r]
        else:
            ids = np.concatenate([step.sample_ids, step.top_ids[r]])
            ref = np.concatenate([step.logit_sample[r], step.top_vals[r]])
            got = logits[r][ids]
        err = float(np.abs(got - ref).max())
        cos = float(np.dot(got, ref) / (np.linalg.norm(got) * np.linalg.norm(ref)))
        stats["max_err"] = max(stats.get("max_err", 0.0), err)
        stats["min_cos"] = min(stats.get("min_cos", 1.0), cos)
        assert err <= LOGIT_TOL, f"{kp} drafts, row {r} at L={step.kv_len_before}: |dlogit| {err}"
        assert cos >= COS_TOL, f"{kp} drafts, row {r} at L={step.kv_len_before}: cosine {cos}"
        if int(y[r]) != step.y[r]:
            assert step.margin[r] < MARGIN_TOL and int(y[r]) in step.near_best[r], f"{kp} drafts, row {r}: token {y[r]}"
            if flipped is None:
                flipped = r
    want = min(step.accept, kp)
    if flipped is None or flipped > want:
        assert a == want, f"{kp} drafts: accept length {a} vs {want} at L={step.kv_len_before}"
    stats["prefix_checks"] = stats.get("prefix_checks", 0) + 1
