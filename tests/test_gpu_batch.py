"""Batched verify through the C-ABI: several sequences share one pass over the weights, and every sequence
must come out as the oracle computes it on its own (the oracle has no batch: a batched step is defined as
the independent steps of its sequences).  Tolerances as in test_gpu_parity.py."""
import os

import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import get_config, make_context, make_weights
from paper_2510_15312_b200 import binding as B
from paper_2510_15312_b200.binding import Sdv, SdvError, config_from
from helpers import check_verified, steps_from_golden, steps_from_oracle

pytestmark = pytest.mark.gpu
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def gpu_prefill(s, ctx, chunk):
    n = len(ctx)
    for i in range(0, n, chunk):
        s.prefill_chunk(ctx[i:i + chunk], is_last=(i + chunk >= n))


def corrupted_continuation(greedy, n_ctx, gen, k, vocab):
    """Forced drafts: the true continuation, wrong at a position that cycles through 1..k+1."""
    step = [0]

    def drafter(hist, kk):
        i0 = len(hist) - n_ctx
        d = [greedy[i0 + i] if i0 + i < gen else 0 for i in range(k)]
        e = step[0] % (k + 1) + 1
        step[0] += 1
        if e <= k:
            d[e - 1] = (d[e - 1] + 1) % vocab
        return d
    return drafter


@pytest.mark.parametrize("name", ["tiny", "mini_gqa", "mini_hd128"])
def test_batched_steps_match_each_sequences_own_oracle(name):
    """Three sequences of different lengths and kinds of draft (the drafter's own; forced drafts of k and of
    k - 1 tokens) advance together; a sequence that finishes leaves the batch, so batches of 3, 2 and 1 run."""
    cfg = get_config(name)
    w = make_weights(cfg)
    k = min(cfg.k, 9)   # three sequences' rows fit one launch (at most 32), and pass 16 rows where k allows
    lens = [cfg.n_ctx, cfg.n_ctx - 37, cfg.n_ctx // 2 + 5]
    gens = [cfg.gen, cfg.gen - 3, cfg.gen + 4]
    ks = [k, k, k - 1]
    ctxs = [make_context(cfg.with_(n_ctx=n), seed=cfg.seed + 11 * i)[:n] for i, n in enumerate(lens)]
    refs = []
    for i in range(3):
        model = O.OracleModel(w)
        if i == 0:
            toks, steps = O.spec_decode(model, ctxs[i], gens[i], cfg.chunk, ks[i], cfg.ngram_n, cfg.ngram_min, keep_logits=True)
        else:
            greedy = O.greedy_decode(O.OracleModel(w), ctxs[i], gens[i], cfg.chunk)
            toks, steps = O.spec_decode(model, ctxs[i], gens[i], cfg.chunk, ks[i], cfg.ngram_n, cfg.ngram_min,
                                        drafter=corrupted_continuation(greedy, lens[i], gens[i], ks[i], cfg.vocab),
                                        keep_logits=True)
            assert toks == greedy
        refs.append((toks, steps_from_oracle(steps, from_drafter=(i == 0))))
    lead = Sdv(config_from(cfg, max_seq=cfg.n_ctx + cfg.gen + 64))
    lead.load_weights(w)
    seqs = [lead, lead.follower(), lead.follower()]
    assert seqs[1].workspace_bytes < lead.workspace_bytes
    for i, s in enumerate(seqs):
        s.set_parity_mode(True)
        gpu_prefill(s, ctxs[i], cfg.chunk)
        s.debug_set_history(list(ctxs[i]) + [refs[i][0][0]], lens[i])
    at = [0, 0, 0]
    stats = [{}, {}, {}]
    sizes = set()
    while True:
        live = [i for i in range(3) if at[i] < len(refs[i][1])]
        if not live:
            break
        sizes.add(len(live))
        for i in live:
            st = refs[i][1][at[i]]
            assert seqs[i].kv_len() == st.kv_len_before
            if st.from_drafter:
                assert seqs[i].draft(ks[i]) == st.draft
            else:
                seqs[i].debug_set_draft(st.draft)
        acc = Sdv.verify_batch([seqs[i] for i in live])
        for n, i in enumerate(live):
            y, a = seqs[i].get_verified()
            assert a == acc[n]
            check_verified(seqs[i], refs[i][1][at[i]], y, a, stats[i])
            at[i] += 1
    assert sizes == {1, 2, 3}
    for i in range(3):
        assert seqs[i].kv_len() == lens[i] + gens[i] - 1
        if i > 0:   # the forced drafts go wrong at a cycling position
            assert len(set(stats[i]["accepts"])) >= 2
    print(name, [(round(st["max_err"], 4), round(st["min_cos"], 6)) for st in stats])
    for s in reversed(seqs):
        s.close()


def test_a_batch_of_one_and_rows_without_a_draft():
    """A single-sequence batch is sdv_verify; a sequence that has not drafted contributes its pending token only."""
    cfg = get_config("tiny")
    w = make_weights(cfg)
    ctx = make_context(cfg)
    model = O.OracleModel(w)
    last = model.prefill(ctx, cfg.chunk)
    T = O.argmax(last)
    lg = model.forward([T], len(ctx))
    lead = Sdv(config_from(cfg))
    lead.load_weights(w)
    fol = lead.follower()
    for s in (lead, fol):
        s.set_parity_mode(True)
        gpu_prefill(s, ctx, cfg.chunk)
        s.debug_set_history(list(ctx) + [T], cfg.n_ctx)
    y1, a1 = lead.verify([])
    one = lead.get_logits(1).copy()
    assert Sdv.verify_batch([lead]) == [0]
    y2, a2 = lead.get_verified()
    assert int(y1[0]) == int(y2[0]) and a1 == a2 == 0
    assert np.abs(lead.get_logits(1) - one).max() <= 1e-2   # the same rows twice: fp32 reduction order differs from run to run
    assert np.abs(one[0] - lg[0]).max() <= 0.05
    # both sequences, neither has drafted: two rows, each its own pending token at its own position
    assert Sdv.verify_batch([fol, lead]) == [0, 0]
    for s in (lead, fol):
        assert np.abs(s.get_logits(1)[0] - lg[0]).max() <= 0.05
        assert int(s.get_verified()[0][0]) == O.argmax(lg[0])
    e, _ = fol.commit()
    assert list(e) == [O.argmax(lg[0])] and fol.kv_len() == cfg.n_ctx + 1
    assert lead.kv_len() == cfg.n_ctx   # nothing was committed on the other sequence
    fol.close()
    lead.close()


def test_batch_argument_checks():
    cfg = get_config("tiny")
    w = make_weights(cfg)
    ctx = make_context(cfg)
    lead = Sdv(config_from(cfg))
    with pytest.raises(SdvError) as e:   # no weights yet: nothing to follow
        lead.follower()
    assert e.value.code == B.ESTATE
    lead.load_weights(w)
    other = Sdv(config_from(cfg))
    other.load_weights(w)
    fols = [lead.follower() for _ in range(4)]
    with pytest.raises(SdvError) as e:   # a follower owns no weight regions
        fols[0].load_weights(w)
    assert e.value.code == B.ESTATE
    with pytest.raises(SdvError) as e:   # followers follow an owner, not one another
        fols[0].follower()
    assert e.value.code == B.EINVAL
    with pytest.raises(SdvError) as e:   # before prefill
        Sdv.verify_batch([lead, fols[0]])
    assert e.value.code == B.ESTATE
    for s in [lead, other] + fols:
        gpu_prefill(s, ctx, cfg.chunk)
    with pytest.raises(SdvError) as e:   # the same sequence twice
        Sdv.verify_batch([lead, lead])
    assert e.value.code == B.EINVAL
    with pytest.raises(SdvError) as e:   # contexts with different weights
        Sdv.verify_batch([lead, other])
    assert e.value.code == B.EINVAL
    for s in [lead] + fols:
        s.draft(cfg.k)
    if 5 * (cfg.k + 1) > 32:
        with pytest.raises(SdvError) as e:   # more rows than one launch takes
            Sdv.verify_batch([lead] + fols)
        assert e.value.code == B.EINVAL
    n = min(32 // (cfg.k + 1), 5)
    assert len(Sdv.verify_batch(([lead] + fols)[:n])) == n
    for s in reversed([lead, other] + fols):
        s.close()


@pytest.mark.parametrize("name", ["qwen1.5b"])
def test_full_size_batch_against_the_stored_trajectory(name):
    """Full size: three sequences on the stored trajectory of the benchmark's context, each at a different
    step of it (so with different KV lengths and drafts), advance in batched steps; every sequence's rows are
    compared with the stored step it is at."""
    path = os.path.join(GOLD, f"{name}.npz")
    if not os.path.exists(path):
        pytest.skip(f"{path} not generated")
    g = np.load(path)
    cfg = get_config(name)
    k = int(g["k"])
    w = make_weights(cfg, threads=16)
    ctx = make_context(cfg)
    steps = steps_from_golden(g)
    lead = Sdv(config_from(cfg, k_max=k))
    lead.load_weights(w)
    seqs = [lead, lead.follower(), lead.follower()]
    at = [0, 1, 3]
    for i, s in enumerate(seqs):
        s.set_parity_mode(True)
        gpu_prefill(s, ctx, cfg.chunk)
        s.debug_set_history(list(ctx) + [int(g["first_token"])], cfg.n_ctx)
        for j in range(at[i]):   # bring the sequence to its starting step along the stored outcome
            s.debug_set_draft(steps[j].draft)
            s.verify(None, fetch=False)
            s.debug_force_commit(len(steps[j].emitted) - 1, steps[j].emitted[-1])
    stats = [{}, {}, {}]
    rounds = 0
    while max(at) < len(steps) and rounds < 6:
        for i, s in enumerate(seqs):
            st = steps[at[i]]
            assert s.kv_len() == st.kv_len_before
            if st.from_drafter:
                assert s.draft(k) == st.draft
            else:
                s.debug_set_draft(st.draft)
        acc = Sdv.verify_batch(seqs)
        for i, s in enumerate(seqs):
            y, a = s.get_verified()
            assert a == acc[i]
            check_verified(s, steps[at[i]], y, a, stats[i])
            at[i] += 1
        rounds += 1
    assert rounds >= 3
    print(name, [(round(st["max_err"], 4), round(st["min_cos"], 6)) for st in stats], "batched step us", lead.last_verify_ms() * 1e3)
    for s in reversed(seqs):
        s.close()
