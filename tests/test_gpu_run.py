"""sdv_decode_steps: a run of draft -> verify -> commit steps enqueued without the host in between.
Its emitted stream must be the one the oracle's loop produces (lossless: the plain greedy stream) up to
the first position where the oracle's own top-2 margin is below the tolerance, the token budget must cut
the run exactly, and the run must leave the context where the same calls made one by one leave it."""
import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import get_config, make_context, make_weights
from paper_2510_15312_b200 import binding as B
from paper_2510_15312_b200.binding import Sdv, SdvError, config_from
from helpers import MARGIN_TOL

pytestmark = pytest.mark.gpu


def gpu_prefill(s, ctx, chunk):
    n = len(ctx)
    for i in range(0, n, chunk):
        s.prefill_chunk(ctx[i:i + chunk], is_last=(i + chunk >= n))


def oracle_stream(cfg, w, ctx, extension=None):
    ref = O.OracleModel(w)
    last = ref.prefill(ctx, cfg.chunk)
    toks, steps = O.spec_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min,
                                search_history=True, extension=extension)
    margins = [O.top2_margin(last)]
    for st in steps:
        margins.extend(st.margin[:len(st.emitted)])
    first_tie = next((i for i, m in enumerate(margins) if m < MARGIN_TOL), len(margins))
    return toks, steps, first_tie


def matched_prefix(a, b):
    n = 0
    for x, y in zip(a, b):
        if x != y:
            break
        n += 1
    return n


@pytest.mark.parametrize("name", ["tiny", "mini_gqa", "mini_hd128"])
def test_run_emits_the_oracle_stream_and_stops_at_the_budget(name):
    cfg = get_config(name)
    w, ctx = make_weights(cfg), make_context(cfg)
    toks, steps, first_tie = oracle_stream(cfg, w, ctx)
    s = Sdv(config_from(cfg, search_history=True, max_seq=cfg.n_ctx + 4 * cfg.gen * (cfg.k + 1) + 64))
    s.load_weights(w)
    gpu_prefill(s, ctx, cfg.chunk)
    budget = cfg.gen - 1                      # the first token is the pending one prefill leaves
    n_steps = budget + 3                      # more steps than needed: the run must end by its budget
    out, kv = s.decode_steps(cfg.k, n_steps, max_tokens=budget)
    assert len(out) == budget and kv == cfg.n_ctx + budget == s.kv_len()
    required = max(0, min(first_tie, len(toks)) - 1)
    assert matched_prefix(out, toks[1:]) >= required, (matched_prefix(out, toks[1:]), first_tie)
    ms = s.run_kernel_ms(n_steps)
    used = int((ms > 0.02).sum())             # steps behind the end of the run return at once
    assert used <= len(steps) + 2 and used < n_steps and np.all(ms[used:] < 0.02)
    if required == len(toks) - 1:
        assert used == len(steps)             # same stream, same accept lengths, same number of steps
    # the context goes on where the run stopped, by single calls and by another run alike
    s.draft(cfg.k, fetch=False)
    s.verify(None, fetch=False)
    e1, kv1 = s.commit()
    s.rollback(kv)
    e2, kv2 = s.decode_steps(cfg.k, 1)
    assert e1 == e2 and kv1 == kv2
    s.close()


@pytest.mark.parametrize("name", ["tiny", "mini_gqa"])
def test_run_equals_the_same_calls_made_one_by_one(name):
    """Two contexts on the same weights and context: one stepped by single calls, one by runs of several
    steps.  Integer state is compared after every run; streams may part only at a near-tie."""
    cfg = get_config(name)
    w, ctx = make_weights(cfg), make_context(cfg)
    toks, _, first_tie = oracle_stream(cfg, w, ctx)
    a = Sdv(config_from(cfg, search_history=True, max_seq=cfg.n_ctx + 2 * cfg.gen * (cfg.k + 1) + 64))
    a.load_weights(w)
    b = a.follower()
    for s in (a, b):
        gpu_prefill(s, ctx, cfg.chunk)
    out_a, out_b = [], []
    for n in (1, 2, 5, 3):
        for _ in range(n):
            a.draft(cfg.k, fetch=False)
            a.verify(None, fetch=False)
            e, _ = a.commit()
            out_a += e
        e, kv_b = b.decode_steps(cfg.k, n)
        out_b += e
        m = matched_prefix(out_a, out_b)
        if m < min(len(out_a), len(out_b)):
            assert m + 1 >= first_tie, (m, first_tie)   # parted: only where the oracle itself is near a tie
            break
        assert out_a == out_b and a.kv_len() == kv_b == b.kv_len()
    assert len(out_b) >= 4
    b.close()
    a.close()


def test_run_with_draft_extension_matches_the_oracle_loop():
    cfg = get_config("mini_gqa").with_(k=6, gen=60)
    max_total, max_life = 20, 3
    w, ctx = make_weights(cfg), make_context(cfg)
    ext = O.DraftExtension(max_total=max_total, max_life=max_life)
    toks, steps, first_tie = oracle_stream(cfg, w, ctx, extension=ext)
    s = Sdv(config_from(cfg, k_max=max_total, search_history=True, max_seq=cfg.n_ctx + 80 * (max_total + 1)))
    s.load_weights(w)
    gpu_prefill(s, ctx, cfg.chunk)
    out, kv = s.decode_steps(cfg.k, cfg.gen + 2, max_tokens=cfg.gen - 1, ext_max_total=max_total, ext_max_life=max_life)
    assert len(out) == cfg.gen - 1 and kv == cfg.n_ctx + cfg.gen - 1
    required = max(0, min(first_tie, len(toks)) - 1)
    assert matched_prefix(out, toks[1:]) >= required
    s.close()


def test_run_argument_and_capacity_errors():
    cfg = get_config("tiny")
    w, ctx = make_weights(cfg), make_context(cfg)
    s = Sdv(config_from(cfg, max_seq=cfg.n_ctx + 40))
    s.load_weights(w)
    with pytest.raises(SdvError) as e:
        s.decode_steps(cfg.k, 2)
    assert e.value.code == B.ESTATE            # before prefill
    gpu_prefill(s, ctx, cfg.chunk)
    for bad in (dict(k=0, n_steps=1), dict(k=cfg.k + 1, n_steps=1), dict(k=cfg.k, n_steps=0),
                dict(k=cfg.k, n_steps=1, ext_max_total=cfg.k - 1, ext_max_life=1),
                dict(k=cfg.k, n_steps=1, ext_max_total=cfg.k, ext_max_life=0)):
        with pytest.raises(SdvError) as e:
            s.decode_steps(**bad)
        assert e.value.code == B.EINVAL, bad
    with pytest.raises(SdvError) as e:
        s.decode_steps(cfg.k, 9)               # 9 x 5 rows do not fit behind the context
    assert e.value.code == B.ECAPACITY
    with pytest.raises(SdvError) as e:
        s.run_kernel_ms(1)                     # no run yet
    assert e.value.code == B.ESTATE
    out, kv = s.decode_steps(cfg.k, 8)
    assert kv == cfg.n_ctx + len(out) and len(out) >= 8
    s.close()


@pytest.mark.parametrize("name", ["tiny", "mini_gqa"])
def test_one_call_step_equals_draft_verify_commit(name):
    """sdv_step against the same step made of sdv_draft / sdv_verify / sdv_commit on a second sequence: emitted
    tokens, KV length and the draft handed back for the next step, with host drafts and with the device's."""
    cfg = get_config(name)
    w, ctx = make_weights(cfg), make_context(cfg)
    toks, _, first_tie = oracle_stream(cfg, w, ctx)
    a = Sdv(config_from(cfg, search_history=True, max_seq=cfg.n_ctx + 2 * cfg.gen * (cfg.k + 1) + 64))
    a.load_weights(w)
    b = a.follower()
    for s in (a, b):
        gpu_prefill(s, ctx, cfg.chunk)
    da = a.draft(cfg.k)
    db = b.draft(cfg.k)
    assert da == db
    out_a, out_b = [], []
    for i in range(min(cfg.gen - 2, 16)):
        ya, _ = a.verify(da if i % 2 else None)          # host draft on odd steps, the device's own on even ones
        ea, kva = a.commit()
        da = a.draft(cfg.k)
        eb, db, kvb = b.step(db if i % 2 else None, cfg.k)
        out_a += ea
        out_b += eb
        if out_a != out_b:
            assert matched_prefix(out_a, out_b) + 1 >= first_tie   # parted at a near-tie only
            break
        assert kva == kvb == b.kv_len() and da == db
    assert len(out_b) >= 4 and matched_prefix(out_b, toks[1:]) >= max(0, min(first_tie, len(out_b) + 1) - 1)
    eb, db, _ = b.step(None, 0)                          # no next draft asked for
    assert db == [] and len(eb) >= 1
    with pytest.raises(SdvError) as e:
        b.step([cfg.vocab], cfg.k)
    assert e.value.code == B.EINVAL
    b.close()
    a.close()
