"""Draft extension (paper Sec. 4.4, Eq. 3) on the GPU against the oracle: the integer state machine
bit for bit on forced drafts and predictions, verify steps of up to 32 rows, and the decoding loop
with the extension switched on, step by step."""
import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import get_config, make_context, make_weights
import paper_2510_15312_b200 as pkg
from paper_2510_15312_b200.binding import Sdv, config_from

from helpers import compare_step, steps_from_oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("max_total,max_life", [(31, 3), (12, 1), (20, 32), (1, 2)])
def test_extension_state_machine_bit_exact(max_total, max_life):
    """No model: drafts and predictions are given; extend / accept / update must reproduce the
    oracle's retained segment, lifetime and extended drafts exactly."""
    s = Sdv(config_from(get_config("tiny"), k_max=31, max_seq=4096))
    rng = np.random.default_rng(max_total * 100 + max_life)
    s.debug_set_history(rng.integers(0, 50, 40).astype(np.int32), 30)
    ext = O.DraftExtension(max_total=max_total, max_life=max_life)
    seen_used = seen_drop = seen_replace = 0
    for step in range(400):
        base = rng.integers(0, 6, int(rng.integers(0, min(max_total, 12) + 1))).tolist()
        s.debug_set_draft(base)
        before = list(ext.seg)
        want = ext.extend(base)
        got = s.extend_draft(max_total)
        assert got == want, (step, base, before)
        seen_used += ext.used
        seen_drop += bool(before) and not ext.seg
        # predictions: agree with the draft with probability p (runs of agreement behind a reject)
        p = rng.choice([0.3, 0.6, 0.9])
        y = [t if rng.random() < p else int(rng.integers(0, 6)) for t in want] + [int(rng.integers(0, 6))]
        a = s.debug_accept(None, y)
        assert a == O.accept_len(want, y)
        prev = list(ext.seg)
        ext.update(want, y, a)
        seg, life = s.extension_update(max_life)
        assert (seg, life) == (ext.seg, ext.life), (step, want, y, a, prev)
        seen_replace += ext.seg != prev and bool(ext.seg)
    if max_total > 4:   # a one-token draft has nothing beyond its reject point
        assert seen_replace > 10 and seen_used > 10
    s.close()


def test_extension_call_order():
    s = Sdv(config_from(get_config("tiny"), k_max=8, max_seq=4096))
    s.debug_set_history(np.arange(40, dtype=np.int32), 30)
    with pytest.raises(pkg.SdvError):
        s.extension_update(3)            # no verify result
    with pytest.raises(pkg.SdvError):
        s.extend_draft(9)                # beyond k_max
    s.debug_set_draft([1, 2, 3])
    assert s.extend_draft(8) == [1, 2, 3]
    a = s.debug_accept(None, [1, 9, 3, 4])
    assert a == 1
    assert s.extension_update(3) == ([3], 0)
    s.commit()
    s.rollback(s.kv_len())               # a rollback clears the retained segment
    s.debug_set_draft([5])
    assert s.extend_draft(8) == [5]
    s.close()


def _noisy_continuation(cfg, greedy, rate, seed):
    """The true continuation with seeded corruptions that depend on the position only."""
    def drafter(hist, k):
        i0 = len(hist) - cfg.n_ctx
        d = []
        for i in range(k):
            pos = i0 + i
            t = greedy[pos] if pos < cfg.gen else 0
            if np.random.default_rng(seed * 100003 + pos * 31 + len(hist)).random() < rate:
                t = (t + 1) % cfg.vocab
            d.append(int(t))
        return d
    return drafter


@pytest.mark.parametrize("name", ["tiny", "mini_gqa", "mini_hd128"])
def test_verify_up_to_32_rows_matches_oracle(name):
    """Drafts of 17..31 tokens (the lengths the extension produces) through the verify step."""
    base = get_config(name)
    cfg = base.with_(k=31, gen=96)
    w, ctx = make_weights(cfg), make_context(cfg)
    greedy = O.greedy_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk)
    lens = iter([31, 17, 24, 29, 20, 31, 18, 27] * 8)
    cont = _noisy_continuation(cfg, greedy, 0.08, 1)
    drafter = lambda hist, k: cont(hist, next(lens))
    toks, steps = O.spec_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min,
                                drafter=drafter, keep_logits=True)
    assert toks == greedy
    s = Sdv(config_from(cfg))
    s.load_weights(w)
    s.set_parity_mode(True)
    for i in range(0, cfg.n_ctx, cfg.chunk):
        s.prefill_chunk(ctx[i:i + cfg.chunk], is_last=(i + cfg.chunk >= cfg.n_ctx))
    s.debug_set_history(list(ctx) + [toks[0]], cfg.n_ctx)
    stats = {}
    for st in steps_from_oracle(steps, from_drafter=False):
        compare_step(s, st, cfg.k, stats)
    assert max(len(st.draft) for st in steps) >= 29
    assert max(stats["accepts"]) >= 8
    print(name, stats.get("max_err"), stats.get("min_cos"), stats.get("near_tie_flips", 0))
    s.close()


@pytest.mark.parametrize("name", ["tiny", "mini_gqa"])
def test_decoding_loop_with_extension_step_by_step(name):
    """The oracle's loop with the extension against draft / extend / verify / update / commit on the
    GPU: same extended drafts, same predictions (within the logit tolerance), same retained segment."""
    base = get_config(name)
    k, max_total, max_life = 6, 24, 3
    cfg = base.with_(k=k, gen=200)
    w, ctx = make_weights(cfg), make_context(cfg)
    greedy = O.greedy_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk)
    drafter = _noisy_continuation(cfg, greedy, 0.25, 2)
    ext = O.DraftExtension(max_total=max_total, max_life=max_life)
    toks, steps = O.spec_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk, k, cfg.ngram_n, cfg.ngram_min,
                                drafter=drafter, keep_logits=True, extension=ext)
    assert toks == greedy                                   # lossless
    assert any(len(st.draft) > k for st in steps)           # the extension lengthened drafts
    s = Sdv(config_from(cfg, k_max=max_total))
    s.load_weights(w)
    s.set_parity_mode(True)
    for i in range(0, cfg.n_ctx, cfg.chunk):
        s.prefill_chunk(ctx[i:i + cfg.chunk], is_last=(i + cfg.chunk >= cfg.n_ctx))
    hist = list(ctx) + [toks[0]]
    s.debug_set_history(hist, cfg.n_ctx)
    mirror = O.DraftExtension(max_total=max_total, max_life=max_life)
    stats = {}
    for st in steps_from_oracle(steps, from_drafter=False):
        b = drafter(hist, k)
        s.debug_set_draft(b)
        want = mirror.extend(b)
        assert want == st.draft
        assert s.extend_draft(max_total) == st.draft

        def after_verify(y, a, want=want):
            mirror.update(want, y, a)
            assert s.extension_update(max_life) == (mirror.seg, mirror.life)

        flips = stats.get("near_tie_flips", 0)
        compare_step(s, st, k, stats, predrafted=True, before_commit=after_verify)
        if stats.get("near_tie_flips", 0) != flips:
            break   # the device legitimately took the runner-up: its retained segment may now differ
        hist.extend(st.emitted)
    assert stats["steps"] >= min(len(steps), 8)
    print(name, stats.get("steps"), "of", len(steps), stats.get("max_err"), stats.get("near_tie_flips", 0))
    s.close()
