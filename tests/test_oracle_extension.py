"""Pins for the oracle's draft extension (paper Sec. 4.4, Eq. 3, Table 2): the paper's running
example, the three rejection patterns, a textbook longest-run routine, structural invariants and
losslessness of the decoding loop with the extension switched on."""
import itertools
import os
import random

import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import get_config, make_context, make_weights

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _longest_run_textbook(flags):
    """Longest run of ones, earliest among equals, through string splitting (no index arithmetic
    shared with the oracle)."""
    s = "".join("1" if f else "0" for f in flags)
    runs = [r for r in s.split("0") if r]
    if not runs:
        return 0, 0
    best = max(len(r) for r in runs)
    return s.index("1" * best), best


def test_reuse_segment_matches_textbook_longest_run():
    rng = random.Random(5)
    for _ in range(400):
        n = rng.randint(0, 12)
        x = [rng.randint(0, 2) for _ in range(n)]
        y = [rng.randint(0, 2) for _ in range(n + 1)]
        a = O.accept_len(x, y) if n else 0
        first, length = O.reuse_segment(x, y, a)
        # positions up to and including the reject point never qualify
        flags = [i > a and x[i] == y[i] for i in range(n)]
        assert (first, length) == _longest_run_textbook(flags) or (length == 0 and not any(flags))
        if length:
            assert first > a and all(x[i] == y[i] for i in range(first, first + length))
            assert first - 1 <= a or x[first - 1] != y[first - 1]            # maximal on the left
            assert first + length == n or x[first + length] != y[first + length]  # and on the right


def test_reuse_segment_exhaustive_small():
    """Every draft / prediction pair over two symbols up to length 5 against the definition read
    directly: the best (length, -first) over all admissible ranges."""
    for n in range(0, 6):
        for x in itertools.product((0, 1), repeat=n):
            for y in itertools.product((0, 1), repeat=n + 1):
                a = next((i for i in range(n) if x[i] != y[i]), n)
                ranges = [(l - f + 1, -f) for f in range(a + 1, n) for l in range(f, n)
                          if all(x[i] == y[i] for i in range(f, l + 1))]
                first, length = O.reuse_segment(list(x), list(y), a)
                if ranges:
                    bl, bf = max(ranges)
                    assert (first, length) == (-bf, bl)
                else:
                    assert length == 0


def test_table2_patterns():
    """Table 2: 'missing' keeps the drafts right behind the reject point, 'synonym' keeps a later
    part, 'redundant' keeps nothing."""
    # missing: the model inserts tokens, the draft behind the reject point is still what it predicts
    x = [10, 11, 12, 13, 14]
    y = [10, 99, 12, 13, 14, 15]     # reject at x_2; x_3..x_5 agree with the predictions
    assert O.accept_len(x, y) == 1
    assert O.reuse_segment(x, y, 1) == (2, 3)
    # synonym: a few more positions disagree before the agreement resumes
    y = [10, 99, 98, 13, 14, 15]
    assert O.reuse_segment(x, y, 1) == (3, 2)
    # redundant: nothing agrees behind the reject point
    y = [10, 99, 98, 97, 96, 95]
    assert O.reuse_segment(x, y, 1) == (0, 0)
    # full acceptance: no reject point, nothing to keep
    y = [10, 11, 12, 13, 14, 15]
    assert O.reuse_segment(x, y, 5) == (0, 0)
    # two runs of equal length: the earlier one
    x = [1, 2, 3, 4, 5, 6, 7]
    y = [0, 2, 3, 0, 5, 6, 0, 8]
    assert O.reuse_segment(x, y, 0) == (1, 2)


def test_paper_running_example_reuses_the_tail():
    """Sec. 4.3 / 4.4: after "arrived" is emitted, the rest of the model's continuation sits in the
    rejected draft; kept by Eq. 3 and appended to the next draft it is accepted whole."""
    fields = {}
    with open(os.path.join(GOLD, "paper_sec4_3_running_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or ":" not in line:
                continue
            key, val = line.split(":", 1)
            fields[key.strip()] = val.split()
    vocab = {}
    tid = lambda w: vocab.setdefault(w, len(vocab))
    T = tid(fields["committed"][0])
    x = [tid(w) for w in fields["draft"]]
    model_words = fields["model"]
    nxt = {T: tid(model_words[0])}
    for p, q in zip(model_words, model_words[1:]):
        nxt[tid(p)] = tid(q)
    other = tid("<other>")
    predict = lambda row: [nxt.get(prev, other) for prev in row]
    inv = {v: k for k, v in vocab.items()}

    ext = O.DraftExtension()
    d1 = ext.extend(x)
    assert d1 == x                               # nothing retained yet
    y = predict([T] + d1)
    a = O.accept_len(d1, y)
    ext.update(d1, y, a)
    assert [inv[t] for t in ext.seg] == fields["reused"]
    emitted = d1[:a] + [y[a]]
    # next step: the retrieval drafter finds nothing; the draft is the retained segment alone
    T2 = emitted[-1]
    d2 = ext.extend([])
    assert [inv[t] for t in d2] == fields["reused"]
    y2 = predict([T2] + d2)
    a2 = O.accept_len(d2, y2)
    assert a2 == int(fields["next_step_accepted_drafts"][0])
    ext.update(d2, y2, a2)
    assert ext.seg == []                         # spent


def test_extension_state_rules():
    ext = O.DraftExtension(max_total=6, max_life=2)
    x = [1, 2, 3, 4]
    y = [9, 2, 3, 9, 5]
    ext.update(ext.extend(x), y, 0)
    assert ext.seg == [2, 3] and ext.life == 0
    # appended and not reached: ages by one per verify step, survives max_life steps, then goes
    for step in range(1, 4):
        d = ext.extend([7])
        assert d == [7, 2, 3] and ext.used
        ext.update(d, [8, 8, 8, 8], 0)
        if step <= 2:
            assert ext.seg == [2, 3] and ext.life == step
        else:
            assert ext.seg == []
    # a draft that would pass max_total drops the segment instead of cutting it
    ext.update(ext.extend(x), y, 0)
    assert ext.seg == [2, 3]
    assert ext.extend([7, 7, 7, 7, 7]) == [7, 7, 7, 7, 7] and ext.seg == []
    # not appended (extend not reaching it) leaves the lifetime alone; a strictly longer candidate replaces
    ext.update(ext.extend(x), y, 0)
    d = ext.extend([5, 6])
    ext.update(d, [0, 6, 2, 3, 0], 0)       # candidate 6, 2, 3 (length 3) beats the retained pair
    assert ext.seg == [6, 2, 3] and ext.life == 0
    # the same segment found again in its own copy does not renew the lifetime
    d = ext.extend([1])
    ext.update(d, [0, 6, 2, 3, 0], 0)
    assert ext.seg == [6, 2, 3] and ext.life == 1
    # accepted prefix reaching into the segment spends it; what agrees behind the new reject point
    # comes back as a fresh candidate
    d = ext.extend([1])
    ext.update(d, [1, 6, 0, 3, 0], 2)
    assert ext.seg == [3] and ext.life == 0
    d = ext.extend([1])
    ext.update(d, [1, 3, 0], 2)
    assert ext.seg == []


@pytest.fixture(scope="module")
def tiny():
    cfg = get_config("tiny")
    w = make_weights(cfg)
    ctx = make_context(cfg)
    greedy = O.greedy_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk)
    return cfg, w, ctx, greedy


def test_extension_is_lossless_and_bounded(tiny):
    """Whatever is appended, the emitted tokens stay those of plain greedy decoding (Sec. 5.1:
    strict verification), and no draft grows beyond the threshold."""
    cfg, w, ctx, greedy = tiny
    rng = np.random.default_rng(3)

    def noisy(hist, k):
        # the true continuation with random corruptions: rejects followed by agreeing tails
        i0 = len(hist) - cfg.n_ctx
        d = [greedy[i0 + i] if i0 + i < cfg.gen else 0 for i in range(k)]
        for i in range(k):
            if rng.random() < 0.3:
                d[i] = (d[i] + 1) % cfg.vocab
        return d

    for max_total in (cfg.k, cfg.k + 4, 32):
        ext = O.DraftExtension(max_total=max_total, max_life=3)
        m = O.OracleModel(w)
        toks, steps = O.spec_decode(m, ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min,
                                    drafter=noisy, extension=ext)
        assert toks == greedy
        assert all(len(s.draft) <= max(max_total, cfg.k) for s in steps)
        if max_total > cfg.k:
            assert any(len(s.draft) > cfg.k for s in steps)   # the extension did lengthen drafts
