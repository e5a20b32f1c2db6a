"""Pins for the oracle's forward pass and decoding loops: a dense fp64 restatement of the
decoder in matrix form, invariants the paper fixes (lossless decoding, graph equivalence of
chunked prefill, accepted-prefix rule), and brute force for the integer parts."""
import math
import os

import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import bf16_bits_to_f32, get_config, make_context, make_weights

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ dense fp64 decoder
def _w(bits):
    return bf16_bits_to_f32(bits).astype(np.float64)


def dense_forward_fp64(weights, tokens):
    """Whole-sequence decoder in matrix form (explicit T x T causal score matrix), fp64."""
    c = weights.cfg
    T, hd, g = len(tokens), c.head_dim, c.n_q_heads // c.n_kv_heads
    h = _w(weights.emb)[np.asarray(tokens)]
    inv = c.rope_theta ** (-2.0 * np.arange(hd // 2) / hd)
    ang = np.arange(T)[:, None] * inv[None, :]
    cos, sin = np.cos(ang), np.sin(ang)

    def norm(x, w):
        return x / np.sqrt((x * x).mean(-1, keepdims=True) + c.rms_eps) * w

    def rot(x):  # x [T, heads, hd]
        a, b = x[..., :hd // 2], x[..., hd // 2:]
        return np.concatenate([a * cos[:, None] - b * sin[:, None], b * cos[:, None] + a * sin[:, None]], -1)

    mask = np.tril(np.ones((T, T), dtype=bool))
    for L in weights.layers:
        xn = norm(h, L.norm1)
        q = xn @ _w(L.wq).T + (0 if L.bq is None else L.bq)
        k = xn @ _w(L.wk).T + (0 if L.bk is None else L.bk)
        v = xn @ _w(L.wv).T + (0 if L.bv is None else L.bv)
        q = rot(q.reshape(T, c.n_q_heads, hd))
        k = rot(k.reshape(T, c.n_kv_heads, hd))
        v = v.reshape(T, c.n_kv_heads, hd)
        o = np.empty_like(q)
        for a in range(c.n_q_heads):
            s = q[:, a] @ k[:, a // g].T / math.sqrt(hd)
            s = np.where(mask, s, -np.inf)
            p = np.exp(s - s.max(-1, keepdims=True))
            p /= p.sum(-1, keepdims=True)
            o[:, a] = p @ v[:, a // g]
        h = h + o.reshape(T, -1) @ _w(L.wo).T
        xn = norm(h, L.norm2)
        gt, up = xn @ _w(L.wg).T, xn @ _w(L.wu).T
        h = h + (gt / (1 + np.exp(-gt)) * up) @ _w(L.wd).T
    lm = weights.emb if weights.lm_head is None else weights.lm_head
    return norm(h, weights.final_norm) @ _w(lm).T


@pytest.fixture(scope="module", params=["mini_gqa", "mini_hd128"])
def mini(request):
    cfg = get_config(request.param)
    return cfg, make_weights(cfg), make_context(cfg)


def test_forward_matches_dense_fp64(mini):
    cfg, w, ctx = mini
    toks = ctx[:37]
    ref = dense_forward_fp64(w, toks)
    m = O.OracleModel(w)
    got = m.forward(toks, 0, logits_from=0)
    assert np.abs(got - ref).max() < 2e-4
    assert np.array_equal(got.argmax(-1), ref.argmax(-1))
    # the same tokens fed as 20 + 17 with the cache in between
    m2 = O.OracleModel(w)
    m2.forward(toks[:20], 0, logits_from=None)
    got2 = m2.forward(toks[20:], 20, logits_from=0)
    assert np.abs(got2 - ref[20:]).max() < 2e-4


def test_gqa_equals_mha_with_duplicated_kv_heads(mini):
    cfg, w, ctx = mini
    g, hd = cfg.n_q_heads // cfg.n_kv_heads, cfg.head_dim
    import copy
    w2 = copy.copy(w)
    w2.cfg = cfg.with_(n_kv_heads=cfg.n_q_heads)
    w2.layers = []
    for L in w.layers:
        L2 = copy.copy(L)
        dup = lambda a: None if a is None else np.ascontiguousarray(
            np.repeat(a.reshape(cfg.n_kv_heads, hd, *a.shape[1:]), g, axis=0).reshape(-1, *a.shape[1:]))
        L2.wk, L2.wv, L2.bk, L2.bv = dup(L.wk), dup(L.wv), dup(L.bk), dup(L.bv)
        w2.layers.append(L2)
    a = O.OracleModel(w).forward(ctx[:19], 0)
    b = O.OracleModel(w2).forward(ctx[:19], 0)
    np.testing.assert_array_equal(a, b)


def test_chunked_prefill_is_bit_identical(mini):
    """Sec. 4.2 graph equivalence: short pieces one after another == one long run."""
    cfg, w, ctx = mini
    n = 150
    ref_m = O.OracleModel(w)
    ref = ref_m.prefill(ctx[:n], n)
    for chunk in (1, 17, 64):
        m = O.OracleModel(w)
        got = m.prefill(ctx[:n], chunk)
        np.testing.assert_array_equal(got, ref)
        np.testing.assert_array_equal(m.kv_view("k")[:, :, :n], ref_m.kv_view("k")[:, :, :n])
        np.testing.assert_array_equal(m.kv_view("v")[:, :, :n], ref_m.kv_view("v")[:, :, :n])


# ------------------------------------------------------------------ lossless decoding
@pytest.fixture(scope="module")
def tiny():
    cfg = get_config("tiny")
    w = make_weights(cfg)
    ctx = make_context(cfg)
    greedy = O.greedy_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk)
    return cfg, w, ctx, greedy


def _run(tiny, **kw):
    cfg, w, ctx, _ = tiny
    m = O.OracleModel(w)
    toks, steps = O.spec_decode(m, ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min, **kw)
    return m, toks, steps


def _check_kv_closed_form(cfg, m, toks, steps):
    assert len(toks) == cfg.gen
    L = cfg.n_ctx
    for s in steps:
        assert s.kv_len_before == L
        assert 1 <= len(s.emitted) <= s.accept + 1
        L += len(s.emitted)
        assert s.kv_len_after == L
    assert L == cfg.n_ctx + cfg.gen - 1 == m.kv_len   # the last emitted token's KV row is not written yet


def test_ngram_drafts_are_lossless(tiny):
    cfg, _, _, greedy = tiny
    for hist_mode in (False, True):
        m, toks, steps = _run(tiny, search_history=hist_mode)
        assert toks == greedy
        _check_kv_closed_form(cfg, m, toks, steps)
    assert any(s.accept > 0 for s in steps)   # the history search finds the stream's own repeats


def test_wrong_drafts_are_lossless(tiny):
    cfg, _, _, greedy = tiny
    bad = lambda hist, k: [(greedy[len(hist) - cfg.n_ctx + i] + 1) % cfg.vocab if len(hist) - cfg.n_ctx + i < cfg.gen
                           else 0 for i in range(k)]
    m, toks, steps = _run(tiny, drafter=bad)
    assert toks == greedy
    assert all(s.accept == 0 and len(s.emitted) == 1 for s in steps)
    _check_kv_closed_form(cfg, m, toks, steps)


def _true_continuation(cfg, greedy, corrupt_at=None):
    def drafter(hist, k):
        i0 = len(hist) - cfg.n_ctx          # index in `greedy` of the next token
        d = [greedy[i0 + i] if i0 + i < cfg.gen else 0 for i in range(k)]
        if corrupt_at is not None:
            d[corrupt_at - 1] = (d[corrupt_at - 1] + 1) % cfg.vocab
        return d
    return drafter


def test_true_continuation_is_fully_accepted(tiny):
    cfg, _, _, greedy = tiny
    m, toks, steps = _run(tiny, drafter=_true_continuation(cfg, greedy))
    assert toks == greedy
    for s in steps[:-1]:
        assert s.accept == cfg.k and s.emitted == s.draft + [s.y[-1]]
    _check_kv_closed_form(cfg, m, toks, steps)


@pytest.mark.parametrize("e", [1, 2, 3, 4])
def test_corruption_at_e_accepts_e_minus_1(tiny, e):
    """Sec. 4.4: a mismatch at position e leaves the accepted prefix x_1..x_{e-1}, y_e."""
    cfg, _, _, greedy = tiny
    m, toks, steps = _run(tiny, drafter=_true_continuation(cfg, greedy, corrupt_at=e))
    assert toks == greedy
    for s in steps[:-1]:
        assert s.accept == e - 1
        assert s.emitted == s.draft[:e - 1] + [s.y[e - 1]]
    _check_kv_closed_form(cfg, m, toks, steps)


# ------------------------------------------------------------------ integer parts
def brute_force_draft(search, hist, n, n_min, k, exclude_from=None):
    """All (position, length) pairs tried one by one."""
    search, hist = list(search), list(hist)
    lim = len(search) if exclude_from is None else exclude_from
    best = None
    for length in range(1, n + 1):
        if length > len(hist):
            break
        suffix = hist[-length:]
        for end in range(length - 1, len(search)):        # `end` = index of the match's last token
            if end >= lim or end + 1 >= len(search):
                continue
            if search[end - length + 1:end + 1] == suffix and length >= n_min:
                if best is None or (length, end) > best:
                    best = (length, end)
    if best is None:
        return [], -1, 0
    return search[best[1] + 1:best[1] + 1 + k], best[1], best[0]


def test_ngram_matcher_against_brute_force():
    rng = np.random.default_rng(7)
    for trial in range(400):
        V = int(rng.integers(2, 6))
        ns, nh = int(rng.integers(1, 40)), int(rng.integers(1, 12))
        search = rng.integers(0, V, ns)
        hist = rng.integers(0, V, nh)
        n, k = int(rng.integers(1, 5)), int(rng.integers(1, 9))
        n_min = int(rng.integers(1, n + 1))
        d, p, ml = O.ngram_draft(search, hist, n, n_min, k)
        bd, bp, bl = brute_force_draft(search, hist, n, n_min, k)
        assert (d.tolist(), p, ml) == (bd, bp, bl), (trial, search, hist, n, n_min, k)
        # history mode: the history searched against itself, never matching its own tail
        d, p, ml = O.ngram_draft(hist, hist, n, n_min, k, exclude_from=len(hist) - 1)
        bd, bp, bl = brute_force_draft(hist, hist, n, n_min, k, exclude_from=len(hist) - 1)
        assert (d.tolist(), p, ml) == (bd, bp, bl)


def test_ngram_matcher_edge_cases():
    C = [5, 6, 7, 8, 5, 6, 9, 9, 5, 6, 7]
    # latest of two equally long matches wins: "5 6" at 4-5 (then 9 9 5 6) beats 0-1; the one at 8-9 is
    # followed by a single token only, but it is the latest
    assert O.ngram_draft(C, [1, 5, 6], 3, 1, 4)[0].tolist() == [7]
    # the longest match wins over a later shorter one: suffix "5 6 7" matches at 0-2 only in full
    assert O.ngram_draft(C[:10], [5, 6, 7], 3, 1, 3)[0].tolist() == [8, 5, 6]
    # a match ending at the last context token has no continuation and is not a candidate
    assert O.ngram_draft([1, 2, 3], [9, 3], 3, 1, 4)[0].tolist() == []
    assert O.ngram_draft([3, 2, 3], [9, 3], 3, 1, 4)[0].tolist() == [2, 3]
    # nothing matches
    assert O.ngram_draft([1, 2, 3], [4], 3, 1, 4)[0].tolist() == []
    # minimum match length
    assert O.ngram_draft([1, 2, 3, 4], [7, 2], 3, 2, 4)[0].tolist() == []
    assert O.ngram_draft([1, 2, 3, 4], [1, 2], 3, 2, 4)[0].tolist() == [3, 4]
    # history shorter than n
    assert O.ngram_draft([1, 2, 3, 4], [2], 3, 1, 2)[0].tolist() == [3, 4]


def test_accept_scan_on_hand_made_vectors():
    assert O.accept_len([], [9]) == 0
    assert O.accept_len([1, 2, 3], [1, 2, 3, 4]) == 3
    assert O.accept_len([1, 2, 3], [1, 9, 3, 4]) == 1     # a later coincidence (x_3 = y_3) is not accepted
    assert O.accept_len([1, 2, 3], [7, 2, 3, 4]) == 0


def test_paper_running_example_accepts_one_token():
    """Sec. 4.3: the draft "'s security detail has arrived at Des Moines" against a model that
    continues "Clinton" with "arrived at Des Moines" yields one emitted token, "arrived"."""
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
    # table-driven mock model: its prediction after the committed token follows its own continuation;
    # after a draft token it has never produced itself it predicts some unrelated token
    nxt = {T: tid(model_words[0])}
    for a, b in zip(model_words, model_words[1:]):
        nxt[tid(a)] = tid(b)
    other = tid("<other>")
    y = [nxt.get(prev, other) for prev in [T] + x]
    a = O.accept_len(x, y)
    emitted = x[:a] + [y[a]]
    inv = {v: k for k, v in vocab.items()}
    assert a == int(fields["accepted_drafts"][0])
    assert [inv[t] for t in emitted] == fields["emitted"]


@pytest.mark.parametrize("name", ["qwen1.5b", "llama3b", "qwen7b"])
def test_stored_trajectories_are_self_consistent(name):
    """The stored full-size trajectories (written by tests/golden/make_golden.py from the oracle
    alone) obey what the method fixes: y is the greedy token of its row, the stored margin is the
    gap to the runner-up, the accept length is the length of the matching prefix, the emitted
    tokens are x_1..x_a, y_{a+1} (Sec. 4.4) and the KV length advances by the emitted count."""
    g = np.load(os.path.join(GOLD, f"{name}.npz"))
    S = len(g["accept"])
    emitted_all = [int(g["first_token"])]
    for i in range(S):
        dl, a, ne = int(g["draft_len"][i]), int(g["accept"][i]), int(g["n_emitted"][i])
        x, y = g["draft"][i, :dl].tolist(), g["y"][i, :dl + 1].tolist()
        assert a == O.accept_len(x, y)
        want = x[:a] + [y[a]]
        assert g["emitted"][i, :ne].tolist() == want[:ne] and (ne == len(want) or i == S - 1)
        if i + 1 < S:
            assert int(g["kv_len_before"][i + 1]) == int(g["kv_len_before"][i]) + ne
            assert int(g["pending"][i + 1]) == want[ne - 1]
        for r in range(dl + 1):
            ids, vals = g["top_ids"][i, r], g["top_vals"][i, r]
            assert int(ids[0]) == y[r]
            assert np.all(vals[:-1] >= vals[1:])
            ties = vals[:-1] == vals[1:]
            assert np.all(ids[:-1][ties] < ids[1:][ties])          # equal values: lower id first
            assert float(g["margin"][i, r]) == float(vals[0] - vals[1])
        emitted_all += want[:ne]
    assert emitted_all == g["tokens"].tolist()[:len(emitted_all)]
