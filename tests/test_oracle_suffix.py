"""Pins for longest-suffix retrieval (the drafter with an unbounded suffix length over context and
generated tokens: the match a suffix automaton returns, cited as SAM in Sec. 5.1 (3) of the paper):
the oracle's matcher against Python's own substring search on byte strings."""
import numpy as np
import pytest

from oracle import sdv_oracle as O

N_MAX = 4096


def _by_substring_search(search: bytes, hist: bytes, n_min: int, exclude_from: int):
    """Longest suffix of hist (at least n_min, at most N_MAX bytes) that occurs in search ending at
    a position p with a continuation (p + 1 < len(search)) and p < exclude_from; among its
    occurrences the latest.  Returns (p, length) or (-1, 0).  Uses bytes.rfind only."""
    last_p = min(len(search) - 2, exclude_from - 1)     # latest admissible end position
    for length in range(min(len(hist), N_MAX, last_p + 1), max(n_min, 1) - 1, -1):
        idx = search.rfind(hist[len(hist) - length:], 0, last_p + 1)
        if idx >= 0:
            return idx + length - 1, length
    return -1, 0


@pytest.mark.parametrize("search_history", [False, True])
def test_longest_suffix_equals_substring_search(search_history):
    rng = np.random.default_rng(21 + search_history)
    hits = 0
    for trial in range(300):
        V = int(rng.integers(2, 5))
        n_ctx = int(rng.integers(1, 200))
        n_gen = int(rng.integers(1, 40))
        hist = rng.integers(0, V, n_ctx + n_gen).astype(np.int32)
        if trial % 3 == 0 and n_ctx > 60:                 # plant a long repeat of the suffix
            L = int(rng.integers(5, 40))
            p = int(rng.integers(L, n_ctx - 10))
            hist[p - L:p] = hist[-L:]
        n_min = int(rng.integers(1, 4))
        k = int(rng.integers(1, 17))
        if search_history:
            search, ex = hist, len(hist) - 1
        else:
            search, ex = hist[:n_ctx], n_ctx
        draft, mp, ml = O.ngram_draft(search, hist, N_MAX, n_min, k, exclude_from=ex)
        rp, rl = _by_substring_search(bytes(search.astype(np.uint8)), bytes(hist.astype(np.uint8)), n_min, ex)
        assert (mp, ml) == (rp, rl), (trial, n_ctx, n_gen, n_min)
        if rl:
            hits += rl > 8
            assert draft.tolist() == search[rp + 1:rp + 1 + k].tolist()
        else:
            assert len(draft) == 0
    assert hits > 20      # matches longer than any n-gram window did occur


def test_longest_suffix_reduces_to_the_ngram_matcher_when_capped():
    """A cap of n turns longest-suffix retrieval into the n-gram matcher: same winner whenever the
    unbounded match is not longer than n."""
    rng = np.random.default_rng(4)
    for _ in range(200):
        hist = rng.integers(0, 3, int(rng.integers(10, 120))).astype(np.int32)
        ex = len(hist) - 1
        _, p_long, m_long = O.ngram_draft(hist, hist, N_MAX, 1, 4, exclude_from=ex)
        for n in (1, 2, 3, 8):
            _, p_n, m_n = O.ngram_draft(hist, hist, n, 1, 4, exclude_from=ex)
            assert m_n == min(m_long, n)
            if m_long <= n:
                assert p_n == p_long


def test_periodic_text():
    """A history of period 3: the suffix matches itself shifted by one period (overlapping
    occurrences count); the draft continues the period."""
    hist = np.array([1, 2, 3] * 20, dtype=np.int32)
    draft, p, m = O.ngram_draft(hist, hist, N_MAX, 1, 5, exclude_from=len(hist) - 1)
    assert (p, m) == (len(hist) - 4, len(hist) - 3)
    assert draft.tolist() == [1, 2, 3]          # only three tokens follow the match


def test_database_retrieval_rule():
    """Request text and extra database (Sec. 5.1 (3)): the longer suffix match supplies the draft,
    the request's own text on equal length; checked against substring search on both arrays."""
    rng = np.random.default_rng(9)
    seen = {"own": 0, "db": 0, None: 0}
    for trial in range(300):
        V = int(rng.integers(2, 5))
        n_ctx = int(rng.integers(2, 80))
        hist = rng.integers(0, V, n_ctx + int(rng.integers(1, 20))).astype(np.int32)
        db = rng.integers(0, V, int(rng.integers(0, 120))).astype(np.int32)
        if trial % 3 == 0 and len(db) > 30:               # plant the suffix in the database
            L = int(rng.integers(3, 15))
            L = min(L, len(hist))
            p = int(rng.integers(L, len(db) - 5))
            db[p - L:p] = hist[-L:]
        n_min = int(rng.integers(1, 3))
        k = int(rng.integers(1, 9))
        draft, src, mp, ml = O.retrieve_draft(hist[:n_ctx], hist, db, N_MAX, n_min, k)
        p1, l1 = _by_substring_search(bytes(hist[:n_ctx].astype(np.uint8)), bytes(hist.astype(np.uint8)), n_min, n_ctx)
        p2, l2 = (-1, 0)
        if len(db) >= 2:
            p2, l2 = _by_substring_search(bytes(db.astype(np.uint8)), bytes(hist.astype(np.uint8)), n_min, len(db))
        if l2 > l1:
            assert (src, mp, ml) == ("db", p2, l2)
            assert draft.tolist() == db[p2 + 1:p2 + 1 + k].tolist()
        elif l1 > 0:
            assert (src, mp, ml) == ("own", p1, l1)
            assert draft.tolist() == hist[:n_ctx][p1 + 1:p1 + 1 + k].tolist()
        else:
            assert src is None and len(draft) == 0
        seen[src] += 1
    assert seen["own"] > 30 and seen["db"] > 30
    # by hand: equal length -> the request's own text; longer -> the database
    hist = np.array([5, 1, 2, 7, 7, 9, 9, 1, 2], dtype=np.int32)
    ctx = hist[:5]
    d, src, mp, ml = O.retrieve_draft(ctx, hist, np.array([1, 2, 4, 4], dtype=np.int32), 8, 1, 2)
    assert (d.tolist(), src, mp, ml) == ([7, 7], "own", 2, 2)
    d, src, mp, ml = O.retrieve_draft(ctx, hist, np.array([3, 9, 1, 2, 4, 4], dtype=np.int32), 8, 1, 2)
    assert (d.tolist(), src, mp, ml) == ([4, 4], "db", 3, 3)
