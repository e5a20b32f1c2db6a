"""GPU tests of the single kernels through the C-ABI: the weight-streaming GEMM, the n-gram
drafter, the accept scan / commit, and the error paths.  Oracle = oracle/sdv_oracle."""
import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import bf16_bits_to_f32, f32_to_bf16_bits, get_config, make_weights
import paper_2510_15312_b200 as pkg
from paper_2510_15312_b200.binding import Sdv, config_from

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx_tiny():
    s = Sdv(config_from(get_config("tiny"), k_max=16, max_seq=4096))
    yield s
    s.close()


@pytest.mark.parametrize("M,N,K", [(1, 16, 64), (9, 256, 256), (17, 1024, 256), (9, 768, 1024), (8, 2000 + 16, 320 - 64),
                                   (32, 4096, 256), (24, 144, 1024), (16, 16 * 149, 64 * 5), (3, 16 * 300, 64 * 7)])
def test_gemm_matches_oracle_matmul(ctx_tiny, M, N, K):
    rng = np.random.default_rng(M * 1000 + N + K)
    x = rng.standard_normal((M, K)).astype(np.float32)
    wb = f32_to_bf16_bits(rng.standard_normal((N, K)).astype(np.float32))
    ref = O.matmul(bf16_bits_to_f32(f32_to_bf16_bits(x)), wb)      # the kernel rounds x to bf16 on the way in
    y, ms = ctx_tiny.debug_gemm(x, wb)
    # both sides use exact bf16 products; only the fp32 summation order differs
    np.testing.assert_allclose(y, ref, rtol=0, atol=2e-5 * np.sqrt(K))
    assert ms > 0


def test_gemm_rejects_bad_shapes(ctx_tiny):
    x = np.zeros((4, 64), np.float32)
    w = np.zeros((24, 64), np.uint16)        # N not a multiple of 16
    with pytest.raises(pkg.SdvError) as e:
        ctx_tiny.debug_gemm(x, w)
    assert e.value.code == pkg.EINVAL
    with pytest.raises(pkg.SdvError):
        ctx_tiny.debug_gemm(np.zeros((33, 64), np.float32), np.zeros((16, 64), np.uint16))   # too many rows
    with pytest.raises(pkg.SdvError):
        ctx_tiny.debug_gemm(np.zeros((4, 96), np.float32), np.zeros((16, 96), np.uint16))    # K not a multiple of 64


def _draft_case(s, search_history, hist, n_ctx, k):
    s.debug_set_history(hist, n_ctx)
    return s.draft(k)


@pytest.mark.parametrize("search_history", [False, True])
def test_drafter_bit_exact_on_random_arrays(search_history):
    cfg = get_config("tiny").with_(ngram_n=3, ngram_min=1)
    rng = np.random.default_rng(11 + search_history)
    for n, n_min in ((3, 1), (4, 2), (1, 1), (8, 3)):
        s = Sdv(config_from(cfg.with_(ngram_n=n, ngram_min=n_min), k_max=16, max_seq=9000,
                            search_history=search_history))
        for trial in range(250):
            V = int(rng.integers(2, 7))
            n_ctx = int(rng.integers(1, 60)) if trial % 5 else int(rng.integers(1500, 8200))
            n_gen = int(rng.integers(1, 12))
            hist = rng.integers(0, V, n_ctx + n_gen).astype(np.int32)
            if trial % 7 == 0 and n_ctx > 40:       # plant the suffix so that long matches exist
                p = int(rng.integers(n + 1, n_ctx - 20))
                hist[p - n:p] = hist[-n:]
            k = int(rng.integers(1, 17))
            got = _draft_case(s, search_history, hist, n_ctx, k)
            if search_history:
                ref = O.ngram_draft(hist, hist, n, n_min, k, exclude_from=len(hist) - 1)[0].tolist()
            else:
                ref = O.ngram_draft(hist[:n_ctx], hist, n, n_min, k)[0].tolist()
            assert got == ref, (trial, n, n_min, k, n_ctx, n_gen)
        s.close()


@pytest.mark.parametrize("search_history", [False, True])
def test_longest_suffix_drafter_bit_exact(search_history):
    """Suffix length up to 4096 (longest-suffix retrieval): planted repeats of 5..3000 tokens,
    contexts up to 8200, and the degenerate constant and periodic texts (longest compare loops)."""
    cfg = get_config("tiny").with_(ngram_n=4096, ngram_min=2)
    s = Sdv(config_from(cfg, k_max=16, max_seq=9000, search_history=search_history))
    rng = np.random.default_rng(31 + search_history)
    longest = 0
    cases = []
    for trial in range(120):
        V = int(rng.integers(2, 50))
        n_ctx = int(rng.integers(10, 200)) if trial % 3 else int(rng.integers(3500, 8200))
        n_gen = int(rng.integers(1, 400)) if n_ctx > 3000 else int(rng.integers(1, 30))
        hist = rng.integers(0, V, n_ctx + n_gen).astype(np.int32)
        if n_ctx > 3000:
            L = int(rng.integers(5, 3000))
            p = int(rng.integers(L, n_ctx - 20))
            hist[p - L:p] = hist[-L:]
        cases.append((hist, n_ctx))
    cases.append((np.full(8000, 7, dtype=np.int32), 7000))                 # constant text
    cases.append((np.array([1, 2, 3, 4, 5] * 1600, dtype=np.int32), 6000))   # periodic text
    for hist, n_ctx in cases:
        k = int(rng.integers(1, 17))
        got = _draft_case(s, search_history, hist, n_ctx, k)
        if search_history:
            ref, _, ml = O.ngram_draft(hist, hist, 4096, 2, k, exclude_from=len(hist) - 1)
        else:
            ref, _, ml = O.ngram_draft(hist[:n_ctx], hist, 4096, 2, k)
        assert got == ref.tolist(), (len(hist), n_ctx, k, ml)
        longest = max(longest, ml)
    assert longest == 4096
    s.close()


def test_drafter_with_extra_database_bit_exact():
    """The drafter over the request's text and an extra token database against the oracle's rule."""
    cfg = get_config("tiny").with_(ngram_n=64, ngram_min=1)
    s = Sdv(config_from(cfg, k_max=16, max_seq=9000))
    rng = np.random.default_rng(77)
    from_db = 0
    for trial in range(200):
        V = int(rng.integers(2, 8))
        n_ctx = int(rng.integers(2, 300))
        hist = rng.integers(0, V, n_ctx + int(rng.integers(1, 30))).astype(np.int32)
        db = rng.integers(0, V, int(rng.integers(0, 6000)) if trial % 4 else int(rng.integers(0, 3))).astype(np.int32)
        if trial % 3 == 0 and len(db) > 100:
            L = min(int(rng.integers(3, 40)), len(hist))
            p = int(rng.integers(L, len(db) - 20))
            db[p - L:p] = hist[-L:]
        k = int(rng.integers(1, 17))
        s.set_database(db)
        got = _draft_case(s, False, hist, n_ctx, k)
        ref, src, _, _ = O.retrieve_draft(hist[:n_ctx], hist, db, 64, 1, k)
        assert got == ref.tolist(), (trial, len(db), n_ctx, k, src)
        from_db += src == "db"
    assert from_db > 20
    s.set_database([])                                      # removed: back to the request's text alone
    hist = np.array([5, 1, 2, 7, 7, 9, 9, 1, 2], dtype=np.int32)
    s.set_database([3, 9, 1, 2, 4, 4])
    assert _draft_case(s, False, hist, 5, 2) == [4, 4]      # the longer match is in the database
    s.set_database([1, 2, 4, 4])
    assert _draft_case(s, False, hist, 5, 2) == [7, 7]      # equal length: the request's own text
    s.set_database([])
    assert _draft_case(s, False, hist, 5, 2) == [7, 7]
    with pytest.raises(pkg.SdvError):
        s.set_database([cfg.vocab])                         # token out of range
    s.close()


def test_drafter_edge_cases(ctx_tiny):
    s = ctx_tiny
    assert _draft_case(s, False, [1, 2, 3, 9, 3], 3, 4) == []           # only match ends at the last context token
    assert _draft_case(s, False, [3, 2, 3, 9, 3], 3, 4) == [2, 3]
    assert _draft_case(s, False, [1, 2, 3, 4], 3, 4) == []              # nothing matches
    assert _draft_case(s, False, [5, 6, 7, 8, 5, 6, 9, 9, 5, 6, 7, 1, 5, 6], 11, 4) == [7]   # latest of equal matches
    assert _draft_case(s, False, [5, 6, 7, 8, 5, 6, 9, 9, 5, 6, 5, 6, 7], 10, 3) == [8, 5, 6]  # longest wins
    assert _draft_case(s, False, [1, 2, 3, 4, 2], 4, 2) == [3, 4]       # continuation cut at the context's end
    assert _draft_case(s, False, [7], 0, 4) == []                       # empty context


def test_accept_scan_and_commit(ctx_tiny):
    s = ctx_tiny
    rng = np.random.default_rng(5)
    hist = rng.integers(0, 50, 40).astype(np.int32)
    for trial in range(300):
        s.debug_set_history(hist, 30)
        dl = int(rng.integers(0, 17))
        x = rng.integers(0, 4096, dl)
        y = rng.integers(0, 4096, dl + 1)
        e = int(rng.integers(0, dl + 2))            # first e drafts agree
        y[:min(e, dl)] = x[:min(e, dl)]
        a = s.debug_accept(x, y)
        assert a == O.accept_len(x, y)
        max_emit = int(rng.integers(0, 4))
        emitted, kv = s.commit(max_emit)
        ref = list(x[:a]) + [int(y[a])]
        if max_emit > 0:
            ref = ref[:max_emit]
        assert emitted == [int(t) for t in ref]
        assert kv == 39 + len(ref) == s.kv_len()
        # the drafter now sees the committed tokens at the end of the history
        s.rollback(39)
        assert s.kv_len() == 39


def test_call_order_and_capacity_errors():
    cfg = get_config("tiny")
    s = Sdv(config_from(cfg, max_seq=64))
    L = pkg.lib()
    assert L.sdv_verify(s._h, None, 0, None, None) == pkg.ESTATE           # before prefill
    assert L.sdv_draft(s._h, 4, None, None) == pkg.ESTATE
    assert L.sdv_commit(s._h, 0, None, None, None) == pkg.ESTATE
    toks = np.zeros(80, np.int32)
    assert L.sdv_prefill_chunk(s._h, toks.ctypes.data, 8, 0) == pkg.ESTATE  # weights not loaded yet
    s.debug_set_history(np.arange(20, dtype=np.int32), 20)
    assert L.sdv_verify(s._h, None, 0, None, None) == pkg.ESTATE           # still no weights
    s.load_weights(make_weights(cfg))
    assert L.sdv_draft(s._h, 5, None, None) == pkg.EINVAL                   # k > k_max
    assert L.sdv_verify(s._h, toks.ctypes.data, 5, None, None) == pkg.EINVAL
    bad = np.array([4096], np.int32)
    assert L.sdv_verify(s._h, bad.ctypes.data, 1, None, None) == pkg.EINVAL  # token id out of range
    assert L.sdv_rollback(s._h, 25) == pkg.EINVAL
    assert L.sdv_debug_set_history(s._h, toks.ctypes.data, 80, 10) == pkg.ECAPACITY
    s.debug_set_history(np.arange(63, dtype=np.int32), 20)
    assert L.sdv_verify(s._h, toks.ctypes.data, 4, None, None) == pkg.ECAPACITY   # 62 + 5 rows > 64
    s.close()


def test_bounded_wait_reports_timeout_and_context_survives(ctx_tiny):
    assert ctx_tiny.debug_timeout_probe() == pkg.ETIMEOUT
    # the context is still usable afterwards
    assert _draft_case(ctx_tiny, False, [3, 2, 3, 9, 3], 3, 4) == [2, 3]
