"""GPU parity of tree-structured drafts and the in-context calibration (Sec. 4.1, Sec. 4.3) against the
oracle: integer parts bit-exact, logits within the stated tolerance, all through the C-ABI."""
import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import get_config, make_context, make_weights
from paper_2510_15312_b200.binding import Sdv, SdvError, config_from, EINVAL, ESTATE
from helpers import COS_TOL, LOGIT_TOL, MARGIN_TOL

pytestmark = pytest.mark.gpu


def gpu_prefill(s, ctx, chunk):
    n = len(ctx)
    for i in range(0, n, chunk):
        s.prefill_chunk(ctx[i:i + chunk], is_last=(i + chunk >= n))


def _forced_tree_builder(cfg, greedy, rng):
    """Trees around the true greedy continuation: wrong siblings, side branches, a wrong tail, so that
    paths of every length up to 5 get accepted and rows off the path are exercised."""
    def builder(hist):
        i0 = len(hist) - cfg.n_ctx
        cont = [greedy[i] if i < cfg.gen else 0 for i in range(i0, i0 + 6)]
        tokens, parent = [hist[-1]], [-1]

        def add(par, tok):
            tokens.append(int(tok))
            parent.append(par)
            return len(tokens) - 1
        add(0, (cont[0] + 1) % cfg.vocab)
        cur, depth = 0, int(rng.integers(0, 6))
        for d in range(depth):
            nxt = add(cur, cont[d])
            add(cur, (cont[d] + 2) % cfg.vocab)
            if d % 2:
                add(nxt, (cont[d + 1] + 5) % cfg.vocab)
            cur = nxt
        add(cur, (cont[depth] + 3) % cfg.vocab)
        return tokens, parent
    return builder


@pytest.mark.parametrize("name", ["tiny", "mini_gqa", "mini_hd128"])
def test_tree_verify_teacher_forced_against_the_oracle(name):
    cfg = get_config(name)
    w, ctx = make_weights(cfg), make_context(cfg)
    greedy = O.greedy_decode(O.OracleModel(w), ctx, cfg.gen, cfg.chunk)
    ref = O.OracleModel(w)
    toks, steps, _ = O.spec_decode_tree(ref, ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min, 3, 24,
                                        tree_builder=_forced_tree_builder(cfg, greedy, np.random.default_rng(21)),
                                        keep_logits=True)
    assert toks == greedy
    s = Sdv(config_from(cfg, k_max=24))
    s.load_weights(w)
    s.set_parity_mode(True)
    gpu_prefill(s, ctx, cfg.chunk)
    s.debug_set_history(list(ctx) + [toks[0]], cfg.n_ctx)
    max_err, flips, lens = 0.0, 0, set()
    for st in steps:
        assert s.kv_len() == st["kv_len_before"]
        tokens, parent = st["tokens"], st["parent"]
        y, path = s.verify_tree(tokens[1:], parent[1:])
        logits = s.get_logits(len(tokens))
        first_bad = None
        for r in range(len(tokens)):
            err = float(np.abs(logits[r] - st["logits"][r]).max())
            cos = float(np.dot(logits[r], st["logits"][r]) / (np.linalg.norm(logits[r]) * np.linalg.norm(st["logits"][r])))
            max_err = max(max_err, err)
            assert err <= LOGIT_TOL and cos >= COS_TOL, (name, st["kv_len_before"], r, err, cos)
            if y[r] != st["y"][r]:
                assert st["margin"][r] < MARGIN_TOL and y[r] == O.top2(st["logits"][r])[1]
                flips += 1
                if first_bad is None and (r == 0 or r in st["path"]):
                    first_bad = r
        if first_bad is None:
            assert path == st["path"], (name, st["kv_len_before"])
        lens.add(len(st["path"]))
        # teacher forcing: the oracle's path and next token
        nxt = st["emitted"][-1]
        keep = st["path"][:len(st["emitted"]) - 1]
        s.debug_force_commit_tree(keep, nxt)
        assert s.kv_len() == st["kv_len_before"] + len(st["emitted"])
    assert len(lens) >= 3
    # the cache after all the moves: the rows of the emitted tokens sit where plain decoding puts them
    g = O.OracleModel(w)
    O.greedy_decode(g, ctx, cfg.gen, cfg.chunk)
    L = cfg.n_ctx + cfg.gen - 1
    for layer in (0, cfg.n_layers - 1):
        for which, nm in ((0, "k"), (1, "v")):
            got = s.debug_read_kv(layer, which, cfg.n_ctx, L - cfg.n_ctx)
            want = g.kv_view(nm)[layer][:, cfg.n_ctx:L]
            assert np.abs(got - want).max() <= 0.02 * np.abs(want).max() + 1e-3, (layer, nm)
    print(name, "tree max |dlogit|", max_err, "near-tie flips", flips)
    s.close()


def test_single_path_tree_equals_chain_verify_on_the_gpu():
    cfg = get_config("mini_gqa")
    w, ctx = make_weights(cfg), make_context(cfg)
    s = Sdv(config_from(cfg, k_max=16))
    s.load_weights(w)
    s.set_parity_mode(True)
    gpu_prefill(s, ctx, cfg.chunk)
    L0 = s.kv_len()
    draft = [int(t) for t in ctx[10:18]]
    y1, a1 = s.verify(draft)
    l1 = s.get_logits(9)
    s.rollback(L0)
    y2, path = s.verify_tree(draft, list(range(8)))
    l2 = s.get_logits(9)
    # same rows, same positions, same masks: only the order of the fp32 atomic adds differs between the two
    # launches (low-order bits, now and then one bf16 rounding further down)
    assert np.abs(l1 - l2).max() <= 1e-2
    clear = all(O.top2_margin(l1[r]) > 0.03 for r in range(9))
    if clear:
        assert [int(t) for t in y1[:9]] == [int(t) for t in y2[:9]] and path == list(range(1, a1 + 1))
    s.close()


def test_top_successor_kernel_bit_exact():
    cfg = get_config("tiny")
    s = Sdv(config_from(cfg))
    rng = np.random.default_rng(8)
    for trial in range(6):
        rows = int(rng.integers(1, 25))
        lg = rng.standard_normal((rows, cfg.vocab)).astype(np.float32)
        if trial % 2:
            for r in range(rows):        # exact ties, also at the top
                lg[r, rng.integers(0, cfg.vocab, size=5)] = lg[r].max()
        b = int(rng.integers(1, 5))
        got = s.debug_top_successors(lg, b)
        want = np.array([O.top_successors(lg[r], b) for r in range(rows)], dtype=np.int32)
        np.testing.assert_array_equal(got, want)
    s.close()


@pytest.mark.parametrize("name", ["tiny", "mini_gqa"])
def test_calibration_tables_and_tree_drafts_against_the_oracle(name):
    cfg = get_config(name)
    w, ctx = make_weights(cfg), make_context(cfg)
    B = 3
    ref = O.OracleModel(w)
    logits_all = ref.prefill_all_logits(ctx, cfg.chunk)
    succ_o, occ_o = O.calibrate(ctx, logits_all, B)
    s = Sdv(config_from(cfg, k_max=24))
    s.load_weights(w)
    s.set_calibration(B)
    gpu_prefill(s, ctx, cfg.chunk)
    with pytest.raises(SdvError):
        s.set_calibration(2)             # only before prefill
    succ, occ = s.get_calibration(cfg.n_ctx)
    # "Sample" is decided by floating point: both sides rank their own logits; the device's choice must be one
    # the oracle's logits allow (every pick within the logit tolerance of the oracle's b-th best), and equal
    # wherever the oracle's ranking is clear-cut
    exact = 0
    for p in range(cfg.n_ctx):
        row = logits_all[p]
        srt = np.sort(row)[::-1]
        clear = all(srt[i] - srt[i + 1] > 2 * LOGIT_TOL for i in range(B))
        if clear:
            assert succ[p].tolist() == succ_o[p].tolist(), p
            exact += 1
        else:
            assert all(row[t] >= srt[B - 1] - 2 * LOGIT_TOL for t in succ[p]), p
    assert exact >= cfg.n_ctx // 20      # random-init logits are crowded at the top: clear-cut rows are a minority
    # "Search" is integer work on the device's own table: bit-exact against a host search
    rev = [int(t) for t in ctx[::-1]]
    for p in range(cfg.n_ctx):
        for i in range(B):
            t = int(succ[p, i])
            assert int(occ[p, i]) == (cfg.n_ctx - 1 - rev.index(t) if t in rev else -1)
    # tree drafts: the device builds from its own tables what the oracle's builder builds from the same tables
    T0 = O.argmax(logits_all[-1])
    rng = np.random.default_rng(4)
    for trial in range(40):
        T = int(ctx[rng.integers(0, cfg.n_ctx)]) if trial % 4 else int(rng.integers(0, cfg.vocab))
        tail = [int(t) for t in ctx[rng.integers(0, cfg.n_ctx - 4):][:2]] if trial % 3 else []
        hist = [int(t) for t in ctx] + tail + [T]
        s.debug_set_history(hist, cfg.n_ctx)
        k = [0, 4, cfg.k][trial % 3]
        max_nodes = [24, 5, 9][trial % 3]
        chain = O.ngram_draft(ctx, hist, cfg.ngram_n, cfg.ngram_min, k)[0].tolist() if k else []
        want_t, want_p = O.build_draft_tree(T, chain, ctx, succ, occ, max_nodes)
        got_t, got_p = s.draft_tree(k, max_nodes)
        assert got_t == want_t[1:] and got_p == want_p[1:], trial
    s.close()


def test_tree_decoding_loop_on_the_device_is_lossless_until_a_near_tie():
    """draft_tree -> verify_tree -> commit, nothing forced: the emitted stream equals the oracle's greedy
    stream up to the first position whose top-2 margin is inside the tolerance."""
    cfg = get_config("mini_gqa")
    w, ctx = make_weights(cfg), make_context(cfg)
    g = O.OracleModel(w)
    last = g.prefill(ctx, cfg.chunk)
    g2 = O.OracleModel(w)
    toks, steps = O.spec_decode(g2, ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min)
    margins = [O.top2_margin(last)]
    for st in steps:
        margins.extend(st.margin[:len(st.emitted)])
    s = Sdv(config_from(cfg, k_max=24))
    s.load_weights(w)
    s.set_calibration(3)
    gpu_prefill(s, ctx, cfg.chunk)
    out, accepted = [], 0
    while len(out) < cfg.gen - 1:
        s.draft_tree(cfg.k, 24, fetch=False)
        y, path = s.verify_tree()
        accepted += len(path)
        emitted, kv = s.commit(max_emit=cfg.gen - 1 - len(out))
        out.extend(emitted)
        assert kv == cfg.n_ctx + len(out)
    first_tie = next((i for i, m in enumerate(margins) if m < MARGIN_TOL), len(margins))
    n = min(first_tie, len(out) + 1)
    assert ([toks[0]] + out)[:n] == toks[:n]
    print("tree loop: accepted draft nodes", accepted, "matched tokens", n)
    s.close()


def test_tree_call_order_and_argument_errors():
    cfg = get_config("tiny")
    w, ctx = make_weights(cfg), make_context(cfg)
    s = Sdv(config_from(cfg, k_max=8))
    s.load_weights(w)
    with pytest.raises(SdvError) as e:
        s.verify_tree([1], [0])
    assert e.value.code == ESTATE
    gpu_prefill(s, ctx, cfg.chunk)
    with pytest.raises(SdvError) as e:
        s.verify_tree([1, 2], [0, 2])        # node 2 cannot continue itself
    assert e.value.code == EINVAL
    with pytest.raises(SdvError) as e:
        s.verify_tree()                      # no device tree pending
    assert e.value.code == ESTATE
    with pytest.raises(SdvError) as e:
        s.get_calibration(4)                 # calibration was never switched on
    assert e.value.code == ESTATE
    s.close()
