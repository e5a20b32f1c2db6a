"""Pins for the oracle's tree-structured drafts and the in-context calibration (Sec. 4.1, Sec. 4.3):
a tree row equals the linear-chain row of its root path bit for bit, tree decoding is lossless,
the calibration structure agrees with sorting / searching done another way, and the paper's
word-level example produces the calibrated draft the paper names.  No CUDA path involved."""
import os

import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import get_config, make_context, make_weights

GOLD = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def mini():
    cfg = get_config("mini_gqa").with_(n_ctx=40, gen=20)
    return cfg, make_weights(cfg), make_context(cfg)


def _random_tree(rng, n_nodes, vocab):
    tokens = [int(rng.integers(0, vocab))]
    parent = [-1]
    for j in range(1, n_nodes + 1):
        parent.append(int(rng.integers(0, j)))
        tokens.append(int(rng.integers(0, vocab)))
    return tokens, parent


def _path(parent, j):
    out = []
    while j > 0:
        out.append(j)
        j = parent[j]
    return [0] + out[::-1]


def test_single_path_tree_is_the_linear_chain_bit_for_bit(mini):
    cfg, w, ctx = mini
    toks = [int(t) for t in ctx[:9]]
    a, b = O.OracleModel(w), O.OracleModel(w)
    a.prefill(ctx, cfg.chunk)
    b.prefill(ctx, cfg.chunk)
    la = a.forward(toks, cfg.n_ctx, logits_from=0)
    lb = b.forward(toks, cfg.n_ctx, logits_from=0, parent=[0] + list(range(0, 8)))
    np.testing.assert_array_equal(la, lb)
    np.testing.assert_array_equal(a.kcache, b.kcache)
    np.testing.assert_array_equal(a.vcache, b.vcache)


def test_every_tree_row_equals_the_chain_of_its_root_path(mini):
    """Row j sees the cache and its own path only, so its logits and its K/V rows must be those of a
    linear verify over the path's tokens: a wrong ancestor set, position or cache slot fails this."""
    cfg, w, ctx = mini
    rng = np.random.default_rng(5)
    for trial in range(3):
        tokens, parent = _random_tree(rng, 12, cfg.vocab)
        m = O.OracleModel(w)
        m.prefill(ctx, cfg.chunk)
        lt = m.forward(tokens, cfg.n_ctx, logits_from=0, parent=[0] + parent[1:])
        kt, vt = m.kv_view("k").copy(), m.kv_view("v").copy()
        for j in range(len(tokens)):
            path = _path(parent, j)
            ref = O.OracleModel(w)
            ref.prefill(ctx, cfg.chunk)
            lc = ref.forward([tokens[i] for i in path], cfg.n_ctx, logits_from=0)
            np.testing.assert_array_equal(lt[j], lc[-1])
            d = len(path) - 1
            np.testing.assert_array_equal(kt[:, :, cfg.n_ctx + j], ref.kv_view("k")[:, :, cfg.n_ctx + d])
            np.testing.assert_array_equal(vt[:, :, cfg.n_ctx + j], ref.kv_view("v")[:, :, cfg.n_ctx + d])


def test_tree_forward_rejects_a_parent_that_is_not_earlier(mini):
    cfg, w, ctx = mini
    m = O.OracleModel(w)
    m.prefill(ctx, cfg.chunk)
    with pytest.raises(ValueError):
        m.forward([1, 2, 3], cfg.n_ctx, parent=[0, 1, 1])
    with pytest.raises(ValueError):
        m.forward([1, 2, 3], cfg.n_ctx, parent=[0, 0, 5])


def test_tree_decoding_is_lossless(mini):
    """Whatever the trees hold, the emitted tokens are those of one-token-at-a-time greedy decoding
    (Sec. 5.1: lossless), and the cache ends up as greedy decoding leaves it."""
    cfg, w, ctx = mini
    g = O.OracleModel(w)
    greedy = O.greedy_decode(g, ctx, cfg.gen, cfg.chunk)
    rng = np.random.default_rng(11)

    def builder(hist):
        i0 = len(hist) - cfg.n_ctx          # index into `greedy` of the token after the pending one
        cont = [greedy[i] if i < cfg.gen else 0 for i in range(i0, i0 + 6)]
        tokens, parent = [hist[-1]], [-1]

        def add(par, tok):
            tokens.append(int(tok))
            parent.append(par)
            return len(tokens) - 1
        # a wrong sibling first, then the true continuation for a random number of steps, with wrong
        # side branches hanging off it and a wrong token behind its end
        add(0, (cont[0] + 1) % cfg.vocab)
        cur, depth = 0, int(rng.integers(0, 5))
        for d in range(depth):
            nxt = add(cur, cont[d])
            add(cur, (cont[d] + 2) % cfg.vocab)
            cur = nxt
        add(cur, (cont[depth] + 3) % cfg.vocab)
        return tokens, parent

    m = O.OracleModel(w)
    toks, steps, _ = O.spec_decode_tree(m, ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min, 3, 24,
                                        tree_builder=builder)
    assert toks == greedy
    assert max(len(s["path"]) for s in steps) >= 3 and min(len(s["path"]) for s in steps) == 0
    L = cfg.n_ctx + cfg.gen - 1              # rows of the context and of every emitted token but the last
    np.testing.assert_array_equal(m.kv_view("k")[:, :, :L], g.kv_view("k")[:, :, :L])
    np.testing.assert_array_equal(m.kv_view("v")[:, :, :L], g.kv_view("v")[:, :, :L])
    # and with the calibrated trees themselves
    m2 = O.OracleModel(w)
    toks2, steps2, (succ, occ) = O.spec_decode_tree(m2, ctx, cfg.gen, cfg.chunk, cfg.k, cfg.ngram_n, cfg.ngram_min, 3, 24)
    assert toks2 == greedy
    assert any(len(s["tokens"]) > 1 for s in steps2)


def test_top_successors_and_occurrences():
    rng = np.random.default_rng(3)
    for _ in range(50):
        v = int(rng.integers(4, 60))
        row = rng.standard_normal(v).astype(np.float32)
        if rng.random() < 0.4:
            row[rng.integers(0, v, size=3)] = row.max()        # ties
        b = int(rng.integers(1, 5))
        want = sorted(range(v), key=lambda i: (-row[i], i))[:b]
        assert O.top_successors(row, b) == want
    n, v, b = 30, 12, 3
    ctx = rng.integers(0, v, size=n)
    logits = rng.standard_normal((n, v)).astype(np.float32)
    succ, occ = O.calibrate(ctx, logits, b)
    rev = ctx[::-1].tolist()
    for p in range(n):
        assert succ[p].tolist() == sorted(range(v), key=lambda i: (-logits[p, i], i))[:b]
        for i in range(b):
            t = int(succ[p, i])
            assert int(occ[p, i]) == (n - 1 - rev.index(t) if t in rev else -1)


def test_draft_tree_construction_by_hand():
    # context 5 6 7 5 8; T = 5 occurs last at position 3; its successors 8, 6, 9; 8 occurs at 4, 6 at 1, 9 nowhere
    ctx = [5, 6, 7, 5, 8]
    succ = np.array([[1, 1], [7, 2], [0, 0], [8, 6], [3, 7]], dtype=np.int32)
    succ3 = np.array([[1, 1, 1], [7, 2, 4], [0, 0, 0], [8, 6, 9], [3, 7, 2]], dtype=np.int32)
    occ3 = np.array([[-1] * 3, [2, -1, -1], [-1] * 3, [4, 1, -1], [-1, 2, -1]], dtype=np.int32)
    tokens, parent = O.build_draft_tree(5, [8, 3], ctx, succ3, occ3, max_nodes=31)
    # chain 8 -> 3 first; successor 8 is the chain's first node: reused, its children 3 (already there), 7, 2 added;
    # then 6 with children 7, 2, 4; then 9 (a leaf: it does not occur in the context)
    assert tokens == [5, 8, 3, 7, 2, 6, 7, 2, 4, 9]
    assert parent == [-1, 0, 1, 1, 1, 0, 5, 5, 5, 0]
    # a budget cuts the tail off and never splits the parent order
    t2, p2 = O.build_draft_tree(5, [8, 3], ctx, succ3, occ3, max_nodes=5)
    assert t2 == tokens[:6] and p2 == parent[:6]
    # a committed token that is not in the context gets the chain only
    t3, p3 = O.build_draft_tree(4, [8, 3], ctx, succ3, occ3, max_nodes=31)
    assert t3 == [4, 8, 3] and p3 == [-1, 0, 1]
    assert all(p3[c] < c for c in range(1, len(p3)))


def test_tree_accept_walk():
    tokens, parent = [5, 8, 3, 7, 2, 6], [-1, 0, 1, 1, 1, 0]
    # prediction at the root 8 -> node 1; at node 1: 7 -> node 3; at node 3: 9 -> no child
    assert O.tree_accept(tokens, parent, [8, 7, 0, 9, 0, 0]) == [1, 3]
    assert O.tree_accept(tokens, parent, [6, 0, 0, 0, 0, 1]) == [5]
    assert O.tree_accept(tokens, parent, [1, 7, 0, 9, 0, 0]) == []
    # on a single path the walk is the accepted-prefix rule
    rng = np.random.default_rng(9)
    for _ in range(200):
        n = int(rng.integers(1, 10))
        x = rng.integers(0, 3, size=n).tolist()
        y = rng.integers(0, 3, size=n + 1).tolist()
        path = O.tree_accept([99] + x, [-1] + list(range(n)), y)
        assert path == list(range(1, O.accept_len(x, y) + 1))
    # two children with the same token: the lower-numbered one
    assert O.tree_accept([5, 8, 8], [-1, 0, 0], [8, 1, 2]) == [1]


def test_paper_calibration_example_yields_the_calibrated_draft():
    """Sec. 4.3: for "Clinton" the calibrated draft is "Clinton arrived at", which the model accepts."""
    fields = {}
    with open(os.path.join(GOLD, "paper_sec4_3_calibration_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or ":" not in line:
                continue
            key, val = line.split(":", 1)
            fields[key.strip()] = val.split()
    vocab = {}
    tid = lambda w: vocab.setdefault(w, len(vocab))
    request = [tid(wd) for wd in fields["request"]]
    prefs = {tid("Clinton"): [tid(wd) for wd in fields["after_Clinton"]],
             tid("arrived"): [tid(wd) for wd in fields["after_arrived"]]}
    model = [tid(wd) for wd in fields["model"]]
    V = len(vocab) + 1
    # prefill logits: the stated preferences where the paper gives them, a flat row with the next request
    # word on top elsewhere
    logits = np.zeros((len(request), V), dtype=np.float32)
    for p, t in enumerate(request):
        if t in prefs:
            for rank, s in enumerate(prefs[t]):
                logits[p, s] = 3.0 - rank
        elif p + 1 < len(request):
            logits[p, request[p + 1]] = 1.0
    succ, occ = O.calibrate(request, logits, 3)
    T = tid("Clinton")
    tokens, parent = O.build_draft_tree(T, [], request, succ, occ, max_nodes=31)
    inv = {v: k for k, v in vocab.items()}
    # the table-driven model follows its own continuation after "Clinton"
    nxt = {T: model[0]}
    for a, b in zip(model, model[1:]):
        nxt[a] = b
    y = [nxt.get(t, V - 1) for t in tokens]
    path = O.tree_accept(tokens, parent, y)
    assert [inv[tokens[c]] for c in path] == fields["calibrated_draft"]
    assert len(path) == int(fields["accepted_drafts"][0])
    # the tree holds the three sampled successors of "Clinton" and, below "arrived", its own three
    assert [inv[tokens[c]] for c in range(1, len(tokens)) if parent[c] == 0] == fields["after_Clinton"]
    arrived = [c for c in range(1, len(tokens)) if parent[c] == 0 and inv[tokens[c]] == "arrived"][0]
    assert [inv[tokens[c]] for c in range(1, len(tokens)) if parent[c] == arrived] == fields["after_arrived"]
