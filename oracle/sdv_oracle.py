"""ctypes front end of the CPU oracle (oracle/sdv_oracle.c) and the decoding loops built on it.

TEST INFRASTRUCTURE ONLY.  Nothing under the product package imports this module, and this
module imports nothing from the product package; both only share the seeded input generators.

The decoding loops restate, step by step, retrieval-based greedy speculative decoding as the
paper states it (Sec. 3.2: draft, verify in parallel, keep drafts up to the first mismatch;
Sec. 4.4: accepted prefix x_1..x_{e-1}, y_e), plus plain one-token-at-a-time greedy decoding,
which the method must reproduce exactly (lossless, Sec. 5.1 "Metrics and Configuration").
"""
from __future__ import annotations

import ctypes as C
import hashlib
import os
import subprocess
from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sdv_oracle.c")


def _host_tag() -> str:
    """The shared object is built with -march=native, so key it by the host CPU."""
    model = ""
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.startswith("flags"):
                    model = line
                    break
    except OSError:
        pass
    with open(_SRC, "rb") as fh:
        src = fh.read()
    return hashlib.sha1(model.encode() + src).hexdigest()[:12]


def build(verbose: bool = False) -> str:
    """Compile the oracle's C source for this host (no-op when up to date); returns the path."""
    out = os.path.join(_HERE, f"liborc_{_host_tag()}.so")
    if not os.path.exists(out):
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fno-fast-math", "-ffp-contract=fast",
               "-shared", "-fPIC", "-o", out + ".tmp", _SRC, "-lm"]
        if verbose:
            print(" ".join(cmd))
        subprocess.run(cmd, check=True)
        os.replace(out + ".tmp", out)
    return out


class _Cfg(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                       "vocab", "max_seq", "tied_lm_head", "qkv_bias")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class _Layer(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2",
                                          "bq", "bk", "bv")]


class _Weights(C.Structure):
    _fields_ = [("emb", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("layers", C.POINTER(_Layer))]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.orc_matmul.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int]
        L.orc_matmul.restype = None
        L.orc_matmul_plain.argtypes = L.orc_matmul.argtypes
        L.orc_matmul_plain.restype = None
        L.orc_rmsnorm.argtypes = [C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_int]
        L.orc_rmsnorm.restype = None
        L.orc_rope.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_float]
        L.orc_rope.restype = None
        L.orc_attention_row.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        L.orc_attention_row.restype = None
        L.orc_swiglu.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int]
        L.orc_swiglu.restype = None
        L.orc_argmax.argtypes = [C.c_void_p, C.c_int]
        L.orc_argmax.restype = C.c_int
        L.orc_forward.argtypes = [C.POINTER(_Cfg), C.POINTER(_Weights), C.c_void_p, C.c_int, C.c_int, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_forward.restype = C.c_int
        L.orc_forward_tree.argtypes = [C.POINTER(_Cfg), C.POINTER(_Weights), C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                       C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_forward_tree.restype = C.c_int
        L.orc_ngram_draft.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int,
                                      C.c_void_p, C.POINTER(C.c_int), C.POINTER(C.c_int)]
        L.orc_ngram_draft.restype = C.c_int
        L.orc_accept_len.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_accept_len.restype = C.c_int
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


# ---------------------------------------------------------------- single operations
def matmul(x, w_bits, bias=None) -> np.ndarray:
    """x [M,K] fp32 times bf16 weights [N,K] (uint16 bit patterns), transposed: returns [M,N]."""
    x = _f32(x)
    w_bits = np.ascontiguousarray(w_bits, dtype=np.uint16)
    M, K = x.shape
    N = w_bits.shape[0]
    assert w_bits.shape[1] == K
    b = None if bias is None else _f32(bias)
    y = np.empty((M, N), dtype=np.float32)
    lib().orc_matmul(_p(x), _p(w_bits), _p(b), _p(y), M, N, K)
    return y


def matmul_plain(x, w_bits, bias=None) -> np.ndarray:
    """The same product by the plain triple loop (the definition; slow)."""
    x = _f32(x)
    w_bits = np.ascontiguousarray(w_bits, dtype=np.uint16)
    M, K = x.shape
    N = w_bits.shape[0]
    assert w_bits.shape[1] == K
    b = None if bias is None else _f32(bias)
    y = np.empty((M, N), dtype=np.float32)
    lib().orc_matmul_plain(_p(x), _p(w_bits), _p(b), _p(y), M, N, K)
    return y


def rmsnorm(x, w, eps) -> np.ndarray:
    x, w = _f32(x), _f32(w)
    y = np.empty_like(x)
    lib().orc_rmsnorm(_p(x), _p(w), float(eps), _p(y), x.shape[0])
    return y


def rope(v, pos: int, theta: float) -> np.ndarray:
    v = _f32(v).copy()
    lib().orc_rope(_p(v), v.shape[0], int(pos), float(theta))
    return v


def attention_row(q, k, v) -> np.ndarray:
    """q [hd], k/v [n_keys, hd] -> softmax(q.k/sqrt(hd)) v."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    n, hd = k.shape
    out = np.empty(hd, dtype=np.float32)
    scr = np.empty(n, dtype=np.float32)
    lib().orc_attention_row(_p(q), _p(k), _p(v), n, hd, _p(out), _p(scr))
    return out


def swiglu(g, u) -> np.ndarray:
    g, u = _f32(g).ravel(), _f32(u).ravel()
    act = np.empty_like(g)
    lib().orc_swiglu(_p(g), _p(u), _p(act), g.shape[0])
    return act


def argmax(x) -> int:
    x = _f32(x)
    return int(lib().orc_argmax(_p(x), x.shape[0]))


def ngram_draft(search, hist, n: int, n_min: int, k: int, exclude_from: Optional[int] = None):
    """Returns (draft int32 array of length draft_len, match_pos, match_len)."""
    search = np.ascontiguousarray(search, dtype=np.int32)
    hist = np.ascontiguousarray(hist, dtype=np.int32)
    out = np.empty(max(k, 1), dtype=np.int32)
    mp, ml = C.c_int(-1), C.c_int(0)
    ex = len(search) if exclude_from is None else int(exclude_from)
    dl = lib().orc_ngram_draft(_p(search), len(search), _p(hist), len(hist), int(n), int(n_min), int(k), ex,
                               _p(out), C.byref(mp), C.byref(ml))
    return out[:dl].copy(), mp.value, ml.value


def retrieve_draft(search, hist, database, n: int, n_min: int, k: int, exclude_from: Optional[int] = None):
    """Drafting from the request's text and an extra token database (Sec. 5.1 (3), Sec. 5.5): both
    arrays are searched with the same suffix matcher; the longer match supplies the draft, the
    request's own text on equal length (the paper names no rule).  Returns (draft, source, match_pos,
    match_len) with source "own", "db" or None."""
    d1, p1, m1 = ngram_draft(search, hist, n, n_min, k, exclude_from)
    if database is None or len(database) < 2:
        return d1, ("own" if m1 else None), p1, m1
    d2, p2, m2 = ngram_draft(database, hist, n, n_min, k)
    if m2 > m1:
        return d2, "db", p2, m2
    return d1, ("own" if m1 else None), p1, m1


def accept_len(x: Sequence[int], y: Sequence[int]) -> int:
    x = np.ascontiguousarray(x, dtype=np.int32)
    y = np.ascontiguousarray(y, dtype=np.int32)
    assert len(y) == len(x) + 1
    return int(lib().orc_accept_len(_p(x), _p(y), len(x)))


# ---------------------------------------------------------------- draft extension (Sec. 4.4)
def reuse_segment(x: Sequence[int], y: Sequence[int], a: int):
    """Eq. 3: among the drafts beyond the reject point, the longest run on which the draft agrees
    with the model's own predictions.

    x = x_1..x_n (x[i] is x_{i+1}), y = y_1..y_{n+1}, a = accept length, so the reject position is
    e = a + 1 (x[a] != y[a]) when a < n.  Every pair (first, last) with a < first <= last < n is
    tried, as the equation states it; the constraint is x_i = y_i on the whole range.  The paper
    names no tie rule: the earliest longest run wins.  Returns (first index into x, length),
    (0, 0) when nothing qualifies (no reject, or no agreement beyond it: the "redundant" pattern
    of Table 2).
    """
    n = len(x)
    assert len(y) == n + 1 and 0 <= a <= n
    best_first, best_len = 0, 0
    for first in range(a + 1, n):
        for last in range(first, n):
            if all(x[i] == y[i] for i in range(first, last + 1)) and last - first + 1 > best_len:
                best_first, best_len = first, last - first + 1
    return best_first, best_len


class DraftExtension:
    """Reuse of rejected drafts (Sec. 4.4 "Reuse strategy"): one retained segment with a lifetime.

    The paper fixes: the segment is the solution of Eq. 3; it is appended to later drafts; it is
    kept for at least one decoding step and dropped when either its age or the length of the
    whole draft passes a limit (32 in Sec. 5.1).  Readings taken where it is silent:
    * lifetime counts the verify steps the segment was appended to;
    * a draft that would grow beyond `max_total` with the segment drops the segment instead of
      cutting it;
    * a segment into which the accepted prefix reached is spent (its leading tokens were emitted;
      what still matches behind the new reject point comes back as a new candidate);
    * a new candidate replaces the retained segment only when strictly longer (length-first), so
      the retained segment found again in its own appended copy does not renew its lifetime.
    """

    def __init__(self, max_total: int = 32, max_life: int = 32):
        self.max_total, self.max_life = int(max_total), int(max_life)
        self.seg: List[int] = []
        self.life = 0
        self.used = False      # the segment is part of the draft under verification
        self.base_len = 0      # length of that draft before the segment was appended

    def extend(self, draft: Sequence[int]) -> List[int]:
        draft = [int(t) for t in draft]
        self.base_len, self.used = len(draft), False
        if self.seg:
            if len(draft) + len(self.seg) <= self.max_total:
                self.used = True
                return draft + list(self.seg)
            self.seg, self.life = [], 0
        return draft

    def update(self, x: Sequence[int], y: Sequence[int], a: int) -> None:
        """After the verify step of draft x (as returned by extend) with predictions y, accept a."""
        if self.used:
            self.life += 1
        if self.seg and ((self.used and a > self.base_len) or self.life > self.max_life):
            self.seg, self.life = [], 0
        first, length = reuse_segment(x, y, a)
        if length > len(self.seg):
            self.seg, self.life = [int(t) for t in x[first:first + length]], 0
        self.used = False


# ---------------------------------------------------------------- in-context calibration and tree drafts (Sec. 4.3, Sec. 4.1)
def top_successors(logits_row, b: int) -> List[int]:
    """"Sample" (Sec. 4.3): the b highest-logit token ids of one prefill position, best first; among equal
    logits the lower id first (the greedy tie rule).  Taken one at a time: the greedy token, then the
    greedy token of what is left."""
    row = np.array(logits_row, dtype=np.float32, copy=True)
    out = []
    for _ in range(min(b, len(row))):
        i = argmax(row)
        out.append(i)
        row[i] = -np.inf
    return out


def calibrate(context: Sequence[int], prefill_logits: np.ndarray, b: int):
    """The calibration structure of Sec. 4.3 for one request.

    succ[p] = top_successors(logits of context position p): with the context token C[p] each of them
    is an anchor <C[p], prediction>.  "Search": occ[p][i] = the position in the context where the
    prediction succ[p][i] occurs (the paper names no rule for several occurrences: the latest one,
    as in the retrieval drafter), -1 where it does not occur; a matched anchor is expanded with
    that position's own successors, which gives the two-level token tree of the text.
    Returns (succ [n, b] int32, occ [n, b] int32)."""
    ctx = [int(t) for t in context]
    n = len(ctx)
    assert prefill_logits.shape[0] == n
    succ = np.zeros((n, b), dtype=np.int32)
    occ = np.full((n, b), -1, dtype=np.int32)
    for p in range(n):
        s = top_successors(prefill_logits[p], b)
        succ[p, :len(s)] = s
        for i, tok in enumerate(s):
            for q in range(n - 1, -1, -1):
                if ctx[q] == tok:
                    occ[p, i] = q
                    break
    return succ, occ


def build_draft_tree(T: int, chain: Sequence[int], context: Sequence[int], succ: np.ndarray, occ: np.ndarray,
                     max_nodes: int):
    """Tree-structured draft for one step (Sec. 4.1, Sec. 4.3).  Node 0 is the committed token T.

    The retrieval drafter's chain x_1..x_m comes first, as one path.  Then the calibrated tree of T:
    with p the latest position of T in the context (none: no calibrated branches), each successor
    succ[p][i] becomes a child of the root, followed at once by its own children succ[q] when the
    anchor was matched at q = occ[p][i] (depth first, two levels, as the text describes).  A token
    that a node already has as a child is not added twice (the existing child is used).  At most
    max_nodes draft nodes; what does not fit is left out.  Returns (tokens, parent) including node 0,
    parent[0] = -1; every parent index is smaller than its child's."""
    tokens, parent = [int(T)], [-1]

    def child_with(node, tok):
        for c in range(1, len(tokens)):
            if parent[c] == node and tokens[c] == tok:
                return c
        return -1

    def add(node, tok):
        c = child_with(node, tok)
        if c >= 0:
            return c
        if len(tokens) - 1 >= max_nodes:
            return -1
        tokens.append(int(tok))
        parent.append(node)
        return len(tokens) - 1

    cur = 0
    for x in chain:
        cur = add(cur, int(x))
        if cur < 0:
            break
    ctx = [int(t) for t in context]
    p = -1
    for q in range(len(ctx) - 1, -1, -1):
        if ctx[q] == int(T):
            p = q
            break
    if p >= 0:
        for i in range(succ.shape[1]):
            c = add(0, int(succ[p, i]))
            q = int(occ[p, i])
            if c >= 0 and q >= 0:
                for i2 in range(succ.shape[1]):
                    add(c, int(succ[q, i2]))
    return tokens, parent


def tree_accept(tokens: Sequence[int], parent: Sequence[int], y: Sequence[int]) -> List[int]:
    """Strict acceptance on a tree: starting at the root, step to the child whose token is the model's
    prediction at the current node (the lowest-numbered one, should several carry it), until no child
    does.  Returns the accepted path (node indices, root excluded).  The emitted tokens are the
    path's tokens followed by the prediction at its last node: on a single path this is the
    accepted-prefix rule x_1..x_{e-1}, y_e of Sec. 4.4."""
    path, cur = [], 0
    while True:
        nxt = -1
        for c in range(1, len(tokens)):
            if parent[c] == cur and tokens[c] == y[cur]:
                nxt = c
                break
        if nxt < 0:
            return path
        path.append(nxt)
        cur = nxt


# ---------------------------------------------------------------- the model
class OracleModel:
    """Holds the weight arrays (bf16 bit patterns from sdv_inputs) and an fp32 KV cache."""

    def __init__(self, weights, max_seq: Optional[int] = None):
        cfg = weights.cfg
        self.cfg = cfg
        self.max_seq = int(max_seq or cfg.max_seq)
        self._keep = weights
        self._c = _Cfg(cfg.n_layers, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn,
                       cfg.vocab, self.max_seq, int(cfg.tied_lm_head), int(cfg.qkv_bias),
                       cfg.rope_theta, cfg.rms_eps)
        arr = (_Layer * cfg.n_layers)()
        for i, lw in enumerate(weights.layers):
            for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2", "bq", "bk", "bv"):
                a = getattr(lw, name)
                if a is not None:
                    assert a.flags["C_CONTIGUOUS"]
                setattr(arr[i], name, None if a is None else a.ctypes.data)
        self._layers = arr
        self._w = _Weights(weights.emb.ctypes.data,
                           None if weights.lm_head is None else weights.lm_head.ctypes.data,
                           weights.final_norm.ctypes.data, arr)
        n = cfg.n_layers * cfg.n_kv_heads * self.max_seq * cfg.head_dim
        self.kcache = np.zeros(n, dtype=np.float32)
        self.vcache = np.zeros(n, dtype=np.float32)
        self.kv_len = 0

    def kv_view(self, which: str) -> np.ndarray:
        c = self.cfg
        a = self.kcache if which == "k" else self.vcache
        return a.reshape(c.n_layers, c.n_kv_heads, self.max_seq, c.head_dim)

    def forward(self, tokens, start_pos: int, logits_from: Optional[int] = 0, want_hidden: bool = False,
                parent: Optional[Sequence[int]] = None):
        """Runs the decoder over `tokens` at positions start_pos.. and writes their KV rows.

        parent (tree-structured drafts, Sec. 4.1): row j continues row parent[j] < j (parent[0] is
        ignored); row j is at position start_pos + depth(j), its KV rows go to cache slot
        start_pos + j, and it attends to the cache and to its own path from the root.

        Returns logits [m - logits_from, V] (None when logits_from is None), and the final
        residual stream [m, d] when want_hidden.
        """
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        m = len(tokens)
        par = None
        if parent is not None:
            par = np.ascontiguousarray(parent, dtype=np.int32)
            assert len(par) == m
        logits = None
        lf = m
        if logits_from is not None:
            lf = int(logits_from)
            logits = np.empty((m - lf, self.cfg.vocab), dtype=np.float32)
        hid = np.empty((m, self.cfg.d_model), dtype=np.float32) if want_hidden else None
        if par is None:
            rc = lib().orc_forward(C.byref(self._c), C.byref(self._w), _p(tokens), m, int(start_pos), _p(self.kcache),
                                   _p(self.vcache), _p(logits), lf, _p(hid))
        else:
            rc = lib().orc_forward_tree(C.byref(self._c), C.byref(self._w), _p(tokens), _p(par), m, int(start_pos),
                                        _p(self.kcache), _p(self.vcache), _p(logits), lf, _p(hid))
        if rc != 0:
            raise ValueError("orc_forward: bad argument")
        return (logits, hid) if want_hidden else logits

    def prefill(self, context, chunk: int) -> np.ndarray:
        """Chunked prefill (Sec. 4.1): returns the logits of the last context position."""
        context = np.ascontiguousarray(context, dtype=np.int32)
        n = len(context)
        last = None
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            if e == n:
                last = self.forward(context[s:e], s, logits_from=e - s - 1)[0]
            else:
                self.forward(context[s:e], s, logits_from=None)
        self.kv_len = n
        return last

    def prefill_all_logits(self, context, chunk: int) -> np.ndarray:
        """Chunked prefill that keeps the logits of every context position, [n, V] (what the
        calibration of Sec. 4.3 starts from)."""
        context = np.ascontiguousarray(context, dtype=np.int32)
        n = len(context)
        rows = []
        for s in range(0, n, chunk):
            e = min(n, s + chunk)
            rows.append(self.forward(context[s:e], s, logits_from=0))
        self.kv_len = n
        return np.concatenate(rows, axis=0)

    def move_kv_rows(self, src: Sequence[int], dst: Sequence[int]) -> None:
        """Copies cache rows src[i] -> dst[i] (all layers and KV heads), in the order given."""
        for which in ("k", "v"):
            a = self.kv_view(which)
            for s_, d_ in zip(src, dst):
                if s_ != d_:
                    a[:, :, d_, :] = a[:, :, s_, :]


# ---------------------------------------------------------------- decoding loops
@dataclass
class StepRecord:
    kv_len_before: int
    pending: int               # T: the committed token whose KV row is not yet in the cache
    draft: List[int]           # x_1..x_dl
    y: List[int]               # y_1..y_{dl+1}
    accept: int                # a: leading drafts equal to the model's predictions
    emitted: List[int]         # x_1..x_a, y_{a+1} (cut to the generation budget on the last step)
    kv_len_after: int
    logits: Optional[np.ndarray] = None   # [dl+1, V] when kept
    margin: List[float] = field(default_factory=list)  # top-1 minus top-2 logit per row


def top2(row: np.ndarray):
    """The greedy choice of a logits row, the token that would replace it, and the gap between them.

    Returns (best id, runner-up id, margin): best = the greedy token (largest value, lowest id among
    equals); runner-up = the greedy token of the row with `best` removed; margin = their difference
    (0.0 on an exact tie).  The parity tolerance forgives a flipped token only where this margin is
    small, and then only towards this runner-up.
    """
    row = np.asarray(row)
    best = argmax(row)
    rest = np.array(row, dtype=np.float32, copy=True)
    rest[best] = -np.inf
    second = argmax(rest)
    return best, second, float(row[best] - row[second])


def top2_margin(row: np.ndarray) -> float:
    return top2(row)[2]


def greedy_decode(model: OracleModel, context, gen: int, chunk: int):
    """One token at a time: T_{i+1} = argmax logits(all previous tokens).  Returns the gen tokens."""
    last = model.prefill(context, chunk)
    out = [argmax(last)]
    L = len(context)
    while len(out) < gen:
        lg = model.forward([out[-1]], L, logits_from=0)[0]
        L += 1
        out.append(argmax(lg))
    model.kv_len = L
    return out


def spec_decode(model: OracleModel, context, gen: int, chunk: int, k: int, ngram_n: int, ngram_min: int,
                drafter=None, search_history: bool = False, keep_logits: bool = False,
                extension: Optional[DraftExtension] = None):
    """Retrieval-based greedy speculative decoding.

    `drafter(history, k) -> list` overrides the n-gram drafter (tests use it to force drafts).
    `extension` appends the retained segment of earlier rejected drafts to every draft (Sec. 4.4).
    The first generated token comes from prefill; each step then verifies [T, x_1..x_dl] at
    positions L..L+dl, accepts a drafts, emits x_1..x_a, y_{a+1} and sets L += a+1.
    Returns (tokens, steps).
    """
    context = np.ascontiguousarray(context, dtype=np.int32)
    last = model.prefill(context, chunk)
    hist = list(int(t) for t in context)
    T = argmax(last)
    hist.append(T)
    out = [T]
    L = len(context)
    steps: List[StepRecord] = []
    while len(out) < gen:
        if drafter is not None:
            draft = [int(t) for t in drafter(hist, k)][:k]
        elif search_history:
            draft = ngram_draft(hist, hist, ngram_n, ngram_min, k, exclude_from=len(hist) - 1)[0].tolist()
        else:
            draft = ngram_draft(context, hist, ngram_n, ngram_min, k)[0].tolist()
        if extension is not None:
            draft = extension.extend(draft)
        dl = len(draft)
        logits = model.forward([T] + draft, L, logits_from=0)
        y = [argmax(logits[j]) for j in range(dl + 1)]
        a = accept_len(draft, y)
        if extension is not None:
            extension.update(draft, y, a)
        emitted = draft[:a] + [y[a]]
        room = gen - len(out)
        emitted = emitted[:room]
        rec = StepRecord(L, T, draft, y, a, emitted, L + len(emitted),
                         logits.copy() if keep_logits else None,
                         [top2_margin(logits[j]) for j in range(dl + 1)])
        steps.append(rec)
        L += len(emitted)
        out.extend(emitted)
        hist.extend(emitted)
        T = emitted[-1]
    model.kv_len = L
    return out, steps


def spec_decode_tree(model: OracleModel, context, gen: int, chunk: int, k: int, ngram_n: int, ngram_min: int,
                     calib_top: int, max_nodes: int, tree_builder=None, keep_logits: bool = False):
    """Greedy speculative decoding with tree-structured drafts: the retrieval chain plus the branches
    of the calibrated token tree (Sec. 4.3), verified in one pass; the accepted path's KV rows are
    moved to consecutive cache slots.  `tree_builder(history) -> (tokens, parent)` overrides the
    draft construction (tests force trees with it).  Returns (tokens, steps, (succ, occ)); a step
    is a dict with the tree, the predictions, the accepted path and the emitted tokens."""
    context = np.ascontiguousarray(context, dtype=np.int32)
    logits_all = model.prefill_all_logits(context, chunk)
    succ, occ = calibrate(context, logits_all, calib_top)
    hist = [int(t) for t in context]
    T = argmax(logits_all[-1])
    hist.append(T)
    out = [T]
    L = len(context)
    steps = []
    while len(out) < gen:
        if tree_builder is not None:
            tokens, parent = tree_builder(hist)
        else:
            chain = ngram_draft(context, hist, ngram_n, ngram_min, k)[0].tolist()
            tokens, parent = build_draft_tree(T, chain, context, succ, occ, max_nodes)
        assert tokens[0] == T
        logits = model.forward(tokens, L, logits_from=0, parent=[0] + list(parent[1:]))
        y = [argmax(logits[j]) for j in range(len(tokens))]
        path = tree_accept(tokens, parent, y)
        emitted = [tokens[c] for c in path] + [y[path[-1] if path else 0]]
        emitted = emitted[:gen - len(out)]
        keep = path[:len(emitted) - 1] if len(emitted) <= len(path) else path
        model.move_kv_rows([L + c for c in keep], [L + 1 + i for i in range(len(keep))])
        steps.append(dict(kv_len_before=L, pending=T, tokens=list(tokens), parent=list(parent), y=y, path=list(path),
                          emitted=list(emitted), logits=logits.copy() if keep_logits else None,
                          margin=[top2_margin(logits[j]) for j in range(len(tokens))]))
        L += len(emitted)
        out.extend(emitted)
        hist.extend(emitted)
        T = emitted[-1]
    model.kv_len = L
    return out, steps, (succ, occ)
