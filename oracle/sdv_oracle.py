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

    def forward(self, tokens, start_pos: int, logits_from: Optional[int] = 0, want_hidden: bool = False):
        """Runs the decoder over `tokens` at positions start_pos.. and writes their KV rows.

        Returns logits [m - logits_from, V] (None when logits_from is None), and the final
        residual stream [m, d] when want_hidden.
        """
        tokens = np.ascontiguousarray(tokens, dtype=np.int32)
        m = len(tokens)
        logits = None
        lf = m
        if logits_from is not None:
            lf = int(logits_from)
            logits = np.empty((m - lf, self.cfg.vocab), dtype=np.float32)
        hid = np.empty((m, self.cfg.d_model), dtype=np.float32) if want_hidden else None
        rc = lib().orc_forward(C.byref(self._c), C.byref(self._w), _p(tokens), m, int(start_pos), _p(self.kcache),
                               _p(self.vcache), _p(logits), lf, _p(hid))
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
