"""ctypes binding of libsdv.so.  Method names follow the C entry points (include/sdv.h)."""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

from .build import LIB_PATH, build

OK, EINVAL, ENOMEM, ECAPACITY, ESTATE, ECUDA, ETIMEOUT, ETOOBIG = 0, -1, -2, -3, -4, -5, -6, -7
K_MAX = 31

EXPORTS = [
    "sdv_workspace_bytes", "sdv_create", "sdv_load_weights", "sdv_prefill_chunk", "sdv_draft", "sdv_verify",
    "sdv_commit", "sdv_set_database", "sdv_extend_draft", "sdv_extension_update", "sdv_debug_set_draft", "sdv_rollback", "sdv_kv_len", "sdv_set_parity_mode", "sdv_get_logits", "sdv_destroy",
    "sdv_strerror", "sdv_last_cuda_error", "sdv_step_bytes", "sdv_debug_set_history", "sdv_debug_accept",
    "sdv_debug_force_commit", "sdv_debug_read_kv", "sdv_debug_read_hidden", "sdv_debug_gemm",
    "sdv_debug_timeout_probe", "sdv_debug_profile", "sdv_launch_count", "sdv_last_verify_ms",
    "sdv_gemm_noalloc", "sdv_debug_layout_check", "sdv_debug_plan",
    "sdv_set_calibration", "sdv_get_calibration", "sdv_draft_tree", "sdv_verify_tree", "sdv_debug_force_commit_tree",
    "sdv_debug_top_successors",
    "sdv_follower_workspace_bytes", "sdv_create_follower", "sdv_verify_batch", "sdv_get_verified",
    "sdv_decode_steps", "sdv_run_kernel_ms", "sdv_step",
]


class SdvConfig(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                       "vocab", "max_seq", "k_max", "tied_lm_head", "qkv_bias", "ngram_n",
                                       "ngram_min", "search_history")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class _LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2",
                                          "bq", "bk", "bv")]


class _Weights(C.Structure):
    _fields_ = [("emb", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("layers", C.POINTER(_LayerWeights))]


class SdvError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        self.code = code
        msg = lib().sdv_strerror(code).decode() if _lib is not None else str(code)
        super().__init__(f"{where}: {msg} ({code})" + (f", CUDA error {cuda}" if cuda else ""))


_lib = None


def load_library(path: Optional[str] = None):
    """Loads (building it first if the sources are newer) the CUDA library.  Fails loudly."""
    global _lib
    if _lib is not None:
        return _lib
    path = path or build()
    L = C.CDLL(path)
    vp, ip, i32p = C.c_void_p, C.POINTER(C.c_int), C.c_void_p
    L.sdv_workspace_bytes.argtypes = [C.POINTER(SdvConfig)]
    L.sdv_workspace_bytes.restype = C.c_size_t
    L.sdv_create.argtypes = [C.POINTER(SdvConfig), vp, C.c_size_t, vp, C.POINTER(vp)]
    L.sdv_load_weights.argtypes = [vp, C.POINTER(_Weights)]
    L.sdv_prefill_chunk.argtypes = [vp, i32p, C.c_int, C.c_int]
    L.sdv_draft.argtypes = [vp, C.c_int, i32p, ip]
    L.sdv_verify.argtypes = [vp, i32p, C.c_int, i32p, ip]
    L.sdv_commit.argtypes = [vp, C.c_int, i32p, ip, ip]
    L.sdv_set_database.argtypes = [vp, i32p, C.c_int]
    L.sdv_extend_draft.argtypes = [vp, C.c_int, i32p, ip]
    L.sdv_extension_update.argtypes = [vp, C.c_int, i32p, ip, ip]
    L.sdv_debug_set_draft.argtypes = [vp, i32p, C.c_int]
    L.sdv_rollback.argtypes = [vp, C.c_int]
    L.sdv_kv_len.argtypes = [vp]
    L.sdv_set_parity_mode.argtypes = [vp, C.c_int]
    L.sdv_get_logits.argtypes = [vp, vp, C.c_int]
    L.sdv_destroy.argtypes = [vp]
    L.sdv_follower_workspace_bytes.argtypes = [C.POINTER(SdvConfig)]
    L.sdv_follower_workspace_bytes.restype = C.c_size_t
    L.sdv_create_follower.argtypes = [vp, vp, C.c_size_t, C.POINTER(vp)]
    L.sdv_verify_batch.argtypes = [C.POINTER(vp), C.c_int, ip]
    L.sdv_get_verified.argtypes = [vp, i32p, ip]
    L.sdv_decode_steps.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, i32p, ip, ip]
    L.sdv_run_kernel_ms.argtypes = [vp, vp, C.c_int]
    L.sdv_step.argtypes = [vp, i32p, C.c_int, C.c_int, i32p, ip, i32p, ip, ip]
    L.sdv_strerror.argtypes = [C.c_int]
    L.sdv_strerror.restype = C.c_char_p
    L.sdv_last_cuda_error.argtypes = [vp]
    L.sdv_step_bytes.argtypes = [vp, C.c_int, C.c_int, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    L.sdv_debug_set_history.argtypes = [vp, i32p, C.c_int, C.c_int]
    L.sdv_debug_accept.argtypes = [vp, i32p, C.c_int, i32p, ip]
    L.sdv_debug_force_commit.argtypes = [vp, C.c_int, C.c_int]
    L.sdv_debug_read_kv.argtypes = [vp, C.c_int, C.c_int, C.c_int, C.c_int, vp]
    L.sdv_debug_read_hidden.argtypes = [vp, C.c_int, vp]
    L.sdv_debug_gemm.argtypes = [vp, vp, vp, vp, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_float)]
    L.sdv_debug_timeout_probe.argtypes = [vp]
    L.sdv_debug_profile.argtypes = [vp, C.c_int, vp, C.c_int]
    L.sdv_launch_count.argtypes = [vp]
    L.sdv_launch_count.restype = C.c_longlong
    L.sdv_last_verify_ms.argtypes = [vp, C.POINTER(C.c_float)]
    L.sdv_gemm_noalloc.argtypes = [vp, vp, vp, C.c_int, C.c_int, C.c_int, vp]
    L.sdv_debug_layout_check.argtypes = [C.POINTER(C.c_int), C.POINTER(C.c_int), C.c_int]
    L.sdv_debug_plan.argtypes = [C.POINTER(SdvConfig), C.c_int, C.c_int, C.POINTER(C.c_int)]
    L.sdv_set_calibration.argtypes = [vp, C.c_int]
    L.sdv_get_calibration.argtypes = [vp, vp, vp, C.c_int]
    L.sdv_draft_tree.argtypes = [vp, C.c_int, C.c_int, i32p, i32p, ip]
    L.sdv_verify_tree.argtypes = [vp, i32p, i32p, C.c_int, i32p, i32p, ip]
    L.sdv_debug_force_commit_tree.argtypes = [vp, i32p, C.c_int, C.c_int]
    L.sdv_debug_top_successors.argtypes = [vp, vp, C.c_int, C.c_int, vp]
    for name in EXPORTS:
        if name not in ("sdv_workspace_bytes", "sdv_follower_workspace_bytes", "sdv_strerror", "sdv_launch_count"):
            getattr(L, name).restype = C.c_int
    _lib = L
    return L


def lib():
    return load_library()


def config_from(cfg, k_max: Optional[int] = None, max_seq: Optional[int] = None,
                search_history: bool = False) -> SdvConfig:
    """Builds the C configuration from an object with the ModelConfig field names."""
    return SdvConfig(cfg.n_layers, cfg.d_model, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.d_ffn, cfg.vocab,
                     int(max_seq or cfg.max_seq), int(k_max or cfg.k), int(cfg.tied_lm_head), int(cfg.qkv_bias),
                     cfg.ngram_n, cfg.ngram_min, int(search_history), cfg.rope_theta, cfg.rms_eps)


def _ptr(a):
    if a is None:
        return None
    if isinstance(a, np.ndarray):
        return a.ctypes.data
    return a.data_ptr()  # torch tensor


class Sdv:
    """One sequence on the current CUDA device.  Owns the torch workspace tensor."""

    def __init__(self, cconfig: SdvConfig, stream=None, leader: Optional["Sdv"] = None):
        """leader: another Sdv whose weights this sequence reads (it then needs no load_weights and can
        join the leader in verify_batch); the leader must stay open while its followers are in use."""
        import torch
        if not torch.cuda.is_available():
            raise SdvError(ECUDA, "Sdv: no CUDA device (there is no CPU fallback)")
        L = lib()
        self.cfg = cconfig
        self._leader = leader
        nbytes = L.sdv_workspace_bytes(C.byref(cconfig)) if leader is None else L.sdv_follower_workspace_bytes(C.byref(cconfig))
        if nbytes == 0:
            raise SdvError(EINVAL, "sdv_workspace_bytes")
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self._stream = stream
        sp = None if stream is None else stream.cuda_stream
        h = C.c_void_p()
        self._h = None
        if leader is None:
            self._check(L.sdv_create(C.byref(cconfig), base, nbytes, sp, C.byref(h)), "sdv_create", ctx=None)
        else:
            self._check(L.sdv_create_follower(leader._h, base, nbytes, C.byref(h)), "sdv_create_follower", ctx=None)
        self._h = h
        self.workspace_bytes = nbytes

    def follower(self) -> "Sdv":
        """A further sequence on this one's weights (same configuration and stream)."""
        return Sdv(self.cfg, stream=self._stream, leader=self)

    # -- helpers
    def _check(self, rc: int, where: str, ctx="self"):
        if rc != OK:
            cuda = lib().sdv_last_cuda_error(self._h) if (ctx and self._h) else 0
            raise SdvError(rc, where, cuda)

    def close(self):
        if self._h is not None:
            lib().sdv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the calls
    def load_weights(self, weights):
        """weights: an object with the ModelWeights field names (numpy arrays or CUDA tensors)."""
        n = len(weights.layers)
        arr = (_LayerWeights * n)()
        for i, lw in enumerate(weights.layers):
            for name in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "norm1", "norm2", "bq", "bk", "bv"):
                setattr(arr[i], name, _ptr(getattr(lw, name)))
        w = _Weights(_ptr(weights.emb), _ptr(weights.lm_head), _ptr(weights.final_norm), arr)
        self._check(lib().sdv_load_weights(self._h, C.byref(w)), "sdv_load_weights")

    def prefill_chunk(self, tokens, is_last: bool):
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        self._check(lib().sdv_prefill_chunk(self._h, t.ctypes.data, len(t), int(is_last)), "sdv_prefill_chunk")

    def draft(self, k: int, fetch: bool = True) -> Optional[List[int]]:
        if not fetch:
            self._check(lib().sdv_draft(self._h, k, None, None), "sdv_draft")
            return None
        out = np.zeros(K_MAX, dtype=np.int32)
        dl = C.c_int(0)
        self._check(lib().sdv_draft(self._h, k, out.ctypes.data, C.byref(dl)), "sdv_draft")
        return out[:dl.value].tolist()

    def verify(self, draft: Optional[Sequence[int]] = None, fetch: bool = True) -> Optional[Tuple[List[int], int]]:
        """draft=None verifies the device draft left by draft(); returns (y, accept_len) when fetch."""
        d = None if draft is None else np.ascontiguousarray(draft, dtype=np.int32)
        dp = None if d is None else (d.ctypes.data if len(d) else np.zeros(1, np.int32).ctypes.data)
        dl = 0 if d is None else len(d)
        if not fetch:
            self._check(lib().sdv_verify(self._h, dp, dl, None, None), "sdv_verify")
            return None
        y = np.zeros(K_MAX + 1, dtype=np.int32)
        a = C.c_int(0)
        self._check(lib().sdv_verify(self._h, dp, dl, y.ctypes.data, C.byref(a)), "sdv_verify")
        return y, a.value

    @staticmethod
    def verify_batch(seqs: Sequence["Sdv"], fetch: bool = True) -> Optional[List[int]]:
        """One verify step over several sequences that share weights (each after its own draft());
        returns their accept lengths when fetch.  Commit each sequence afterwards."""
        hs = (C.c_void_p * len(seqs))(*[q._h for q in seqs])
        a = (C.c_int * len(seqs))()
        seqs[0]._check(lib().sdv_verify_batch(hs, len(seqs), a if fetch else None), "sdv_verify_batch")
        return list(a) if fetch else None

    def step(self, draft: Optional[Sequence[int]], k_next: int) -> Tuple[List[int], List[int], int]:
        """Verify `draft` (None: the device draft), accept, commit and draft k_next tokens for the next step:
        one call, one synchronisation.  Returns (emitted tokens, next draft, KV length)."""
        d = None if draft is None else np.ascontiguousarray(draft, dtype=np.int32)
        dp = None if d is None else (d.ctypes.data if len(d) else np.zeros(1, np.int32).ctypes.data)
        em = np.zeros(K_MAX + 1, dtype=np.int32)
        nd = np.zeros(K_MAX + 1, dtype=np.int32)
        n, ndl, kv = C.c_int(0), C.c_int(0), C.c_int(0)
        self._check(lib().sdv_step(self._h, dp, 0 if d is None else len(d), k_next, em.ctypes.data, C.byref(n),
                                   nd.ctypes.data, C.byref(ndl), C.byref(kv)), "sdv_step")
        return em[:n.value].tolist(), nd[:ndl.value].tolist(), kv.value

    def decode_steps(self, k: int, n_steps: int, max_tokens: int = 0, ext_max_total: int = 0,
                     ext_max_life: int = 0) -> Tuple[List[int], int]:
        """n_steps of draft -> verify -> commit enqueued back to back (one synchronisation at the end);
        returns (emitted tokens, KV length)."""
        rows = (ext_max_total if ext_max_total > 0 else k) + 1
        out = np.zeros(n_steps * rows + 1, dtype=np.int32)
        n, kv = C.c_int(0), C.c_int(0)
        self._check(lib().sdv_decode_steps(self._h, k, n_steps, max_tokens, ext_max_total, ext_max_life, out.ctypes.data,
                                           C.byref(n), C.byref(kv)), "sdv_decode_steps")
        return out[:n.value].tolist(), kv.value

    def run_kernel_ms(self, n: int) -> np.ndarray:
        """Forward-kernel times (ms) of the first n steps of the last decode_steps run."""
        ms = np.zeros(n, dtype=np.float32)
        self._check(lib().sdv_run_kernel_ms(self._h, ms.ctypes.data, n), "sdv_run_kernel_ms")
        return ms

    def get_verified(self) -> Tuple[np.ndarray, int]:
        """(y, accept_len) of the outstanding verify step of this sequence."""
        y = np.zeros(K_MAX + 1, dtype=np.int32)
        a = C.c_int(0)
        self._check(lib().sdv_get_verified(self._h, y.ctypes.data, C.byref(a)), "sdv_get_verified")
        return y, a.value

    def set_database(self, tokens):
        """Extra token database the drafter searches besides the request's own text (empty: none)."""
        t = np.ascontiguousarray(tokens, dtype=np.int32)
        self._check(lib().sdv_set_database(self._h, t.ctypes.data if len(t) else None, len(t)), "sdv_set_database")

    def extend_draft(self, max_total: int, fetch: bool = True) -> Optional[List[int]]:
        """Appends the retained segment of rejected drafts to the device draft (Sec. 4.4)."""
        if not fetch:
            self._check(lib().sdv_extend_draft(self._h, max_total, None, None), "sdv_extend_draft")
            return None
        out = np.zeros(K_MAX, dtype=np.int32)
        dl = C.c_int(0)
        self._check(lib().sdv_extend_draft(self._h, max_total, out.ctypes.data, C.byref(dl)), "sdv_extend_draft")
        return out[:dl.value].tolist()

    def extension_update(self, max_life: int, fetch: bool = True) -> Optional[Tuple[List[int], int]]:
        """Eq. 3 on the last verify step; returns (retained segment, lifetime) when fetch."""
        if not fetch:
            self._check(lib().sdv_extension_update(self._h, max_life, None, None, None), "sdv_extension_update")
            return None
        seg = np.zeros(K_MAX, dtype=np.int32)
        n, life = C.c_int(0), C.c_int(0)
        self._check(lib().sdv_extension_update(self._h, max_life, seg.ctypes.data, C.byref(n), C.byref(life)),
                    "sdv_extension_update")
        return seg[:n.value].tolist(), life.value

    # ---- in-context calibration and tree drafts (Sec. 4.3, Sec. 4.1)
    def set_calibration(self, top_b: int):
        self._check(lib().sdv_set_calibration(self._h, int(top_b)), "sdv_set_calibration")
        self._calib_b = int(top_b)

    def get_calibration(self, n_positions: int):
        """(succ, occ) as int32 [n_positions, top_b]."""
        b = max(1, getattr(self, "_calib_b", 0))
        succ = np.zeros((n_positions, b), dtype=np.int32)
        occ = np.zeros((n_positions, b), dtype=np.int32)
        self._check(lib().sdv_get_calibration(self._h, succ.ctypes.data, occ.ctypes.data, n_positions), "sdv_get_calibration")
        return succ, occ

    def draft_tree(self, k: int, max_nodes: int, fetch: bool = True):
        """Returns (tokens, parent) of the draft nodes when fetch: node i+1 continues row parent[i]."""
        if not fetch:
            self._check(lib().sdv_draft_tree(self._h, k, max_nodes, None, None, None), "sdv_draft_tree")
            return None
        tok = np.zeros(K_MAX, dtype=np.int32)
        par = np.zeros(K_MAX, dtype=np.int32)
        n = C.c_int(0)
        self._check(lib().sdv_draft_tree(self._h, k, max_nodes, tok.ctypes.data, par.ctypes.data, C.byref(n)), "sdv_draft_tree")
        return tok[:n.value].tolist(), par[:n.value].tolist()

    def verify_tree(self, tokens: Optional[Sequence[int]] = None, parent: Optional[Sequence[int]] = None, fetch: bool = True):
        """tokens / parent of the draft nodes (None: the device tree); returns (y, accepted path rows) when fetch."""
        t = None if tokens is None else np.ascontiguousarray(tokens, dtype=np.int32)
        p = None if parent is None else np.ascontiguousarray(parent, dtype=np.int32)
        n = 0 if t is None else len(t)
        one = np.zeros(1, np.int32)
        tp = None if t is None else (t.ctypes.data if n else one.ctypes.data)
        pp = None if t is None else (p.ctypes.data if n else one.ctypes.data)
        if not fetch:
            self._check(lib().sdv_verify_tree(self._h, tp, pp, n, None, None, None), "sdv_verify_tree")
            return None
        y = np.zeros(K_MAX + 1, dtype=np.int32)
        path = np.zeros(K_MAX, dtype=np.int32)
        a = C.c_int(0)
        self._check(lib().sdv_verify_tree(self._h, tp, pp, n, y.ctypes.data, path.ctypes.data, C.byref(a)), "sdv_verify_tree")
        return y.tolist(), path[:a.value].tolist()

    def debug_force_commit_tree(self, path: Sequence[int], next_token: int):
        p = np.ascontiguousarray(path, dtype=np.int32)
        self._check(lib().sdv_debug_force_commit_tree(self._h, p.ctypes.data if len(p) else None, len(p), int(next_token)),
                    "sdv_debug_force_commit_tree")

    def debug_top_successors(self, logits: np.ndarray, top_b: int) -> np.ndarray:
        lg = np.ascontiguousarray(logits, dtype=np.float32)
        out = np.zeros((lg.shape[0], top_b), dtype=np.int32)
        self._check(lib().sdv_debug_top_successors(self._h, lg.ctypes.data, lg.shape[0], top_b, out.ctypes.data),
                    "sdv_debug_top_successors")
        return out

    def commit(self, max_emit: int = 0) -> Tuple[List[int], int]:
        out = np.zeros(K_MAX + 1, dtype=np.int32)
        n, kv = C.c_int(0), C.c_int(0)
        self._check(lib().sdv_commit(self._h, max_emit, out.ctypes.data, C.byref(n), C.byref(kv)), "sdv_commit")
        return out[:n.value].tolist(), kv.value

    def rollback(self, new_kv_len: int):
        self._check(lib().sdv_rollback(self._h, new_kv_len), "sdv_rollback")

    def kv_len(self) -> int:
        return lib().sdv_kv_len(self._h)

    def set_parity_mode(self, on: bool):
        self._check(lib().sdv_set_parity_mode(self._h, int(on)), "sdv_set_parity_mode")

    def get_logits(self, rows: int) -> np.ndarray:
        out = np.empty((rows, self.cfg.vocab), dtype=np.float32)
        self._check(lib().sdv_get_logits(self._h, out.ctypes.data, rows), "sdv_get_logits")
        return out

    def step_bytes(self, rows: int, kv_len: int) -> Tuple[float, float]:
        w, k = C.c_double(0), C.c_double(0)
        self._check(lib().sdv_step_bytes(self._h, rows, kv_len, C.byref(w), C.byref(k)), "sdv_step_bytes")
        return w.value, k.value

    def launch_count(self) -> int:
        return int(lib().sdv_launch_count(self._h))

    def last_verify_ms(self) -> float:
        ms = C.c_float(0)
        self._check(lib().sdv_last_verify_ms(self._h, C.byref(ms)), "sdv_last_verify_ms")
        return ms.value

    # -- test / measurement entry points
    def debug_set_history(self, hist, n_ctx: int):
        h = np.ascontiguousarray(hist, dtype=np.int32)
        self._check(lib().sdv_debug_set_history(self._h, h.ctypes.data, len(h), n_ctx), "sdv_debug_set_history")

    def debug_set_draft(self, draft):
        d = np.ascontiguousarray(draft, dtype=np.int32)
        dp = d.ctypes.data if len(d) else None
        self._check(lib().sdv_debug_set_draft(self._h, dp, len(d)), "sdv_debug_set_draft")

    def debug_accept(self, draft, y) -> int:
        """draft=None: the accept scan runs on the draft already on the device (len(y) - 1 tokens)."""
        yy = np.ascontiguousarray(y, dtype=np.int32)
        a = C.c_int(0)
        if draft is None:
            self._check(lib().sdv_debug_accept(self._h, None, len(yy) - 1, yy.ctypes.data, C.byref(a)), "sdv_debug_accept")
            return a.value
        d = np.ascontiguousarray(draft, dtype=np.int32)
        dp = d.ctypes.data if len(d) else None
        self._check(lib().sdv_debug_accept(self._h, dp, len(d), yy.ctypes.data, C.byref(a)), "sdv_debug_accept")
        return a.value

    def debug_force_commit(self, accept_len: int, next_token: int):
        self._check(lib().sdv_debug_force_commit(self._h, accept_len, next_token), "sdv_debug_force_commit")

    def debug_read_kv(self, layer: int, which: int, pos0: int, n: int) -> np.ndarray:
        out = np.empty((self.cfg.n_kv_heads, n, self.cfg.head_dim), dtype=np.float32)
        self._check(lib().sdv_debug_read_kv(self._h, layer, which, pos0, n, out.ctypes.data), "sdv_debug_read_kv")
        return out

    def debug_read_hidden(self, rows: int) -> np.ndarray:
        out = np.empty((rows, self.cfg.d_model), dtype=np.float32)
        self._check(lib().sdv_debug_read_hidden(self._h, rows, out.ctypes.data), "sdv_debug_read_hidden")
        return out

    def debug_gemm(self, x: np.ndarray, w_bits: np.ndarray) -> Tuple[np.ndarray, float]:
        x = np.ascontiguousarray(x, dtype=np.float32)
        w_bits = np.ascontiguousarray(w_bits, dtype=np.uint16)
        M, K = x.shape
        N = w_bits.shape[0]
        y = np.empty((M, N), dtype=np.float32)
        ms = C.c_float(0)
        self._check(lib().sdv_debug_gemm(self._h, x.ctypes.data, w_bits.ctypes.data, y.ctypes.data, M, N, K,
                                         C.byref(ms)), "sdv_debug_gemm")
        return y, ms.value

    def debug_profile(self, on: bool, n_phases: int = 0) -> Optional[np.ndarray]:
        """Switches per-phase timestamps on/off; with n_phases > 0 first returns the last recording
        as uint64 [n_phases, blocks, 12]."""
        L = lib()
        G = L.sdv_debug_profile(self._h, int(on), None, 0)
        if G < 0:
            raise SdvError(G, "sdv_debug_profile")
        if n_phases <= 0:
            return None
        out = np.zeros((n_phases, G, 12), dtype=np.uint64)
        rc = L.sdv_debug_profile(self._h, int(on), out.ctypes.data, n_phases)
        if rc < 0:
            raise SdvError(rc, "sdv_debug_profile")
        return out

    def debug_timeout_probe(self) -> int:
        return lib().sdv_debug_timeout_probe(self._h)


def layout_check(desc: Sequence[int], gu_desc: Sequence[int], n_blocks: int) -> int:
    """Host-only layout self-check (no GPU): returns the library's status code."""
    a = (C.c_int * 8)(*desc)
    b = (C.c_int * 8)(*gu_desc)
    return lib().sdv_debug_layout_check(a, b, n_blocks)


def plan(cconfig: SdvConfig, n_blocks: int, rows: int):
    """Host-only: ([8 ints per operation] x 5, [NG, NB, ring slots, operand bytes, smem bytes, ok])."""
    out = (C.c_int * 48)()
    rc = lib().sdv_debug_plan(C.byref(cconfig), n_blocks, rows, out)
    if rc != OK:
        raise SdvError(rc, "sdv_debug_plan")
    v = list(out)
    return [v[i * 8:(i + 1) * 8] for i in range(5)], v[40:46]


def gemm_noalloc(x, w_bits, y, stream=None) -> int:
    """y[M][N] = x[M][K] * w[N][K]^T on device tensors, through the entry point that allocates no
    memory.  x: CUDA float32 [M][K]; w_bits: CUDA tensor of bf16 values (dtype bfloat16, or their
    bits as int16 / uint16) [N][K]; y: CUDA float32 [M][N], overwritten.  All contiguous and on the
    current device; x and w_bits must start on a 16-byte boundary (a view such as x[1:] of a tensor
    with an odd row length does not: the library then returns EINVAL and runs nothing).  Returns the
    library's status code (OK, EINVAL, ETOOBIG, ...): marshalling only."""
    import torch
    for t in (x, w_bits, y):
        if not (t.is_cuda and t.is_contiguous()):
            raise ValueError("gemm_noalloc takes contiguous CUDA tensors")
    if x.dtype != torch.float32 or y.dtype != torch.float32 or w_bits.element_size() != 2:
        raise ValueError("gemm_noalloc: x and y float32, w 16-bit")
    M, K = x.shape
    N = w_bits.shape[0]
    if tuple(w_bits.shape) != (N, K) or tuple(y.shape) != (M, N):
        raise ValueError("gemm_noalloc: shapes do not agree")
    s = stream if stream is not None else torch.cuda.current_stream()
    return lib().sdv_gemm_noalloc(x.data_ptr(), w_bits.data_ptr(), y.data_ptr(), M, N, K, s.cuda_stream)
