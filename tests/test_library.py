"""The C-ABI library: it builds, loads and exports every entry point include/sdv.h declares.
No compute call is made here (no GPU needed)."""
import ctypes
import os
import re

import pytest

import paper_2510_15312_b200 as pkg
from paper_2510_15312_b200.binding import SdvConfig

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_header_and_binding_list_the_same_entry_points():
    with open(os.path.join(ROOT, "include", "sdv.h")) as fh:
        text = fh.read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(sdv_[a-z_]+)\s*\(", text))
    assert declared == set(pkg.EXPORTS)


def test_library_exports_every_declared_symbol():
    L = pkg.load_library()
    for name in pkg.EXPORTS:
        assert isinstance(getattr(L, name), ctypes._CFuncPtr)


def test_host_side_argument_checks():
    L = pkg.load_library()
    good = SdvConfig(2, 256, 4, 4, 64, 1024, 4096, 600, 4, 0, 0, 3, 1, 0, 1e4, 1e-6)
    assert L.sdv_workspace_bytes(ctypes.byref(good)) > 0
    for field, bad in (("head_dim", 96), ("d_model", 250), ("vocab", 4097), ("k_max", 32), ("n_kv_heads", 3),
                       ("ngram_min", 4), ("ngram_n", 4097), ("max_seq", 3), ("d_ffn", 1000)):
        c = SdvConfig.from_buffer_copy(good)
        setattr(c, field, bad)
        assert L.sdv_workspace_bytes(ctypes.byref(c)) == 0, field
    # 8 query heads per KV head with 17 rows: the attention step cuts the heads into groups, so this fits
    c = SdvConfig(2, 512, 8, 1, 64, 1024, 4096, 600, 16, 0, 0, 3, 1, 0, 1e4, 1e-6)
    assert L.sdv_workspace_bytes(ctypes.byref(c)) > 0
    c.n_q_heads = 16  # more than 8 query heads per KV head is not supported
    assert L.sdv_workspace_bytes(ctypes.byref(c)) == 0
    assert L.sdv_strerror(pkg.ETIMEOUT).decode().startswith("a bounded")
    assert L.sdv_strerror(-99) == b"unknown error"
    # NULL context: an error code, never a crash
    assert L.sdv_kv_len(None) == pkg.EINVAL
    assert L.sdv_commit(None, 0, None, None, None) == pkg.EINVAL
    out = ctypes.c_void_p()
    assert L.sdv_create(ctypes.byref(good), None, 0, None, ctypes.byref(out)) == pkg.EINVAL


def test_no_cpu_fallback_without_gpu():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    from paper_2510_15312_b200.binding import Sdv
    good = SdvConfig(2, 256, 4, 4, 64, 1024, 4096, 600, 4, 0, 0, 3, 1, 0, 1e4, 1e-6)
    with pytest.raises(pkg.SdvError):
        Sdv(good)
