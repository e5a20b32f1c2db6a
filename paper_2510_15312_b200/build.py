"""Builds the CUDA library in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsdv.so")
_SOURCES = ["sdv.cu", "forward.cuh", "dense.cuh", "layout.cuh", "ptx.cuh", "small_kernels.cuh"]


HASH_PATH = LIB_PATH + ".srchash"


def _source_hash() -> str:
    """Digest of every source the library is built from (file times do not survive a checkout or a copy)."""
    import hashlib
    h = hashlib.sha256()
    deps = [os.path.join(_HERE, "csrc", s) for s in _SOURCES]
    deps.append(os.path.join(os.path.dirname(_HERE), "include", "sdv.h"))
    for d in deps:
        with open(d, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def _stale() -> bool:
    if not os.path.exists(LIB_PATH) or not os.path.exists(HASH_PATH):
        return True
    with open(HASH_PATH) as fh:
        return fh.read().strip() != _source_hash()


def build(force: bool = False, verbose: bool = False) -> str:
    if not force and not _stale():
        return LIB_PATH
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-std=c++17", "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo",
           "-shared", "-Xcompiler", "-fPIC", "-o", LIB_PATH + ".tmp", os.path.join(_HERE, "csrc", "sdv.cu")]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
        print(" ".join(cmd))
    subprocess.run(cmd, check=True)
    os.replace(LIB_PATH + ".tmp", LIB_PATH)
    with open(HASH_PATH, "w") as fh:
        fh.write(_source_hash())
    return LIB_PATH


if __name__ == "__main__":
    print(build(force=True, verbose=True))
