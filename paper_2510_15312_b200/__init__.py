"""sdv: the verify path of retrieval-based greedy speculative decoding on one B200.

Python binding of the C-ABI library declared in include/sdv.h: argument marshalling only,
every step of the path runs in the library's CUDA kernels.  PyTorch is used for device memory
and streams.  There is no CPU fallback: importing works without a GPU, creating a context
does not.
"""
from .binding import (SdvError, Sdv, SdvConfig, lib, load_library, EXPORTS, OK, EINVAL, ENOMEM, ECAPACITY,
                      ESTATE, ECUDA, ETIMEOUT, ETOOBIG, gemm_noalloc)

__all__ = ["SdvError", "Sdv", "SdvConfig", "lib", "load_library", "EXPORTS", "OK", "EINVAL", "ENOMEM",
           "ECAPACITY", "ESTATE", "ECUDA", "ETIMEOUT", "ETOOBIG", "gemm_noalloc"]
