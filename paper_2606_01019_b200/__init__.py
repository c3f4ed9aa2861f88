"""B200 (sm_100a) library for the per-step path of Hybrid Verified Decoding.

The package is a thin ctypes binding of ``libhvd_b200.so`` (built in-tree from ``csrc/`` by
``build.py``).  Every step of the path runs in the library's CUDA kernels; there is no CPU or
PyTorch fallback: importing works without a GPU (so the build can be checked), creating a context
does not.
"""
from .binding import (BF16, F32, FREQ_MAX_OCC, NOALLOC_MAX_BATCH, NOALLOC_MAX_ROWS, REQ_BAD_LEN, REQ_CAPACITY, REQ_OK,
                      STATE_DTYPE, Context, HvdError, exported_symbols, hvd_verify_commit_noalloc,
                      library_path, load_library)

__all__ = ["Context", "HvdError", "F32", "BF16", "REQ_OK", "REQ_CAPACITY", "REQ_BAD_LEN",
           "STATE_DTYPE", "exported_symbols", "library_path", "load_library", "hvd_verify_commit_noalloc",
           "NOALLOC_MAX_ROWS", "NOALLOC_MAX_BATCH", "FREQ_MAX_OCC"]
