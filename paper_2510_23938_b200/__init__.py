"""GPU-resident integrity verification of model-weight bytes on B200 (sm_100a).

Chunked SHA-256 digests, a binary Merkle root and manifest verification, computed by
hand-written CUDA kernels behind the C ABI declared in ``include/iv.h``.  This package is
the thin Python binding (``binding``), the in-tree build (``build``) and the synthetic
input generators used by the tests and the benchmark (``inputs``).
"""
from .binding import (Context, IvError, Manifest, VerifyResult, load_library, n_chunks,  # noqa: F401
                      new_result, read_result, read_results)
