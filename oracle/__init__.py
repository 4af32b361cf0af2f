"""ctypes front end of the plain CPU oracle (``iv_oracle.c``).

Test infrastructure only: the tests, the smoke check and the benchmark's
CPU-baseline leg call it; the CUDA library and its Python binding never do, and
nothing here imports them.  The shared object is compiled with gcc next to the
source (``build()``); loading compiles it first when it is missing or older
than the source.

All functions take and return ``bytes`` / ``numpy`` arrays on the host.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "iv_oracle.c")
_HDR = os.path.join(_HERE, "iv_oracle.h")
_LIB = os.path.join(_HERE, "libiv_oracle.so")

_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc; returns the path of the shared object."""
    newest_src = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest_src:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.run(
            ["gcc", "-O2", "-std=c11", "-Wall", "-Wextra", "-fPIC", "-shared", "-pthread",
             "-o", tmp, _SRC],
            check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is not None:
            return _lib
        lib = ctypes.CDLL(build())
        u8p = ctypes.POINTER(ctypes.c_uint8)
        u32p = ctypes.POINTER(ctypes.c_uint32)
        u64p = ctypes.POINTER(ctypes.c_uint64)
        lib.ivo_constants.argtypes = [u32p, u32p]
        lib.ivo_constants.restype = None
        lib.ivo_sha256.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_sha256.restype = None
        lib.ivo_hash_chunks.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                        ctypes.c_void_p, ctypes.c_int]
        lib.ivo_hash_chunks.restype = ctypes.c_uint64
        lib.ivo_merkle_root.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_merkle_root.restype = None
        lib.ivo_merkle_root_recursive.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_merkle_root_recursive.restype = None
        lib.ivo_verify.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                   ctypes.c_void_p, ctypes.c_void_p, u64p, ctypes.c_uint64,
                                   ctypes.POINTER(ctypes.c_int), u8p, ctypes.c_int]
        lib.ivo_verify.restype = ctypes.c_uint64
        lib.ivo_hash_ragged.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                        ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int]
        lib.ivo_hash_ragged.restype = None
        u64p_ = ctypes.POINTER(ctypes.c_uint64)
        lib.ivo_constants512.argtypes = [u64p_, u64p_]
        lib.ivo_constants512.restype = None
        lib.ivo_sha384.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_sha384.restype = None
        lib.ivo_hash_chunks_sha384.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                               ctypes.c_void_p, ctypes.c_int]
        lib.ivo_hash_chunks_sha384.restype = ctypes.c_uint64
        lib.ivo_merkle_root_sha384.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_merkle_root_sha384.restype = None
        lib.ivo_h0_sha512.argtypes = [u64p_]
        lib.ivo_h0_sha512.restype = None
        lib.ivo_sha512.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_sha512.restype = None
        lib.ivo_hash_chunks_sha512.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                               ctypes.c_void_p, ctypes.c_int]
        lib.ivo_hash_chunks_sha512.restype = ctypes.c_uint64
        lib.ivo_merkle_root_sha512.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_merkle_root_sha512.restype = None
        lib.ivo_hash_chunks_rfc6962.argtypes = [ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint64,
                                                ctypes.c_void_p, ctypes.c_int]
        lib.ivo_hash_chunks_rfc6962.restype = ctypes.c_uint64
        lib.ivo_merkle_root_rfc6962.argtypes = [ctypes.c_void_p, ctypes.c_uint64, u8p]
        lib.ivo_merkle_root_rfc6962.restype = None
        _lib = lib
        return lib


def host_threads() -> int:
    """Number of host cores the threaded entry points use by default."""
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:  # pragma: no cover
        return max(1, os.cpu_count() or 1)


def _as_u8(buf) -> np.ndarray:
    """View any bytes-like / array as a contiguous 1-D uint8 array (no copy if possible)."""
    if isinstance(buf, np.ndarray):
        arr = np.ascontiguousarray(buf).view(np.uint8).reshape(-1)
    else:
        arr = np.frombuffer(buf, dtype=np.uint8)
    return arr


def _ptr(arr: np.ndarray):
    return ctypes.c_void_p(arr.ctypes.data if arr.size else 0)


def constants():
    """(K[64], H0[8]) as numpy uint32 arrays, derived from the primes."""
    k = np.zeros(64, dtype=np.uint32)
    h0 = np.zeros(8, dtype=np.uint32)
    _load().ivo_constants(k.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)),
                          h0.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)))
    return k, h0


def sha256(msg) -> bytes:
    arr = _as_u8(msg)
    out = (ctypes.c_uint8 * 32)()
    _load().ivo_sha256(_ptr(arr), arr.size, out)
    return bytes(out)


def n_chunks(nbytes: int, chunk_bytes: int) -> int:
    return 0 if nbytes == 0 else -(-nbytes // chunk_bytes)


def hash_chunks(data, chunk_bytes: int, nthreads: int = 1) -> np.ndarray:
    """Chunk digests as an (n, 32) uint8 array."""
    arr = _as_u8(data)
    if chunk_bytes <= 0:
        raise ValueError("chunk_bytes must be positive")
    n = n_chunks(arr.size, chunk_bytes)
    out = np.zeros((n, 32), dtype=np.uint8)
    got = _load().ivo_hash_chunks(_ptr(arr), arr.size, chunk_bytes, _ptr(out), nthreads)
    assert got == n
    return out


def merkle_root(leaves, recursive: bool = False) -> bytes:
    arr = _as_u8(leaves)
    assert arr.size % 32 == 0
    out = (ctypes.c_uint8 * 32)()
    fn = _load().ivo_merkle_root_recursive if recursive else _load().ivo_merkle_root
    fn(_ptr(arr), arr.size // 32, out)
    return bytes(out)


def verify(data, chunk_bytes: int, manifest_digests, manifest_root: bytes,
           idx_cap: int | None = None, nthreads: int = 1):
    """Returns (root_ok: bool, n_mismatch: int, idx: list[int] ascending, root: bytes)."""
    arr = _as_u8(data)
    man = _as_u8(manifest_digests)
    n = n_chunks(arr.size, chunk_bytes)
    assert man.size == 32 * n, "manifest digest count does not match the data"
    assert len(manifest_root) == 32
    cap = n if idx_cap is None else idx_cap
    idx = np.zeros(max(cap, 1), dtype=np.uint64)
    root_ok = ctypes.c_int(0)
    root = (ctypes.c_uint8 * 32)()
    mroot = np.frombuffer(manifest_root, dtype=np.uint8)
    bad = _load().ivo_verify(_ptr(arr), arr.size, chunk_bytes, _ptr(man), _ptr(mroot),
                             idx.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)), cap,
                             ctypes.byref(root_ok), root, nthreads)
    return bool(root_ok.value), int(bad), [int(v) for v in idx[:min(bad, cap)]], bytes(root)


def hash_ragged(base, offsets, lengths, nthreads: int = 1) -> np.ndarray:
    """Per-tensor digests as an (n, 32) uint8 array."""
    arr = _as_u8(base)
    off = np.ascontiguousarray(offsets, dtype=np.uint64)
    ln = np.ascontiguousarray(lengths, dtype=np.uint64)
    assert off.shape == ln.shape and off.ndim == 1
    if off.size:
        assert int((off + ln).max()) <= arr.size, "a tensor reaches past the base buffer"
    out = np.zeros((off.size, 32), dtype=np.uint8)
    _load().ivo_hash_ragged(_ptr(arr), _ptr(off), _ptr(ln), off.size, _ptr(out), nthreads)
    return out


# ---------------------------------------------------------------------------------------------
# SHA-384 variant

def constants512():
    """(K[80], H0 of SHA-384 [8]) as numpy uint64 arrays, derived from the primes."""
    k = np.zeros(80, dtype=np.uint64)
    h0 = np.zeros(8, dtype=np.uint64)
    p64 = ctypes.POINTER(ctypes.c_uint64)
    _load().ivo_constants512(k.ctypes.data_as(p64), h0.ctypes.data_as(p64))
    return k, h0


def sha384(msg) -> bytes:
    arr = _as_u8(msg)
    out = (ctypes.c_uint8 * 48)()
    _load().ivo_sha384(_ptr(arr), arr.size, out)
    return bytes(out)


def hash_chunks_sha384(data, chunk_bytes: int, nthreads: int = 1) -> np.ndarray:
    """SHA-384 chunk digests as an (n, 48) uint8 array."""
    arr = _as_u8(data)
    if chunk_bytes <= 0:
        raise ValueError("chunk_bytes must be positive")
    n = n_chunks(arr.size, chunk_bytes)
    out = np.zeros((n, 48), dtype=np.uint8)
    got = _load().ivo_hash_chunks_sha384(_ptr(arr), arr.size, chunk_bytes, _ptr(out), nthreads)
    assert got == n
    return out


def merkle_root_sha384(leaves) -> bytes:
    arr = _as_u8(leaves)
    assert arr.size % 48 == 0
    out = (ctypes.c_uint8 * 48)()
    _load().ivo_merkle_root_sha384(_ptr(arr), arr.size // 48, out)
    return bytes(out)


# ---------------------------------------------------------------------------------------------
# SHA-512 variant

def h0_sha512() -> np.ndarray:
    """The SHA-512 initial value (FIPS 180-4 section 5.3.5) as derived from the first eight primes."""
    h0 = np.zeros(8, dtype=np.uint64)
    _load().ivo_h0_sha512(h0.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)))
    return h0


def sha512(msg) -> bytes:
    arr = _as_u8(msg)
    out = (ctypes.c_uint8 * 64)()
    _load().ivo_sha512(_ptr(arr), arr.size, out)
    return bytes(out)


def hash_chunks_sha512(data, chunk_bytes: int, nthreads: int = 1) -> np.ndarray:
    """SHA-512 chunk digests as an (n, 64) uint8 array."""
    arr = _as_u8(data)
    if chunk_bytes <= 0:
        raise ValueError("chunk_bytes must be positive")
    n = n_chunks(arr.size, chunk_bytes)
    out = np.zeros((n, 64), dtype=np.uint8)
    got = _load().ivo_hash_chunks_sha512(_ptr(arr), arr.size, chunk_bytes, _ptr(out), nthreads)
    assert got == n
    return out


def merkle_root_sha512(leaves) -> bytes:
    arr = _as_u8(leaves)
    assert arr.size % 64 == 0
    out = (ctypes.c_uint8 * 64)()
    _load().ivo_merkle_root_sha512(_ptr(arr), arr.size // 64, out)
    return bytes(out)


# ---------------------------------------------------------------------------------------------
# RFC 6962 mode (domain-separated Merkle Tree Hash)

def hash_chunks_rfc6962(data, chunk_bytes: int, nthreads: int = 1) -> np.ndarray:
    """Leaf hashes SHA-256(0x00 || chunk) as an (n, 32) uint8 array."""
    arr = _as_u8(data)
    if chunk_bytes <= 0:
        raise ValueError("chunk_bytes must be positive")
    n = n_chunks(arr.size, chunk_bytes)
    out = np.zeros((n, 32), dtype=np.uint8)
    got = _load().ivo_hash_chunks_rfc6962(_ptr(arr), arr.size, chunk_bytes, _ptr(out), nthreads)
    assert got == n
    return out


def merkle_root_rfc6962(leaf_hashes) -> bytes:
    arr = _as_u8(leaf_hashes)
    assert arr.size % 32 == 0
    out = (ctypes.c_uint8 * 32)()
    _load().ivo_merkle_root_rfc6962(_ptr(arr), arr.size // 32, out)
    return bytes(out)
