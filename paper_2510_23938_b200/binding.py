"""ctypes binding of libiv.so: the same entry points as include/iv.h.

Argument marshalling only.  Tensors are torch CUDA tensors (torch supplies
device memory and streams); every step of the path runs inside the library's
kernels.  There is no fallback: if the shared library is missing, loading
raises with the build command.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libiv.so")

IV_OK = 0
IV_ERR_INVALID_ARG = -1
IV_ERR_NOMEM = -2
IV_ERR_CUDA = -3
IV_ERR_NO_DEVICE = -4
IV_ERR_TOO_LARGE = -5
NOALLOC_MAX_LEAVES = 512 * 512

EXPORTS = (
    "iv_create", "iv_destroy", "iv_strerror", "iv_last_cuda_error", "iv_kernel_launches",
    "iv_hash_chunks", "iv_merkle_root", "iv_verify_manifest", "iv_ctx_digests",
    "iv_verify_streamed", "iv_hash_ragged", "iv_set_timing", "iv_phase_times", "iv_probe_alu", "iv_device_status",
    "iv_merkle_root_noalloc", "iv_last_leaf_kernel", "iv_last_leaf_instance", "iv_selftest_wait_timeout", "iv_merkle_levels",
    "iv_tree_records", "iv_tree_build", "iv_tree_update",
    "iv_hash_chunks_two_level", "iv_verify_manifest_two_level", "iv_hash_ragged_update", "iv_verify_manifest_batch",
    "iv_hash_chunks_sha384", "iv_merkle_root_sha384", "iv_verify_manifest_sha384",
    "iv_hash_chunks_sha512", "iv_merkle_root_sha512", "iv_verify_manifest_sha512",
    "iv_hash_chunks_rfc6962", "iv_merkle_root_rfc6962", "iv_verify_manifest_rfc6962",
)


class IvError(RuntimeError):
    def __init__(self, code: int, what: str, cuda_error: int = 0):
        self.code = code
        self.cuda_error = cuda_error
        extra = f" (cudaError {cuda_error})" if cuda_error else ""
        super().__init__(f"{what}: {_strerror(code)}{extra}")


class Manifest(ctypes.Structure):
    """iv_manifest: host struct, digest array on the device."""
    _fields_ = [("total_bytes", ctypes.c_uint64), ("chunk_bytes", ctypes.c_uint64),
                ("n_chunks", ctypes.c_uint64), ("d_digests", ctypes.c_void_p),
                ("root", ctypes.c_uint8 * 32)]


class Manifest384(ctypes.Structure):
    """iv_manifest_sha384: host struct, 48-byte digest records on the device."""
    _fields_ = [("total_bytes", ctypes.c_uint64), ("chunk_bytes", ctypes.c_uint64),
                ("n_chunks", ctypes.c_uint64), ("d_digests", ctypes.c_void_p),
                ("root", ctypes.c_uint8 * 48)]


class VerifyResult384(ctypes.Structure):
    """iv_verify_result_sha384 as laid out in device memory (64 bytes)."""
    _fields_ = [("status", ctypes.c_uint32), ("root_ok", ctypes.c_uint32),
                ("n_mismatch", ctypes.c_uint64), ("root", ctypes.c_uint8 * 48)]


class Manifest512(ctypes.Structure):
    """iv_manifest_sha512: host struct, 64-byte digest records on the device."""
    _fields_ = [("total_bytes", ctypes.c_uint64), ("chunk_bytes", ctypes.c_uint64),
                ("n_chunks", ctypes.c_uint64), ("d_digests", ctypes.c_void_p),
                ("root", ctypes.c_uint8 * 64)]


class VerifyResult512(ctypes.Structure):
    """iv_verify_result_sha512 as laid out in device memory (80 bytes)."""
    _fields_ = [("status", ctypes.c_uint32), ("root_ok", ctypes.c_uint32),
                ("n_mismatch", ctypes.c_uint64), ("root", ctypes.c_uint8 * 64)]


class VerifyResult(ctypes.Structure):
    """iv_verify_result as laid out in device memory (48 bytes)."""
    _fields_ = [("status", ctypes.c_uint32), ("root_ok", ctypes.c_uint32),
                ("n_mismatch", ctypes.c_uint64), ("root", ctypes.c_uint8 * 32)]


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libiv.so from the package directory; raises if it was not built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2510_23938_b200.build` "
            "(needs nvcc; there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, u64, i32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_int
    lib.iv_create.argtypes = [ctypes.POINTER(vp), i32]
    lib.iv_create.restype = i32
    lib.iv_destroy.argtypes = [vp]
    lib.iv_destroy.restype = i32
    lib.iv_strerror.argtypes = [i32]
    lib.iv_strerror.restype = ctypes.c_char_p
    lib.iv_last_cuda_error.argtypes = [vp]
    lib.iv_last_cuda_error.restype = i32
    lib.iv_kernel_launches.argtypes = [vp]
    lib.iv_kernel_launches.restype = u64
    lib.iv_hash_chunks.argtypes = [vp, vp, u64, u64, vp, u64, ctypes.POINTER(u64), vp]
    lib.iv_hash_chunks.restype = i32
    lib.iv_merkle_root.argtypes = [vp, vp, u64, vp, vp]
    lib.iv_merkle_root.restype = i32
    lib.iv_merkle_levels.argtypes = [vp, vp, u64, ctypes.c_uint32, vp, u64, ctypes.POINTER(u64), vp]
    lib.iv_merkle_levels.restype = i32
    lib.iv_tree_records.argtypes = [u64]
    lib.iv_tree_records.restype = u64
    lib.iv_tree_build.argtypes = [vp, vp, u64, vp, u64, vp]
    lib.iv_tree_build.restype = i32
    lib.iv_tree_update.argtypes = [vp, vp, u64, u64, vp, u64, vp, u64, vp]
    lib.iv_tree_update.restype = i32
    lib.iv_hash_chunks_two_level.argtypes = [vp, vp, u64, u64, u64, vp, u64, ctypes.POINTER(u64), vp]
    lib.iv_hash_chunks_two_level.restype = i32
    lib.iv_verify_manifest_two_level.argtypes = [vp, vp, u64, ctypes.POINTER(Manifest), u64, vp, vp, u64, vp]
    lib.iv_verify_manifest_two_level.restype = i32
    lib.iv_hash_ragged_update.argtypes = [vp, vp, vp, vp, u64, vp, i32, vp, vp]
    lib.iv_hash_ragged_update.restype = i32
    lib.iv_verify_manifest_batch.argtypes = [vp, ctypes.POINTER(vp), u64, u64, ctypes.POINTER(Manifest), vp, vp, u64, vp]
    lib.iv_verify_manifest_batch.restype = i32
    lib.iv_hash_chunks_sha384.argtypes = [vp, vp, u64, u64, vp, u64, ctypes.POINTER(u64), vp]
    lib.iv_hash_chunks_sha384.restype = i32
    lib.iv_merkle_root_sha384.argtypes = [vp, vp, u64, vp, vp]
    lib.iv_merkle_root_sha384.restype = i32
    lib.iv_hash_chunks_sha512.argtypes = [vp, vp, u64, u64, vp, u64, ctypes.POINTER(u64), vp]
    lib.iv_hash_chunks_sha512.restype = i32
    lib.iv_merkle_root_sha512.argtypes = [vp, vp, u64, vp, vp]
    lib.iv_merkle_root_sha512.restype = i32
    lib.iv_verify_manifest_sha512.argtypes = [vp, vp, u64, ctypes.POINTER(Manifest512), vp, vp, u64, vp]
    lib.iv_verify_manifest_sha512.restype = i32
    lib.iv_verify_manifest_rfc6962.argtypes = [vp, vp, u64, ctypes.POINTER(Manifest), vp, vp, u64, vp]
    lib.iv_verify_manifest_rfc6962.restype = i32
    lib.iv_verify_manifest_sha384.argtypes = [vp, vp, u64, ctypes.POINTER(Manifest384), vp, vp, u64, vp]
    lib.iv_verify_manifest_sha384.restype = i32
    lib.iv_hash_chunks_rfc6962.argtypes = [vp, vp, u64, u64, vp, u64, ctypes.POINTER(u64), vp]
    lib.iv_hash_chunks_rfc6962.restype = i32
    lib.iv_merkle_root_rfc6962.argtypes = [vp, vp, u64, vp, vp]
    lib.iv_merkle_root_rfc6962.restype = i32
    lib.iv_verify_manifest.argtypes = [vp, vp, u64, ctypes.POINTER(Manifest), vp, vp, u64, vp]
    lib.iv_verify_manifest.restype = i32
    lib.iv_ctx_digests.argtypes = [vp]
    lib.iv_ctx_digests.restype = vp
    lib.iv_verify_streamed.argtypes = [vp, ctypes.POINTER(vp), u64, u64, u64, ctypes.POINTER(Manifest),
                                       vp, vp, u64, vp]
    lib.iv_verify_streamed.restype = i32
    lib.iv_set_timing.argtypes = [vp, i32]
    lib.iv_set_timing.restype = i32
    lib.iv_phase_times.argtypes = [vp, ctypes.c_uint32, ctypes.POINTER(ctypes.c_float)]
    lib.iv_phase_times.restype = i32
    lib.iv_hash_ragged.argtypes = [vp, vp, vp, vp, u64, vp, vp]
    lib.iv_hash_ragged.restype = i32
    lib.iv_merkle_root_noalloc.argtypes = [vp, u64, vp, vp]
    lib.iv_merkle_root_noalloc.restype = i32
    lib.iv_last_leaf_kernel.argtypes = [vp]
    lib.iv_last_leaf_kernel.restype = ctypes.c_char_p
    lib.iv_last_leaf_instance.argtypes = [vp]
    lib.iv_last_leaf_instance.restype = ctypes.c_char_p
    lib.iv_selftest_wait_timeout.argtypes = [vp, u64, ctypes.POINTER(u64), vp]
    lib.iv_selftest_wait_timeout.restype = i32
    lib.iv_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.iv_device_status.restype = i32
    lib.iv_probe_alu.argtypes = [vp, i32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                 ctypes.POINTER(ctypes.c_double)]
    lib.iv_probe_alu.restype = i32
    _lib = lib
    return lib


def _strerror(code: int) -> str:
    try:
        return load_library().iv_strerror(code).decode()
    except Exception:  # pragma: no cover
        return f"status {code}"


def n_chunks(nbytes: int, chunk_bytes: int) -> int:
    return 0 if nbytes == 0 else (nbytes - 1) // chunk_bytes + 1


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def _dev_ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None or t.numel() == 0:
        return None
    assert t.is_cuda and t.is_contiguous(), "device tensors must be contiguous CUDA tensors"
    return t.data_ptr()


def _nbytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


class Context:
    """iv_ctx: scratch memory and streams of one verifier on one device."""

    def __init__(self, device: int | None = None):
        lib = load_library()
        if device is None:
            device = torch.cuda.current_device() if torch.cuda.is_available() else 0
        self.device = int(device)
        handle = ctypes.c_void_p()
        rc = lib.iv_create(ctypes.byref(handle), self.device)
        if rc != IV_OK:
            raise IvError(rc, "iv_create")
        self._h = handle
        self._lib = lib

    # -- plumbing ---------------------------------------------------------------------------
    def close(self):
        if getattr(self, "_h", None):
            self._lib.iv_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    def _check(self, rc: int, what: str):
        if rc != IV_OK:
            raise IvError(rc, what, self._lib.iv_last_cuda_error(self._h))

    @property
    def kernel_launches(self) -> int:
        return int(self._lib.iv_kernel_launches(self._h))

    # -- entry points -----------------------------------------------------------------------
    def hash_chunks(self, data: torch.Tensor, chunk_bytes: int, out: torch.Tensor | None = None,
                    nbytes: int | None = None, stream=None) -> torch.Tensor:
        """iv_hash_chunks: (n, 32) uint8 digests of the chunks of `data` (any dtype, read as bytes)."""
        nb = _nbytes(data) if nbytes is None else int(nbytes)
        n = n_chunks(nb, chunk_bytes) if chunk_bytes > 0 else 0
        if out is None:
            out = torch.empty((n, 32), dtype=torch.uint8, device=data.device)
        got = ctypes.c_uint64(0)
        rc = self._lib.iv_hash_chunks(self._h, _dev_ptr(data), nb, chunk_bytes, _dev_ptr(out),
                                      out.numel() // 32, ctypes.byref(got), _stream_ptr(stream))
        self._check(rc, "iv_hash_chunks")
        return out[:got.value]

    def hash_chunks_two_level(self, data: torch.Tensor, chunk_bytes: int, sub_bytes: int, stream=None,
                              out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_hash_chunks_two_level: digest i = Merkle root over the SHA-256 digests of chunk i's sub_bytes pieces."""
        nb = _nbytes(data)
        n = n_chunks(nb, chunk_bytes) if chunk_bytes > 0 else 0
        if out is None:
            out = torch.empty((n, 32), dtype=torch.uint8, device=data.device)
        got = ctypes.c_uint64(0)
        rc = self._lib.iv_hash_chunks_two_level(self._h, _dev_ptr(data), nb, chunk_bytes, sub_bytes, _dev_ptr(out), n,
                                                ctypes.byref(got), _stream_ptr(stream))
        self._check(rc, "iv_hash_chunks_two_level")
        return out[:got.value]

    def verify_manifest_two_level(self, data: torch.Tensor, manifest: Manifest, sub_bytes: int, result: torch.Tensor,
                                  mismatch_idx: torch.Tensor | None, stream=None) -> None:
        """iv_verify_manifest_two_level (asynchronous); the manifest must hold two-level digests."""
        cap = 0 if mismatch_idx is None else mismatch_idx.numel()
        rc = self._lib.iv_verify_manifest_two_level(self._h, _dev_ptr(data), _nbytes(data), ctypes.byref(manifest),
                                                    sub_bytes, _dev_ptr(result), _dev_ptr(mismatch_idx), cap,
                                                    _stream_ptr(stream))
        self._check(rc, "iv_verify_manifest_two_level")

    def merkle_root(self, leaves: torch.Tensor, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
        """iv_merkle_root: 32-byte root (uint8 tensor on the device) of (n, 32) leaf digests."""
        n = leaves.numel() // 32
        if out is None:
            out = torch.empty(32, dtype=torch.uint8, device=leaves.device)
        rc = self._lib.iv_merkle_root(self._h, _dev_ptr(leaves), n, _dev_ptr(out), _stream_ptr(stream))
        self._check(rc, "iv_merkle_root")
        return out

    def hash_chunks_sha384(self, data: torch.Tensor, chunk_bytes: int, stream=None,
                           out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_hash_chunks_sha384: (n, 48) uint8 SHA-384 digests of the chunks of `data`."""
        nb = _nbytes(data)
        n = n_chunks(nb, chunk_bytes) if chunk_bytes > 0 else 0
        if out is None:
            out = torch.empty((n, 48), dtype=torch.uint8, device=data.device)
        got = ctypes.c_uint64(0)
        rc = self._lib.iv_hash_chunks_sha384(self._h, _dev_ptr(data), nb, chunk_bytes, _dev_ptr(out), n,
                                             ctypes.byref(got), _stream_ptr(stream))
        self._check(rc, "iv_hash_chunks_sha384")
        return out[:got.value]

    def merkle_root_sha384(self, leaves: torch.Tensor, stream=None, out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_merkle_root_sha384: 48-byte root of (n, 48) leaf digests."""
        n = leaves.numel() // 48
        if out is None:
            out = torch.empty(48, dtype=torch.uint8, device=leaves.device)
        rc = self._lib.iv_merkle_root_sha384(self._h, _dev_ptr(leaves), n, _dev_ptr(out), _stream_ptr(stream))
        self._check(rc, "iv_merkle_root_sha384")
        return out

    def hash_chunks_sha512(self, data: torch.Tensor, chunk_bytes: int, stream=None,
                           out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_hash_chunks_sha512: (n, 64) uint8 SHA-512 digests of the chunks of `data`."""
        nb = _nbytes(data)
        n = n_chunks(nb, chunk_bytes) if chunk_bytes > 0 else 0
        if out is None:
            out = torch.empty((n, 64), dtype=torch.uint8, device=data.device)
        got = ctypes.c_uint64(0)
        rc = self._lib.iv_hash_chunks_sha512(self._h, _dev_ptr(data), nb, chunk_bytes, _dev_ptr(out), n,
                                             ctypes.byref(got), _stream_ptr(stream))
        self._check(rc, "iv_hash_chunks_sha512")
        return out[:got.value]

    def merkle_root_sha512(self, leaves: torch.Tensor, stream=None, out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_merkle_root_sha512: 64-byte root of (n, 64) leaf digests."""
        n = leaves.numel() // 64
        if out is None:
            out = torch.empty(64, dtype=torch.uint8, device=leaves.device)
        rc = self._lib.iv_merkle_root_sha512(self._h, _dev_ptr(leaves), n, _dev_ptr(out), _stream_ptr(stream))
        self._check(rc, "iv_merkle_root_sha512")
        return out

    def verify_manifest_sha384(self, data: torch.Tensor, total_bytes: int, chunk_bytes: int, digests: torch.Tensor,
                               root: bytes, mismatch_idx: torch.Tensor | None = None, stream=None) -> dict:
        """iv_verify_manifest_sha384: verifies `data` against SHA-384 chunk digests (an (n, 48) device tensor) and
        the 48-byte root; waits for the result and returns it as a dict (status, root_ok, n_mismatch, root)."""
        m = Manifest384()
        m.total_bytes, m.chunk_bytes, m.n_chunks = total_bytes, chunk_bytes, digests.numel() // 48
        m.d_digests = _dev_ptr(digests)
        m.root = (ctypes.c_uint8 * 48).from_buffer_copy(root)
        result = torch.zeros(ctypes.sizeof(VerifyResult384), dtype=torch.uint8, device=data.device)
        cap = 0 if mismatch_idx is None else mismatch_idx.numel()
        rc = self._lib.iv_verify_manifest_sha384(self._h, _dev_ptr(data), _nbytes(data), ctypes.byref(m), _dev_ptr(result),
                                                 _dev_ptr(mismatch_idx), cap, _stream_ptr(stream))
        self._check(rc, "iv_verify_manifest_sha384")
        r = VerifyResult384.from_buffer_copy(bytes(result.cpu().numpy().tobytes()))
        return {"status": int(r.status), "root_ok": bool(r.root_ok), "n_mismatch": int(r.n_mismatch), "root": bytes(r.root)}

    def verify_manifest_sha512(self, data: torch.Tensor, total_bytes: int, chunk_bytes: int, digests: torch.Tensor,
                               root: bytes, mismatch_idx: torch.Tensor | None = None, stream=None) -> dict:
        """iv_verify_manifest_sha512: as verify_manifest_sha384 with (n, 64) digests and a 64-byte root."""
        m = Manifest512()
        m.total_bytes, m.chunk_bytes, m.n_chunks = total_bytes, chunk_bytes, digests.numel() // 64
        m.d_digests = _dev_ptr(digests)
        m.root = (ctypes.c_uint8 * 64).from_buffer_copy(root)
        result = torch.zeros(ctypes.sizeof(VerifyResult512), dtype=torch.uint8, device=data.device)
        cap = 0 if mismatch_idx is None else mismatch_idx.numel()
        rc = self._lib.iv_verify_manifest_sha512(self._h, _dev_ptr(data), _nbytes(data), ctypes.byref(m), _dev_ptr(result),
                                                 _dev_ptr(mismatch_idx), cap, _stream_ptr(stream))
        self._check(rc, "iv_verify_manifest_sha512")
        r = VerifyResult512.from_buffer_copy(bytes(result.cpu().numpy().tobytes()))
        return {"status": int(r.status), "root_ok": bool(r.root_ok), "n_mismatch": int(r.n_mismatch), "root": bytes(r.root)}

    def hash_chunks_rfc6962(self, data: torch.Tensor, chunk_bytes: int, stream=None,
                            out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_hash_chunks_rfc6962: (n, 32) uint8 leaf hashes SHA-256(0x00 || chunk)."""
        nb = _nbytes(data)
        n = n_chunks(nb, chunk_bytes) if chunk_bytes > 0 else 0
        if out is None:
            out = torch.empty((n, 32), dtype=torch.uint8, device=data.device)
        got = ctypes.c_uint64(0)
        rc = self._lib.iv_hash_chunks_rfc6962(self._h, _dev_ptr(data), nb, chunk_bytes, _dev_ptr(out), n,
                                              ctypes.byref(got), _stream_ptr(stream))
        self._check(rc, "iv_hash_chunks_rfc6962")
        return out[:got.value]

    def merkle_root_rfc6962(self, leaves: torch.Tensor, stream=None, out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_merkle_root_rfc6962: 32-byte root with 0x01-prefixed nodes over (n, 32) leaf hashes."""
        n = leaves.numel() // 32
        if out is None:
            out = torch.empty(32, dtype=torch.uint8, device=leaves.device)
        rc = self._lib.iv_merkle_root_rfc6962(self._h, _dev_ptr(leaves), n, _dev_ptr(out), _stream_ptr(stream))
        self._check(rc, "iv_merkle_root_rfc6962")
        return out

    def merkle_levels(self, nodes: torch.Tensor, levels: int, stream=None, out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_merkle_levels: the (ceil(n / 2^levels), 32) nodes `levels` levels above `nodes`."""
        n = nodes.numel() // 32
        n_out = n
        for _ in range(levels):
            if n_out <= 1:
                break
            n_out = (n_out + 1) // 2
        if out is None:
            out = torch.empty((n_out, 32), dtype=torch.uint8, device=nodes.device)
        got = ctypes.c_uint64(0)
        rc = self._lib.iv_merkle_levels(self._h, _dev_ptr(nodes), n, levels, _dev_ptr(out), n_out,
                                        ctypes.byref(got), _stream_ptr(stream))
        self._check(rc, "iv_merkle_levels")
        assert got.value == n_out
        return out

    def tree_records(self, n_leaves: int) -> int:
        return int(self._lib.iv_tree_records(n_leaves))

    def tree_build(self, leaves: torch.Tensor, stream=None, out: torch.Tensor | None = None) -> torch.Tensor:
        """iv_tree_build: the retained tree (iv_tree_records(n), 32) of the (n, 32) leaf digests; root = tree[-1]."""
        n = leaves.numel() // 32
        records = int(self._lib.iv_tree_records(n))
        tree = torch.empty((records, 32), dtype=torch.uint8, device=leaves.device) if out is None else out
        rc = self._lib.iv_tree_build(self._h, _dev_ptr(leaves), n, _dev_ptr(tree), records, _stream_ptr(stream))
        self._check(rc, "iv_tree_build")
        return tree

    def tree_update(self, data: torch.Tensor, chunk_bytes: int, dirty: torch.Tensor, tree: torch.Tensor,
                    stream=None) -> None:
        """iv_tree_update: re-hash the chunks whose indices are in the int64 device tensor `dirty`."""
        assert dirty.dtype == torch.int64
        rc = self._lib.iv_tree_update(self._h, _dev_ptr(data), _nbytes(data), chunk_bytes, _dev_ptr(dirty),
                                      dirty.numel(), _dev_ptr(tree), tree.numel() // 32, _stream_ptr(stream))
        self._check(rc, "iv_tree_update")

    def make_manifest(self, total_bytes: int, chunk_bytes: int, digests: torch.Tensor, root: bytes) -> Manifest:
        m = Manifest()
        m.total_bytes = total_bytes
        m.chunk_bytes = chunk_bytes
        m.n_chunks = digests.numel() // 32
        m.d_digests = _dev_ptr(digests)
        m.root = (ctypes.c_uint8 * 32).from_buffer_copy(root)
        m._keepalive = digests
        return m

    def verify_manifest(self, data: torch.Tensor, manifest: Manifest, result: torch.Tensor,
                        mismatch_idx: torch.Tensor | None, nbytes: int | None = None, stream=None) -> None:
        """iv_verify_manifest (asynchronous): `result` is a 48-byte uint8 device tensor,
        `mismatch_idx` an int64 device tensor whose length is the index capacity."""
        nb = _nbytes(data) if nbytes is None else int(nbytes)
        cap = 0 if mismatch_idx is None else mismatch_idx.numel()
        rc = self._lib.iv_verify_manifest(self._h, _dev_ptr(data), nb, ctypes.byref(manifest),
                                          _dev_ptr(result), _dev_ptr(mismatch_idx), cap, _stream_ptr(stream))
        self._check(rc, "iv_verify_manifest")

    def verify_manifest_rfc6962(self, data: torch.Tensor, manifest: Manifest, result: torch.Tensor,
                                mismatch_idx: torch.Tensor | None, stream=None) -> None:
        """iv_verify_manifest_rfc6962 (asynchronous); the manifest holds prefixed leaf hashes and their root."""
        cap = 0 if mismatch_idx is None else mismatch_idx.numel()
        rc = self._lib.iv_verify_manifest_rfc6962(self._h, _dev_ptr(data), _nbytes(data), ctypes.byref(manifest),
                                                  _dev_ptr(result), _dev_ptr(mismatch_idx), cap, _stream_ptr(stream))
        self._check(rc, "iv_verify_manifest_rfc6962")

    def verify_manifest_batch(self, blobs: list, manifest: Manifest, results: torch.Tensor,
                              mismatch_idx: torch.Tensor | None, stream=None) -> None:
        """iv_verify_manifest_batch (asynchronous): `blobs` are equally sized device tensors, `results` a
        (len(blobs), 48) uint8 device tensor, `mismatch_idx` a (len(blobs), cap) int64 device tensor."""
        nb = _nbytes(blobs[0])
        assert all(_nbytes(b) == nb and b.is_cuda and b.is_contiguous() for b in blobs)
        ptrs = (ctypes.c_void_p * len(blobs))(*[b.data_ptr() for b in blobs])
        cap = 0 if mismatch_idx is None else mismatch_idx.shape[1]
        rc = self._lib.iv_verify_manifest_batch(self._h, ptrs, len(blobs), nb, ctypes.byref(manifest), _dev_ptr(results),
                                                _dev_ptr(mismatch_idx), cap, _stream_ptr(stream))
        self._check(rc, "iv_verify_manifest_batch")

    def verify_streamed(self, host_windows, window_bytes: int, nbytes: int, manifest: Manifest,
                        result: torch.Tensor, mismatch_idx: torch.Tensor | None, stream=None) -> None:
        """iv_verify_streamed (asynchronous).  `host_windows` is a CPU uint8 tensor holding the whole
        blob, or a list of CPU tensors, one per window (pinned for overlap; entries may repeat)."""
        if isinstance(host_windows, torch.Tensor):
            flat = host_windows.view(torch.uint8).reshape(-1)
            assert not flat.is_cuda and flat.is_contiguous() and flat.numel() >= nbytes
            host_windows = [flat[o:o + window_bytes] for o in range(0, nbytes, window_bytes)] if window_bytes > 0 else []
        n_win = len(host_windows)
        ptrs = (ctypes.c_void_p * max(n_win, 1))()
        for w, t in enumerate(host_windows):
            assert not t.is_cuda and t.is_contiguous()
            ptrs[w] = t.data_ptr()
        cap = 0 if mismatch_idx is None else mismatch_idx.numel()
        rc = self._lib.iv_verify_streamed(self._h, ptrs, n_win, window_bytes, nbytes, ctypes.byref(manifest),
                                          _dev_ptr(result), _dev_ptr(mismatch_idx), cap, _stream_ptr(stream))
        self._check(rc, "iv_verify_streamed")

    def set_timing(self, enabled: bool) -> None:
        self._check(self._lib.iv_set_timing(self._h, int(enabled)), "iv_set_timing")

    def phase_times(self, calls_back: int = 0) -> tuple[float, float, float]:
        """iv_phase_times: (hash, tree, compare) milliseconds of a recent verification call."""
        ms = (ctypes.c_float * 3)()
        self._check(self._lib.iv_phase_times(self._h, calls_back, ms), "iv_phase_times")
        return float(ms[0]), float(ms[1]), float(ms[2])

    def hash_ragged(self, base: torch.Tensor, offsets: torch.Tensor, lengths: torch.Tensor,
                    out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
        """iv_hash_ragged: (n, 32) digests of base[offset_k : offset_k + length_k) (offsets/lengths int64 on device)."""
        n = offsets.numel()
        assert lengths.numel() == n and offsets.dtype == torch.int64 and lengths.dtype == torch.int64
        if out is None:
            out = torch.empty((n, 32), dtype=torch.uint8, device=base.device)
        rc = self._lib.iv_hash_ragged(self._h, _dev_ptr(base), _dev_ptr(offsets), _dev_ptr(lengths), n,
                                      _dev_ptr(out), _stream_ptr(stream))
        self._check(rc, "iv_hash_ragged")
        return out

    @property
    def last_leaf_kernel(self) -> str:
        return self._lib.iv_last_leaf_kernel(self._h).decode()

    @property
    def last_leaf_instance(self) -> str:
        return self._lib.iv_last_leaf_instance(self._h).decode()

    def selftest_wait_timeout(self, limit_cycles: int, stream=None) -> int:
        """iv_selftest_wait_timeout: a warp waits `limit_cycles` SM clocks on a barrier nobody arrives at, gives
        up and sets the device status to 1; returns the clocks it waited (synchronises the stream)."""
        waited = ctypes.c_uint64(0)
        rc = self._lib.iv_selftest_wait_timeout(self._h, int(limit_cycles), ctypes.byref(waited), _stream_ptr(stream))
        self._check(rc, "iv_selftest_wait_timeout")
        return int(waited.value)

    def device_status(self) -> int:
        """iv_device_status: waits for the device, returns and clears the device-side status word."""
        st = ctypes.c_uint32(0)
        self._check(self._lib.iv_device_status(self._h, ctypes.byref(st)), "iv_device_status")
        return int(st.value)

    PROBE_KINDS = {"iadd3": 0, "lop3": 1, "shf": 2, "prmt": 3, "imad": 4, "mixed": 5, "sha256": 6, "sha256_sched_fma": 7,
                   "lat_iadd3": 8, "lat_lop3": 9, "lat_shf": 10, "lat_imad": 11, "lat_cross": 12,
                   "rounds": 13, "schedule": 14}

    def probe_alu(self, kind: str, warps_per_block: int = 4, blocks_per_sm: int = 1, active_lanes: int = 32,
                  iters: int = 2000) -> tuple[float, float]:
        """iv_probe_alu: (lane-ops or bytes per clock per SM, mean cycles per block)."""
        out = (ctypes.c_double * 2)()
        rc = self._lib.iv_probe_alu(self._h, self.PROBE_KINDS[kind], warps_per_block, blocks_per_sm,
                                    active_lanes, iters, out)
        self._check(rc, "iv_probe_alu")
        return float(out[0]), float(out[1])

    SHA_STATE_BYTES = 48

    def new_sha_states(self, n: int) -> torch.Tensor:
        """Zero-filled iv_sha_state records for n tensors (an (n, 48) uint8 device tensor)."""
        return torch.zeros((n, self.SHA_STATE_BYTES), dtype=torch.uint8, device=f"cuda:{self.device}")

    def hash_ragged_update(self, base: torch.Tensor, offsets: torch.Tensor, lengths: torch.Tensor,
                           states: torch.Tensor, finish: bool, out: torch.Tensor | None = None, stream=None):
        """iv_hash_ragged_update: hash the next part of every tensor; returns the (n, 32) digests when finishing."""
        n = offsets.numel()
        assert lengths.numel() == n and states.numel() == n * self.SHA_STATE_BYTES
        if finish and out is None:
            out = torch.empty((n, 32), dtype=torch.uint8, device=base.device)
        rc = self._lib.iv_hash_ragged_update(self._h, _dev_ptr(base) or base.data_ptr(), _dev_ptr(offsets),
                                             _dev_ptr(lengths), n, _dev_ptr(states), int(finish),
                                             _dev_ptr(out) if out is not None else None, _stream_ptr(stream))
        self._check(rc, "iv_hash_ragged_update")
        return out if finish else None

    def last_digests(self, n: int) -> torch.Tensor:
        """Copy of the chunk digests the last verification on this context computed."""
        ptr = self._lib.iv_ctx_digests(self._h)
        if not ptr:
            raise RuntimeError("no verification has run on this context")
        if n == 0:
            return torch.empty((0, 32), dtype=torch.uint8, device=f"cuda:{self.device}")
        view = torch.as_tensor(_DeviceBytes(ptr, 32 * n), device=f"cuda:{self.device}")
        return view.clone().view(n, 32)


class _DeviceBytes:
    """Exposes a raw device pointer to torch through the CUDA array interface (no ownership)."""

    def __init__(self, ptr: int, nbytes: int):
        self.__cuda_array_interface__ = {"shape": (nbytes,), "typestr": "|u1", "data": (int(ptr), False),
                                         "version": 2}


def merkle_root_noalloc(leaves: torch.Tensor, out: torch.Tensor, n_leaves: int | None = None, stream=None) -> torch.Tensor:
    """iv_merkle_root_noalloc: Merkle root into the caller's 32-byte device tensor `out`.

    For callers that cannot allocate on the device (a pool owns the GPU, or the allocator must not
    be touched): no context, no allocation in the library, and none here -- both tensors are the
    caller's.  At most NOALLOC_MAX_LEAVES leaves; calls must not overlap on the GPU."""
    lib = load_library()
    n = leaves.numel() // 32 if n_leaves is None else int(n_leaves)
    assert out.is_cuda and out.is_contiguous() and out.numel() >= 32
    rc = lib.iv_merkle_root_noalloc(_dev_ptr(leaves), n, out.data_ptr(), _stream_ptr(stream))
    if rc != IV_OK:
        raise IvError(rc, "iv_merkle_root_noalloc")
    return out


def read_result(result: torch.Tensor) -> dict:
    """Decodes a 48-byte iv_verify_result tensor (synchronises on the copy to the host)."""
    raw = bytes(result.cpu().numpy().tobytes())
    r = VerifyResult.from_buffer_copy(raw)
    return {"status": int(r.status), "root_ok": bool(r.root_ok), "n_mismatch": int(r.n_mismatch),
            "root": bytes(r.root)}


def read_results(results: torch.Tensor) -> list:
    """Decodes an (n, 48) tensor of iv_verify_result records."""
    raw = results.cpu().numpy().tobytes()
    size = ctypes.sizeof(VerifyResult)
    out = []
    for o in range(0, len(raw), size):
        r = VerifyResult.from_buffer_copy(raw[o:o + size])
        out.append({"status": int(r.status), "root_ok": bool(r.root_ok), "n_mismatch": int(r.n_mismatch),
                    "root": bytes(r.root)})
    return out


def new_result(device) -> torch.Tensor:
    return torch.zeros(ctypes.sizeof(VerifyResult), dtype=torch.uint8, device=device)
