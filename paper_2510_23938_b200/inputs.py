"""Seeded synthetic inputs shaped like the paper's workloads (model-weight blobs).

Used by the tests, the smoke check and the benchmark; it holds none of the
method's arithmetic (no hashing, no tree).  Every generator is counter based
(a 64-bit mix of ``seed`` and the element index) and written with integer torch
ops only, so the same call gives the same bytes on the CPU and on the GPU and
for any slab size.

Workloads
  * uniform random bytes (the 64 MiB small case),
  * bf16 weights ~N(0, 0.02): the sum of four uniform bytes (Irwin-Hall, 1021
    levels), centred and scaled to a standard deviation of 0.02, rounded to
    bf16 -- 2 bytes per parameter, little endian,
  * weight files: 8-byte little-endian header length, a JSON tensor index
    (name -> dtype, shape, data offsets; padded with spaces to 8 bytes), then
    the tensors back to back, for a 1.3B-parameter GPT-style and an
    8B-parameter Llama-style layer list,
  * a ragged tensor set with log-uniform byte sizes.
"""
from __future__ import annotations

import json
import math
import struct

import numpy as np
import torch

_MASK64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB


def _i64(v: int) -> int:
    """Python int -> the signed 64-bit value with the same bits."""
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    """Logical right shift of int64 (torch's >> is arithmetic)."""
    return (z >> k) & ((1 << (64 - k)) - 1)


def mix64(first_index: int, count: int, seed: int, device) -> torch.Tensor:
    """splitmix64-style finaliser of (seed, index) for index = first_index .. first_index+count-1."""
    idx = torch.arange(first_index, first_index + count, dtype=torch.int64, device=device)
    z = idx * _i64(_GOLDEN) + _i64(seed * _C2 + _GOLDEN)
    z = (z ^ _lsr(z, 30)) * _i64(_C1)
    z = (z ^ _lsr(z, 27)) * _i64(_C2)
    return z ^ _lsr(z, 31)


_SLAB_WORDS = 1 << 24   # 64-bit words generated per step (128 MiB of int64)


def fill_uniform_bytes(out: torch.Tensor, seed: int) -> torch.Tensor:
    """Fills the 1-D uint8 tensor `out` with uniform random bytes; byte 8k..8k+7 = mix64(k)."""
    assert out.dtype == torch.uint8 and out.dim() == 1 and out.is_contiguous()
    n = out.numel()
    words = (n + 7) // 8
    for w0 in range(0, words, _SLAB_WORDS):
        cnt = min(_SLAB_WORDS, words - w0)
        raw = mix64(w0, cnt, seed, out.device).view(torch.uint8)
        lo, hi = 8 * w0, min(8 * (w0 + cnt), n)
        out[lo:hi] = raw[:hi - lo]
    return out


def uniform_bytes(nbytes: int, seed: int, device="cpu") -> torch.Tensor:
    return fill_uniform_bytes(torch.empty(nbytes, dtype=torch.uint8, device=device), seed)


_IH_STD = math.sqrt(4 * (256 ** 2 - 1) / 12.0)   # std of the sum of four uniform bytes


def fill_bf16_normal(out: torch.Tensor, seed: int, std: float = 0.02, first_elem: int = 0) -> torch.Tensor:
    """Fills the uint8 tensor `out` (even length) with bf16 values ~N(0, std).

    Element e (two bytes) comes from the four bytes of half e%2 of mix64(e//2); `first_elem`
    (even) is the index of out's first element within the whole stream, so a blob can be
    generated piecewise."""
    assert out.dtype == torch.uint8 and out.dim() == 1 and out.is_contiguous()
    assert out.numel() % 2 == 0 and first_elem % 2 == 0
    n_elem = out.numel() // 2
    words = (n_elem + 1) // 2
    w_first = first_elem // 2
    scale = torch.tensor(std / _IH_STD, dtype=torch.float32, device=out.device)
    for w0 in range(0, words, _SLAB_WORDS):
        cnt = min(_SLAB_WORDS, words - w0)
        raw = mix64(w_first + w0, cnt, seed, out.device).view(torch.uint8).view(cnt * 2, 4)
        s = raw.sum(dim=1, dtype=torch.int32) - 510                 # Irwin-Hall(4), centred (twice the mean 255)
        vals = (s.to(torch.float32) * scale).to(torch.bfloat16).view(torch.uint8)
        lo, hi = 4 * w0, min(4 * (w0 + cnt), 2 * n_elem)
        out[lo:hi] = vals[:hi - lo]
    return out


def bf16_normal_bytes(n_params: int, seed: int, device="cpu", std: float = 0.02) -> torch.Tensor:
    return fill_bf16_normal(torch.empty(2 * n_params, dtype=torch.uint8, device=device), seed, std)


# ---------------------------------------------------------------------------------------------
# weight files

def gpt_1p3b_tensors() -> list[tuple[str, tuple[int, ...]]]:
    """24 layers, hidden 2048, FFN 8192, vocabulary 50257: about 1.31e9 parameters."""
    h, f, v, layers = 2048, 8192, 50257, 24
    t = [("wte.weight", (v, h))]
    for i in range(layers):
        p = f"h.{i}."
        t += [(p + "ln_1.weight", (h,)), (p + "attn.q.weight", (h, h)), (p + "attn.k.weight", (h, h)),
              (p + "attn.v.weight", (h, h)), (p + "attn.o.weight", (h, h)), (p + "ln_2.weight", (h,)),
              (p + "mlp.fc.weight", (f, h)), (p + "mlp.proj.weight", (h, f))]
    t.append(("ln_f.weight", (h,)))
    return t


def llama_8b_tensors() -> list[tuple[str, tuple[int, ...]]]:
    """32 layers, hidden 4096, FFN 14336, 8 KV heads of 128, vocabulary 128256: 8,030,261,248 parameters."""
    h, f, kv, v, layers = 4096, 14336, 1024, 128256, 32
    t = [("embed_tokens.weight", (v, h))]
    for i in range(layers):
        p = f"layers.{i}."
        t += [(p + "input_layernorm.weight", (h,)), (p + "q_proj.weight", (h, h)), (p + "k_proj.weight", (kv, h)),
              (p + "v_proj.weight", (kv, h)), (p + "o_proj.weight", (h, h)),
              (p + "post_attention_layernorm.weight", (h,)), (p + "gate_proj.weight", (f, h)),
              (p + "up_proj.weight", (f, h)), (p + "down_proj.weight", (h, f))]
    t += [("norm.weight", (h,)), ("lm_head.weight", (v, h))]
    return t


def tiny_tensors(layers: int = 2, h: int = 64, f: int = 160, v: int = 301) -> list[tuple[str, tuple[int, ...]]]:
    """A few-hundred-KB layer list with the same structure, for tests."""
    t = [("embed.weight", (v, h))]
    for i in range(layers):
        p = f"layers.{i}."
        t += [(p + "norm.weight", (h,)), (p + "q.weight", (h, h)), (p + "k.weight", (h // 4, h)),
              (p + "up.weight", (f, h)), (p + "down.weight", (h, f))]
    t.append(("norm.weight", (h,)))
    return t


def weight_file_layout(tensors: list[tuple[str, tuple[int, ...]]]):
    """Header bytes and the (name, absolute offset, byte length) table of a bf16 weight file."""
    index, off = {}, 0
    for name, shape in tensors:
        nbytes = 2 * math.prod(shape)
        index[name] = {"dtype": "BF16", "shape": list(shape), "data_offsets": [off, off + nbytes]}
        off += nbytes
    text = json.dumps(index, separators=(",", ":")).encode("ascii")
    text += b" " * (-len(text) % 8)
    header = struct.pack("<Q", len(text)) + text
    table = [(name, len(header) + e["data_offsets"][0], e["data_offsets"][1] - e["data_offsets"][0])
             for name, e in index.items()]
    return header, table, len(header) + off


def weight_file(tensors, seed: int, device="cpu"):
    """The whole file as a uint8 tensor on `device`, plus the tensor table.

    The total is padded by at most one byte so that the data region starts on an even
    offset inside an even-length buffer (bf16 elements)."""
    header, table, total = weight_file_layout(tensors)
    blob = torch.empty(total, dtype=torch.uint8, device=device)
    blob[:len(header)] = torch.frombuffer(bytearray(header), dtype=torch.uint8).to(device)
    fill_bf16_normal(blob[len(header):], seed)
    return blob, table


# ---------------------------------------------------------------------------------------------
# ragged tensor set

def ragged_sizes(n: int = 10_000, lo_bytes: int = 4096, hi_bytes: int = 64 << 20, seed: int = 5) -> np.ndarray:
    """n even byte sizes, log-uniform in [lo_bytes, hi_bytes]."""
    rng = np.random.default_rng(seed)
    half = np.exp(rng.uniform(math.log(lo_bytes / 2), math.log(hi_bytes / 2), size=n))
    sizes = 2 * np.rint(half).astype(np.int64)
    return np.clip(sizes, lo_bytes, hi_bytes)


def packed_offsets(sizes: np.ndarray, first: int = 0) -> np.ndarray:
    """Offsets of tensors packed back to back starting at byte `first`."""
    off = np.empty_like(sizes)
    off[0:1] = first
    np.cumsum(sizes[:-1], out=off[1:])
    off[1:] += first
    return off


def flip_position(seed: int, nbytes: int) -> tuple[int, int]:
    """A seeded (byte offset, bit) inside a blob of nbytes."""
    rng = np.random.default_rng(seed)
    return int(rng.integers(0, nbytes)), int(rng.integers(0, 8))
