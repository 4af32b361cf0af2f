"""Seeded random shapes through every hashing entry point, each result compared with the CPU oracle
bit for bit: blob sizes, chunk sizes (odd ones, multiples of 16, of 64, of 4096), base alignments, leaf
counts and tensor sets that no hand-written case lists.  All calls go through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_23938_b200 import binding, inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    if not torch.cuda.is_available():
        pytest.fail("the gpu-marked tests need a CUDA device")
    c = binding.Context(0)
    yield c
    c.close()


def _host(t):
    return t.cpu().numpy()


def _cases(seed, count):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(count):
        kind = int(rng.integers(0, 5))
        if kind == 0:      # any chunk size
            chunk = int(rng.integers(1, 70_000))
        elif kind == 1:    # multiple of 16
            chunk = 16 * int(rng.integers(1, 5_000))
        elif kind == 2:    # multiple of 64
            chunk = 64 * int(rng.integers(1, 2_000))
        elif kind == 3:    # multiple of 4096 (the two-warp and migrating kernels)
            chunk = 4096 * int(rng.integers(1, 40))
        else:              # small chunks, many chains
            chunk = int(rng.integers(1, 300))
        n_chunks = int(rng.integers(1, 400 if chunk > 5000 else 3000))
        tail = int(rng.integers(0, chunk)) if rng.integers(0, 2) else 0
        nbytes = max(1, (n_chunks - 1) * chunk + (tail if tail else chunk))
        shift = int(rng.integers(0, 16)) if rng.integers(0, 3) == 0 else 0
        out.append((nbytes, chunk, shift))
    return out


@pytest.mark.parametrize("block", range(6))
def test_chunk_digests_and_roots_of_random_shapes(ctx, block):
    for nbytes, chunk, shift in _cases(100 + block, 12):
        buf = inputs.uniform_bytes(nbytes + 16, seed=7 * nbytes + chunk, device="cuda")
        data = buf[shift:shift + nbytes]
        host = _host(data)
        tag = (nbytes, chunk, shift)
        got = ctx.hash_chunks(data, chunk)
        want = oracle.hash_chunks(host, chunk, nthreads=oracle.host_threads())
        assert np.array_equal(_host(got), want), ("sha256", tag, ctx.last_leaf_kernel)
        assert _host(ctx.merkle_root(got)).tobytes() == oracle.merkle_root(want), ("root", tag)
        got = ctx.hash_chunks_rfc6962(data, chunk)
        want = oracle.hash_chunks_rfc6962(host, chunk, nthreads=oracle.host_threads())
        assert np.array_equal(_host(got), want), ("rfc6962", tag, ctx.last_leaf_kernel)
        assert _host(ctx.merkle_root_rfc6962(got)).tobytes() == oracle.merkle_root_rfc6962(want), ("rfc root", tag)
        got = ctx.hash_chunks_sha384(data, chunk)
        want = oracle.hash_chunks_sha384(host, chunk, nthreads=oracle.host_threads())
        assert np.array_equal(_host(got), want), ("sha384", tag)
        assert _host(ctx.merkle_root_sha384(got)).tobytes() == oracle.merkle_root_sha384(want), ("sha384 root", tag)
    assert ctx.device_status() == 0


def test_migrating_kernel_on_random_large_shapes(ctx):
    """More than 296 warps of chains with chunk sizes that are multiples of 16 bytes and at least 4 KiB: the
    shapes of the two kernels that hand chains from worker to worker through the slice FIFO."""
    rng = np.random.default_rng(77)
    for _ in range(6):
        chunk = 16 * int(rng.integers(256, 6_000))
        n_chunks = int(rng.integers(9_500, 14_000))
        tail = int(rng.integers(1, chunk))
        nbytes = (n_chunks - 1) * chunk + tail
        data = inputs.uniform_bytes(nbytes, seed=nbytes, device="cuda")
        host = _host(data)
        got = ctx.hash_chunks(data, chunk)
        assert ctx.last_leaf_kernel in ("hash_chunks_sliced_kernel", "hash_chunks_pairs_kernel")
        assert np.array_equal(_host(got), oracle.hash_chunks(host, chunk, nthreads=oracle.host_threads())), (nbytes, chunk)
        got = ctx.hash_chunks_rfc6962(data, chunk)
        assert ctx.last_leaf_kernel in ("hash_chunks_sliced_kernel", "hash_chunks_pairs_kernel")
        assert np.array_equal(_host(got), oracle.hash_chunks_rfc6962(host, chunk, nthreads=oracle.host_threads())), (nbytes, chunk)
        got = ctx.hash_chunks_sha384(data, chunk)
        assert np.array_equal(_host(got), oracle.hash_chunks_sha384(host, chunk, nthreads=oracle.host_threads())), (nbytes, chunk)
        del data
    assert ctx.device_status() == 0


def test_sha384_and_sha512_two_warp_kernel_on_random_shapes(ctx):
    """Random group counts from one warp's worth of chains to more groups than worker pairs, chunk sizes of 16 KiB
    to 600 KiB that are multiples of 16 bytes (any remainder mod 128: every tail the producer builds; slice counts
    from 1 to 37), a short last chunk: the shapes of the SHA-384 / SHA-512 kernel on the slice FIFO."""
    rng = np.random.default_rng(512)
    seen = set()
    for k in range(10):
        chunk = 16 * int(rng.integers(1024, 38_000)) if k % 3 else 16 * int(rng.integers(1024, 2_100))
        budget = 700 << 20
        n_chunks = int(rng.integers(1, max(2, min(40_000, budget // chunk))))
        tail = int(rng.integers(1, chunk + 1))
        nbytes = (n_chunks - 1) * chunk + tail
        data = inputs.uniform_bytes(nbytes, seed=nbytes, device="cuda")
        host = _host(data)
        got = ctx.hash_chunks_sha384(data, chunk)
        seen.add(ctx.last_leaf_kernel)
        assert np.array_equal(_host(got), oracle.hash_chunks_sha384(host, chunk, nthreads=oracle.host_threads())), (nbytes, chunk)
        got = ctx.hash_chunks_sha512(data, chunk)
        assert np.array_equal(_host(got), oracle.hash_chunks_sha512(host, chunk, nthreads=oracle.host_threads())), (nbytes, chunk)
        assert _host(ctx.merkle_root_sha512(got)).tobytes() == oracle.merkle_root_sha512(_host(got)), (nbytes, chunk)
        del data
    assert "hash_sha512_pairs_kernel" in seen
    assert ctx.device_status() == 0


def test_sha384_and_sha512_two_warp_kernel_with_many_groups(ctx):
    """Random shapes with three and more groups of 32 chains per SM, where the two-warp kernel runs four or eight
    pairs per SM (or hands short chunks to the one-chain-per-lane kernel): chunks of 16 KiB to 192 KiB (multiples of
    16 bytes), a ragged last group, a short last chunk half of the time, a base that is shifted by 16-byte steps."""
    rng = np.random.default_rng(513)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    buf = inputs.uniform_bytes((2 << 30) + 1024, seed=513, device="cuda")
    seen = set()
    for k in range(8):
        chunk = 16 * int(rng.integers(1024, 12_288))
        groups = int(rng.integers(3 * sms + 1, 17 * sms))
        n_chunks = groups * 32 - int(rng.integers(0, 32))
        while chunk * n_chunks > (2 << 30):
            n_chunks = n_chunks * 3 // 4
        tail = int(rng.integers(1, chunk + 1)) if k % 2 else chunk
        nbytes = (n_chunks - 1) * chunk + tail
        shift = 16 * int(rng.integers(0, 64))
        data = buf[shift:shift + nbytes]
        host = _host(data)
        got = ctx.hash_chunks_sha384(data, chunk)
        seen.add(ctx.last_leaf_kernel + " " + ctx.last_leaf_instance)
        assert np.array_equal(_host(got), oracle.hash_chunks_sha384(host, chunk, nthreads=oracle.host_threads())), (nbytes, chunk, shift)
        got = ctx.hash_chunks_sha512(data, chunk)
        assert np.array_equal(_host(got), oracle.hash_chunks_sha512(host, chunk, nthreads=oracle.host_threads())), (nbytes, chunk, shift)
    assert "hash_sha512_pairs_kernel 4 pairs per SM" in seen, seen
    assert ctx.device_status() == 0


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_tensor_sets(ctx, seed):
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.integers(1, 600))
    lens = np.where(rng.integers(0, 4, size=n) == 0, rng.integers(0, 200, size=n), rng.integers(0, 60_000, size=n)).astype(np.int64)
    gaps = rng.integers(0, 9, size=n).astype(np.int64)
    offs = np.cumsum(gaps + np.concatenate([[0], lens[:-1]])).astype(np.int64)
    total = int(offs[-1] + lens[-1]) + 16
    base = inputs.uniform_bytes(total, seed=seed, device="cuda")
    got = ctx.hash_ragged(base, torch.from_numpy(offs).cuda(), torch.from_numpy(lens).cuda())
    want = oracle.hash_ragged(_host(base), offs.astype(np.uint64), lens.astype(np.uint64), nthreads=oracle.host_threads())
    assert np.array_equal(_host(got), want)
    assert ctx.device_status() == 0
