"""GPU parity of the SHA-384 variant (FIPS 180-4 section 6.5; the digest of the paper's kernel
listings): chunk digests and tree roots from the CUDA library equal the CPU oracle's bit for bit.
All calls go through the C ABI via the ctypes binding."""
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


def _host(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy()


@pytest.mark.parametrize("nbytes,chunk", [
    (64 << 20, 64 << 10),                 # the small configuration
    (1 << 20, 4096), (1 << 20, 128), (1 << 20, 1 << 20), (1 << 20, 2 << 20),
    ((1 << 20) + 77, 4096),               # ragged last chunk
    (100_003, 1000), (100_003, 1001), (100_003, 7), (129, 128), (128, 128), (127, 128), (1, 1),
    # remainders around the one-block / two-block padding boundary (111 | 112 bytes)
    (5 * 4096 + 111, 4096), (5 * 4096 + 112, 4096), (5 * 4096 + 239, 4096), (5 * 4096 + 240, 4096),
    (37 * 48 + 16, 48),                   # multiple of 16 but not of 128
    (20_000 * 4096 + 100, 4096),          # several waves of warps, short last chunk
    (19_000 * 4096, 4096),
    (9_600 * 65536, 65536),               # larger chunks, many chains
    (9_600 * 65536 + 127, 65536), (9_500 * (65536 + 16), 65536 + 16), (9_500 * (65536 + 112), 65536 + 112),
])
def test_hash_chunks_sha384_equals_oracle(ctx, nbytes, chunk):
    data = inputs.uniform_bytes(nbytes, seed=384, device="cuda")
    got = ctx.hash_chunks_sha384(data, chunk)
    want = oracle.hash_chunks_sha384(_host(data), chunk, nthreads=oracle.host_threads())
    assert got.shape == want.shape
    assert np.array_equal(_host(got), want)


@pytest.mark.parametrize("shift", [1, 3, 8, 13])
@pytest.mark.parametrize("chunk", [256, 1000, 4096 + 3])
def test_hash_chunks_sha384_any_base_alignment(ctx, shift, chunk):
    buf = inputs.uniform_bytes(300_000 + 16, seed=385, device="cuda")
    data = buf[shift:shift + 300_000]
    got = ctx.hash_chunks_sha384(data, chunk)
    assert np.array_equal(_host(got), oracle.hash_chunks_sha384(_host(data), chunk))


def test_hash_chunks_sha384_every_tail_length_of_two_blocks(ctx):
    # one message per length 0..256 through the chunk entry point: the padding cases of section 5.1.2
    buf = inputs.uniform_bytes(257, seed=386, device="cuda")
    host = _host(buf)
    for n in range(1, 257):
        got = ctx.hash_chunks_sha384(buf[:n], 512)
        assert _host(got).tobytes() == oracle.sha384(host[:n]), n


def test_hash_chunks_sha384_empty_and_argument_errors(ctx):
    empty = torch.empty(0, dtype=torch.uint8, device="cuda")
    assert ctx.hash_chunks_sha384(empty, 4096).shape == (0, 48)
    with pytest.raises(binding.IvError):
        ctx.hash_chunks_sha384(inputs.uniform_bytes(100, seed=1, device="cuda"), 0)


@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 7, 8, 9, 127, 128, 129, 1000, 1023, 1024, 1025, 40_001])
def test_merkle_root_sha384_equals_oracle(ctx, n):
    leaves = inputs.uniform_bytes(48 * n, seed=387 + n, device="cuda").reshape(n, 48)
    got = _host(ctx.merkle_root_sha384(leaves)).tobytes()
    assert got == oracle.merkle_root_sha384(_host(leaves))


def test_sha384_chunks_then_root_repeated_calls(ctx):
    data = inputs.uniform_bytes((8 << 20) + 5, seed=388, device="cuda")
    want_leaves = oracle.hash_chunks_sha384(_host(data), 4096, nthreads=oracle.host_threads())
    want_root = oracle.merkle_root_sha384(want_leaves)
    for _ in range(3):
        leaves = ctx.hash_chunks_sha384(data, 4096)
        assert _host(ctx.merkle_root_sha384(leaves)).tobytes() == want_root
    # a smaller tree after a larger one reuses the level buffers
    assert _host(ctx.merkle_root_sha384(leaves[:5])).tobytes() == oracle.merkle_root_sha384(want_leaves[:5])
    assert ctx.device_status() == 0


@pytest.mark.parametrize("nbytes,chunk", [((8 << 20) + 300, 4096), (64 << 20, 64 << 10), (100_003, 1001), (5000, 8192)])
def test_verification_against_a_sha384_manifest_from_the_oracle(ctx, nbytes, chunk):
    """Manifest = the oracle's SHA-384 chunk digests and root: clean data passes, flipped bits are located in
    ascending order with the exact count, the recomputed root is the oracle's root of the damaged blob."""
    data = inputs.uniform_bytes(nbytes, seed=3840, device="cuda")
    digests = oracle.hash_chunks_sha384(_host(data), chunk, nthreads=oracle.host_threads())
    root = oracle.merkle_root_sha384(digests)
    d_digests = torch.from_numpy(digests).cuda()
    n = digests.shape[0]
    idx = torch.zeros(4, dtype=torch.int64, device="cuda")
    r = ctx.verify_manifest_sha384(data, nbytes, chunk, d_digests, root, idx)
    assert r == {"status": 0, "root_ok": True, "n_mismatch": 0, "root": root}
    bad = data.clone()
    hits = sorted({inputs.flip_position(s, nbytes) for s in range(11, 18)})
    for off, bit in hits:
        bad[off] ^= (1 << bit)
    want = oracle.hash_chunks_sha384(_host(bad), chunk, nthreads=oracle.host_threads())
    want_idx = [i for i in range(n) if bytes(want[i]) != bytes(digests[i])]
    assert want_idx == sorted({off // chunk for off, _ in hits})
    r = ctx.verify_manifest_sha384(bad, nbytes, chunk, d_digests, root, idx)
    assert (not r["root_ok"]) and r["n_mismatch"] == len(want_idx) and r["root"] == oracle.merkle_root_sha384(want)
    assert [int(v) for v in idx[:min(4, len(want_idx))].cpu()] == want_idx[:4]
    # manifest-side damage: one digest of the manifest changed, the data clean
    d_digests[n // 2, 7] ^= 1
    r = ctx.verify_manifest_sha384(data, nbytes, chunk, d_digests, root, idx)
    assert r["root_ok"] and r["n_mismatch"] == 1 and int(idx[0]) == n // 2
    with pytest.raises(binding.IvError):
        ctx.verify_manifest_sha384(data, nbytes + 1, chunk, d_digests, root, idx)
    assert ctx.device_status() == 0
