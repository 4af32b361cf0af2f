"""GPU parity of the RFC 6962 section 2.1 mode (0x00-prefixed leaf hashes, 0x01-prefixed nodes): leaf
hashes and roots from the CUDA library equal the CPU oracle's bit for bit.  All calls go through the
C ABI via the ctypes binding."""
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
    (1 << 20, 4096), (1 << 20, 64), (1 << 20, 1 << 20), (1 << 20, 2 << 20),
    ((1 << 20) + 77, 4096),
    (100_003, 1000), (100_003, 1001), (100_003, 7), (65, 64), (64, 64), (63, 64), (62, 64), (1, 1),
    # last-chunk lengths around the padding boundaries of the message that is one byte longer
    (5 * 4096 + 54, 4096), (5 * 4096 + 55, 4096), (5 * 4096 + 56, 4096),
    (5 * 4096 + 62, 4096), (5 * 4096 + 63, 4096), (5 * 4096 + 64, 4096),
    (5 * 4096 + 118, 4096), (5 * 4096 + 119, 4096), (5 * 4096 + 127, 4096),
    (37 * 48 + 16, 48),
    (20_000 * 4096 + 100, 4096),          # the migrating kernel (more than 296 warps), short last chunk beside it
    (19_000 * 4096, 4096),
    (9_600 * 65536, 65536),               # several slices per chunk: the carried word crosses slice borders
    (9_600 * 65536 + 63, 65536), (9_500 * (65536 + 16), 65536 + 16),    (60_000 * 4096 + 100, 4096), (57_000 * 16384, 16384),   # 12 or more groups per SM: the twelve-worker instance
    (9_600 * 4096 + 100, 4096), (13_450 * 8192, 8192), (9_473 * 32768 - 32700, 32768),   # the two-warp pairs on the FIFO
])
def test_leaf_hashes_equal_oracle(ctx, nbytes, chunk):
    data = inputs.uniform_bytes(nbytes, seed=6962, device="cuda")
    got = ctx.hash_chunks_rfc6962(data, chunk)
    groups = -(-binding.n_chunks(nbytes, chunk) // 32)
    if chunk >= 4096 and chunk % 16 == 0 and 296 < groups < 422:
        assert ctx.last_leaf_kernel == "hash_chunks_pairs_kernel"
    if chunk >= 4096 and chunk % 16 == 0 and groups <= 296:
        assert ctx.last_leaf_kernel == "hash_chunks_split_kernel"
    want = oracle.hash_chunks_rfc6962(_host(data), chunk, nthreads=oracle.host_threads())
    assert got.shape == want.shape
    assert np.array_equal(_host(got), want)


@pytest.mark.parametrize("shift", [1, 3, 8, 13])
@pytest.mark.parametrize("chunk", [256, 1000, 4096 + 3])
def test_leaf_hashes_any_base_alignment(ctx, shift, chunk):
    buf = inputs.uniform_bytes(300_000 + 16, seed=6963, device="cuda")
    data = buf[shift:shift + 300_000]
    got = ctx.hash_chunks_rfc6962(data, chunk)
    assert np.array_equal(_host(got), oracle.hash_chunks_rfc6962(_host(data), chunk))


def test_every_entry_length_of_three_blocks(ctx):
    buf = inputs.uniform_bytes(208, seed=6964, device="cuda")          # 16-byte aligned base, any length
    host = _host(buf)
    for n in range(1, 193):
        for off in (0, 16):
            got = ctx.hash_chunks_rfc6962(buf[off:off + n], 256)
            assert np.array_equal(_host(got), oracle.hash_chunks_rfc6962(host[off:off + n], 256)), (n, off)


def test_empty_and_argument_errors(ctx):
    empty = torch.empty(0, dtype=torch.uint8, device="cuda")
    assert ctx.hash_chunks_rfc6962(empty, 4096).shape == (0, 32)
    with pytest.raises(binding.IvError):
        ctx.hash_chunks_rfc6962(inputs.uniform_bytes(100, seed=1, device="cuda"), 0)


@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 7, 8, 9, 127, 128, 129, 1000, 1023, 1024, 1025, 40_001])
def test_root_equals_oracle(ctx, n):
    leaves = inputs.uniform_bytes(32 * n, seed=6965 + n, device="cuda").reshape(n, 32)
    got = _host(ctx.merkle_root_rfc6962(leaves)).tobytes()
    assert got == oracle.merkle_root_rfc6962(_host(leaves))


def test_root_unaligned_leaf_pointer(ctx):
    buf = inputs.uniform_bytes(32 * 77 + 5, seed=6966, device="cuda")
    leaves = buf[5:]
    assert _host(ctx.merkle_root_rfc6962(leaves)).tobytes() == oracle.merkle_root_rfc6962(_host(leaves))


def test_leaves_then_root_differs_from_the_default_path_and_repeats(ctx):
    data = inputs.uniform_bytes((8 << 20) + 5, seed=6967, device="cuda")
    want_leaves = oracle.hash_chunks_rfc6962(_host(data), 4096, nthreads=oracle.host_threads())
    want_root = oracle.merkle_root_rfc6962(want_leaves)
    for _ in range(3):
        leaves = ctx.hash_chunks_rfc6962(data, 4096)
        assert _host(ctx.merkle_root_rfc6962(leaves)).tobytes() == want_root
    assert _host(ctx.merkle_root(ctx.hash_chunks(data, 4096))).tobytes() != want_root
    assert ctx.device_status() == 0


def test_verification_in_this_mode_against_a_manifest_from_the_oracle(ctx):
    """Manifest = the oracle's prefixed leaf hashes and root; clean data passes, flipped bits are located, and a
    manifest of the default (unprefixed) path is rejected on every chunk."""
    nbytes, chunk = (8 << 20) + 300, 4096
    data = inputs.uniform_bytes(nbytes, seed=6970, device="cuda")
    leaves = oracle.hash_chunks_rfc6962(_host(data), chunk, nthreads=oracle.host_threads())
    root = oracle.merkle_root_rfc6962(leaves)
    manifest = ctx.make_manifest(nbytes, chunk, torch.from_numpy(leaves).cuda(), root)
    n = leaves.shape[0]

    def verify(blob, man, cap=16):
        res = binding.new_result("cuda")
        idx = torch.zeros(cap, dtype=torch.int64, device="cuda")
        ctx.verify_manifest_rfc6962(blob, man, res, idx)
        r = binding.read_result(res)
        return r, [int(v) for v in idx[:min(cap, r["n_mismatch"])].cpu()]

    r, idx = verify(data, manifest)
    assert r == {"status": 0, "root_ok": True, "n_mismatch": 0, "root": root} and idx == []
    bad = data.clone()
    flips = sorted({inputs.flip_position(s, nbytes) for s in (5, 6, 7)})
    for off, bit in flips:
        bad[off] ^= (1 << bit)
    want_leaves = oracle.hash_chunks_rfc6962(_host(bad), chunk, nthreads=oracle.host_threads())
    want_idx = [i for i in range(n) if bytes(want_leaves[i]) != bytes(leaves[i])]
    r, idx = verify(bad, manifest)
    assert idx == want_idx == sorted({off // chunk for off, _ in flips})
    assert r["n_mismatch"] == len(want_idx) and not r["root_ok"]
    assert r["root"] == oracle.merkle_root_rfc6962(want_leaves)
    # the default path's manifest does not verify in this mode
    plain = oracle.hash_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    plain_manifest = ctx.make_manifest(nbytes, chunk, torch.from_numpy(plain).cuda(), oracle.merkle_root(plain))
    r, idx = verify(data, plain_manifest, cap=4)
    assert r["n_mismatch"] == n and not r["root_ok"] and idx == [0, 1, 2, 3]
