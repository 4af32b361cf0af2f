"""GPU parity of the SHA-384 and SHA-512 variants (FIPS 180-4 sections 6.4 and 6.5; SHA-384 is the digest of
the paper's kernel listings): chunk digests and tree roots from the CUDA library equal the CPU oracle's bit
for bit.  All calls go through the C ABI via the ctypes binding."""
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


class _Variant:
    def __init__(self, name, rec):
        self.name, self.rec = name, rec

    def gpu_chunks(self, ctx, data, chunk):
        return getattr(ctx, f"hash_chunks_{self.name}")(data, chunk)

    def gpu_root(self, ctx, leaves):
        return getattr(ctx, f"merkle_root_{self.name}")(leaves)

    def cpu_chunks(self, host, chunk, nthreads=1):
        return getattr(oracle, f"hash_chunks_{self.name}")(host, chunk, nthreads=nthreads)

    def cpu_root(self, leaves):
        return getattr(oracle, f"merkle_root_{self.name}")(leaves)

    def cpu_hash(self, msg):
        return getattr(oracle, self.name)(msg)

    def __repr__(self):
        return self.name


VARIANTS = [_Variant("sha384", 48), _Variant("sha512", 64)]


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
    # the two-warp kernel: one group, one chunk, one group and a lane; more groups than worker pairs (888 on
    # 148 SMs); many slices per chunk (1 MiB: 64, 4 MiB: 256); the last slice shorter than the others
    (32 * 16384, 16384), (16384, 16384), (33 * 16384, 16384), (30_000 * 16384, 16384), (40 * (1 << 20), 1 << 20),
    (36 * (4 << 20) + 4096, 4 << 20), (70 * (20480 + 48), 20480 + 48), (150 * (5 * 16384 - 128), 5 * 16384 - 128),
    (500 * 32 * 16384, 16384), (4096 * 32 * 16384, 16384),       # group counts the plain kernel keeps
    # the launch shapes of the two-warp kernel on 148 SMs: eight pairs per SM (1,200 groups of 128 KiB chunks; 2,075
    # groups of 64 KiB chunks), four (1,300 and 625 groups), two (below 444 groups: most shapes above); chunks
    # below 64 KiB with many groups go to the plain kernel
    (38_400 * 131072, 131072), (66_400 * 65536, 65536), (41_600 * 65536, 65536), (20_000 * (65536 + 48), 65536 + 48),
    (64_000 * (16384 + 48), 16384 + 48),
])
@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_hash_chunks_equals_oracle(ctx, variant, nbytes, chunk):
    data = inputs.uniform_bytes(nbytes, seed=384, device="cuda")
    got = variant.gpu_chunks(ctx, data, chunk)
    groups = -(-(nbytes // chunk) // 32)
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    pairs_take_it = chunk >= 16384 and chunk % 16 == 0 and nbytes >= chunk and (
        groups < 3 * sms if chunk < 65536 else groups < 4096 if chunk < 262144 else True)
    if pairs_take_it:
        assert ctx.last_leaf_kernel == "hash_sha512_pairs_kernel"
        pairs = (2 if groups < 3 * sms else 8 if groups >= 8 * sms and (chunk >= 131072 or groups >= 14 * sms)
                 else 6 if groups >= 6 * sms and chunk >= (1 << 20) else 4)
        assert ctx.last_leaf_instance == f"{pairs} pairs per SM"
    else:
        assert ctx.last_leaf_kernel == "hash_chunks_sha384_kernel"
        assert ctx.last_leaf_instance == ""
    want = variant.cpu_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    assert got.shape == want.shape
    assert np.array_equal(_host(got), want)
    assert ctx.device_status() == 0


@pytest.mark.parametrize("shift", [1, 3, 8, 13])
@pytest.mark.parametrize("chunk", [256, 1000, 4096 + 3, 16384])
@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_hash_chunks_any_base_alignment(ctx, variant, shift, chunk):
    buf = inputs.uniform_bytes(300_000 + 16, seed=385, device="cuda")
    data = buf[shift:shift + 300_000]
    got = variant.gpu_chunks(ctx, data, chunk)
    assert ctx.last_leaf_kernel == "hash_chunks_sha384_kernel"
    assert np.array_equal(_host(got), variant.cpu_chunks(_host(data), chunk))


@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_hash_chunks_every_tail_length_of_two_blocks(ctx, variant):
    # one message per length 0..256 through the chunk entry point: the padding cases of section 5.1.2
    buf = inputs.uniform_bytes(257, seed=386, device="cuda")
    host = _host(buf)
    for n in range(1, 257):
        got = variant.gpu_chunks(ctx, buf[:n], 512)
        assert _host(got).tobytes() == variant.cpu_hash(host[:n]), n


@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_two_warp_kernel_every_chunk_remainder(ctx, variant):
    """Chunks of 16384 + r bytes for r = 0, 16, ..., 112 and beyond: the tail (remainder + padding) the producer
    builds behind the tiled copies, on both sides of the one-block / two-block padding boundary."""
    for r in range(0, 256, 16):
        chunk = 16384 + r
        data = inputs.uniform_bytes(45 * chunk, seed=390 + r, device="cuda")
        got = variant.gpu_chunks(ctx, data, chunk)
        assert ctx.last_leaf_kernel == "hash_sha512_pairs_kernel"
        assert np.array_equal(_host(got), variant.cpu_chunks(_host(data), chunk)), r
    assert ctx.device_status() == 0


@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_hash_chunks_empty_and_argument_errors(ctx, variant):
    empty = torch.empty(0, dtype=torch.uint8, device="cuda")
    assert variant.gpu_chunks(ctx, empty, 4096).shape == (0, variant.rec)
    with pytest.raises(binding.IvError):
        variant.gpu_chunks(ctx, inputs.uniform_bytes(100, seed=1, device="cuda"), 0)


@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 7, 8, 9, 127, 128, 129, 1000, 1023, 1024, 1025, 40_001])
@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_merkle_root_equals_oracle(ctx, variant, n):
    leaves = inputs.uniform_bytes(variant.rec * n, seed=387 + n, device="cuda").reshape(n, variant.rec)
    got = _host(variant.gpu_root(ctx, leaves)).tobytes()
    assert got == variant.cpu_root(_host(leaves))


@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_chunks_then_root_repeated_calls(ctx, variant):
    data = inputs.uniform_bytes((8 << 20) + 5, seed=388, device="cuda")
    want_leaves = variant.cpu_chunks(_host(data), 4096, nthreads=oracle.host_threads())
    want_root = variant.cpu_root(want_leaves)
    for _ in range(3):
        leaves = variant.gpu_chunks(ctx, data, 4096)
        assert _host(variant.gpu_root(ctx, leaves)).tobytes() == want_root
    # a smaller tree after a larger one reuses the level buffers
    assert _host(variant.gpu_root(ctx, leaves[:5].contiguous())).tobytes() == variant.cpu_root(want_leaves[:5])
    assert ctx.device_status() == 0


@pytest.mark.parametrize("nbytes,chunk", [((8 << 20) + 300, 4096), (64 << 20, 64 << 10), (100_003, 1001), (5000, 8192)])
@pytest.mark.parametrize("variant", VARIANTS, ids=repr)
def test_verification_against_a_manifest_from_the_oracle(ctx, variant, nbytes, chunk):
    """Manifest = the oracle's SHA-384 / SHA-512 chunk digests and root: clean data passes, flipped bits are located in
    ascending order with the exact count, the recomputed root is the oracle's root of the damaged blob."""
    data = inputs.uniform_bytes(nbytes, seed=3840, device="cuda")
    digests = variant.cpu_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    root = variant.cpu_root(digests)
    d_digests = torch.from_numpy(digests).cuda()
    verify = getattr(ctx, f"verify_manifest_{variant.name}")
    n = digests.shape[0]
    idx = torch.zeros(4, dtype=torch.int64, device="cuda")
    r = verify(data, nbytes, chunk, d_digests, root, idx)
    assert r == {"status": 0, "root_ok": True, "n_mismatch": 0, "root": root}
    bad = data.clone()
    hits = sorted({inputs.flip_position(s, nbytes) for s in range(11, 18)})
    for off, bit in hits:
        bad[off] ^= (1 << bit)
    want = variant.cpu_chunks(_host(bad), chunk, nthreads=oracle.host_threads())
    want_idx = [i for i in range(n) if bytes(want[i]) != bytes(digests[i])]
    assert want_idx == sorted({off // chunk for off, _ in hits})
    r = verify(bad, nbytes, chunk, d_digests, root, idx)
    assert (not r["root_ok"]) and r["n_mismatch"] == len(want_idx) and r["root"] == variant.cpu_root(want)
    assert [int(v) for v in idx[:min(4, len(want_idx))].cpu()] == want_idx[:4]
    # manifest-side damage: one digest of the manifest changed, the data clean
    d_digests[n // 2, 7] ^= 1
    r = verify(data, nbytes, chunk, d_digests, root, idx)
    assert r["root_ok"] and r["n_mismatch"] == 1 and int(idx[0]) == n // 2
    with pytest.raises(binding.IvError):
        verify(data, nbytes + 1, chunk, d_digests, root, idx)
    assert ctx.device_status() == 0
