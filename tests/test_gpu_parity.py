"""GPU parity: every digest, root, count and index from the CUDA library equals the CPU oracle's
on the same seeded bytes (bit-exact: the path is integer and byte work only).  All calls go
through the C ABI via the ctypes binding."""
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


def _root_bytes(t: torch.Tensor) -> bytes:
    return _host(t).tobytes()


# ------------------------------------------------------------------------------------------ a2

@pytest.mark.parametrize("nbytes,chunk", [
    (64 << 20, 64 << 10),            # the small configuration: 1024 leaves
    (1 << 20, 4096), (1 << 20, 64), (1 << 20, 1 << 20), (1 << 20, 2 << 20),
    ((1 << 20) + 77, 4096),          # ragged last chunk
    (100_003, 1000), (100_003, 1001), (100_003, 7), (65, 64), (64, 64), (63, 64), (1, 1), (1, 4096),
    (5 * 4096 + 56, 4096), (5 * 4096 + 55, 4096), (5 * 4096 + 119, 4096), (5 * 4096 + 120, 4096),
    (37 * 48 + 16, 48),              # chunk size multiple of 16 but not 64
    (50 * (4096 + 16) + 8, 4096 + 16),   # bulk-copy path with a 16-byte remainder in every chunk
    (33 * 8192 + 4100, 8192), (3 * 65536 + 300, 65536 + 48),
    (20_000 * 4096 + 100, 4096),     # more than 592 warps: the many-chain launch shape, ragged last chunk
    (19_000 * 4096, 4096),    (60_000 * 4096 + 100, 4096), (57_000 * 16384, 16384),   # 12 or more groups per SM: the twelve-worker instance
    # between 2 and 2.85 groups per SM: the two-warp pairs as workers on the slice FIFO
    (9_600 * 4096 + 100, 4096), (9_473 * 65536 + 63, 65536), (12_000 * (4096 + 16), 4096 + 16), (13_450 * 8192, 8192),
    (9_473 * 32768 - 32700, 32768), (10_000 * 262144 + 64, 262144),
])
def test_hash_chunks_equals_oracle(ctx, nbytes, chunk):
    data = inputs.uniform_bytes(nbytes, seed=1, device="cuda")
    got = ctx.hash_chunks(data, chunk)
    groups = -(-binding.n_chunks(nbytes, chunk) // 32)
    if chunk >= 4096 and chunk % 16 == 0 and 296 < groups < 422:
        assert ctx.last_leaf_kernel == "hash_chunks_pairs_kernel"
    want = oracle.hash_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    assert got.shape == want.shape
    assert np.array_equal(_host(got), want)


@pytest.mark.parametrize("shift", [1, 2, 3, 4, 5, 8, 13, 15])
@pytest.mark.parametrize("chunk", [256, 1000, 4096 + 3])
def test_hash_chunks_any_base_alignment(ctx, shift, chunk):
    buf = inputs.uniform_bytes(300_000 + 16, seed=11, device="cuda")
    data = buf[shift:shift + 300_000]
    got = ctx.hash_chunks(data, chunk)
    assert np.array_equal(_host(got), oracle.hash_chunks(_host(data), chunk))


@pytest.mark.parametrize("n_chunks,chunk,last", [
    (19_000, 32768, 777),            # more than 592 warps of sliceable chunks: chains migrate between schedulers
    (19_000, 49152 + 16, 49152),     # chunk size a multiple of 16 but not of 64, several slices per chunk
    (18_945, 65536, 65536),          # exact multiple, last group holds a single chunk
    (20_001, 32768, 63),             # the last group's only chunk is shorter than one block
])
def test_hash_chunks_sliced_launch_shape(ctx, n_chunks, chunk, last):
    nbytes = (n_chunks - 1) * chunk + last
    data = inputs.uniform_bytes(nbytes, seed=77, device="cuda")
    got = ctx.hash_chunks(data, chunk)
    want = oracle.hash_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    assert np.array_equal(_host(got), want)
    assert ctx.device_status() == 0
    # a second call reuses the FIFO scratch
    got2 = ctx.hash_chunks(data, chunk)
    assert torch.equal(got, got2)


def test_hash_chunks_empty_and_argument_errors(ctx):
    data = inputs.uniform_bytes(4096, seed=2, device="cuda")
    assert ctx.hash_chunks(data[:0], 64).shape == (0, 32)
    with pytest.raises(binding.IvError) as e:
        ctx.hash_chunks(data, 0)
    assert e.value.code == binding.IV_ERR_INVALID_ARG
    small = torch.empty((3, 32), dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.IvError):
        ctx.hash_chunks(data, 1024, out=small)      # needs 4 records


def test_hash_chunks_window_split_invariance(ctx):
    """Algorithm 1's loop: hashing window by window into one digest array equals one call."""
    c, n = 4096, 37
    data = inputs.uniform_bytes(n * c - 100, seed=3, device="cuda")
    whole = ctx.hash_chunks(data, c)
    out = torch.zeros((n, 32), dtype=torch.uint8, device="cuda")
    win = 8 * c
    for w, off in enumerate(range(0, data.numel(), win)):
        ctx.hash_chunks(data[off:off + win], c, out=out[8 * w:])
    assert torch.equal(out, whole)


# ------------------------------------------------------------------------------------------ a3

@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 31, 32, 33, 255, 256, 257, 511, 512, 513, 1023, 1024, 1025,
                               2510, 3830, 10_000, 28_672, 512 * 512, 512 * 512 + 5, 300_001])
def test_merkle_root_equals_oracle(ctx, n):
    leaves = inputs.uniform_bytes(32 * n, seed=100 + n, device="cuda").view(n, 32)
    got = _root_bytes(ctx.merkle_root(leaves))
    assert got == oracle.merkle_root(_host(leaves))


def test_merkle_root_unaligned_leaf_pointer(ctx):
    buf = inputs.uniform_bytes(32 * 700 + 8, seed=5, device="cuda")
    leaves = buf[3:3 + 32 * 700]
    assert _root_bytes(ctx.merkle_root(leaves)) == oracle.merkle_root(_host(leaves))


def test_merkle_root_repeated_calls_reuse_scratch(ctx):
    for n in (70_000, 5, 70_000, 1300):
        leaves = inputs.uniform_bytes(32 * n, seed=n, device="cuda")
        assert _root_bytes(ctx.merkle_root(leaves)) == oracle.merkle_root(_host(leaves))


@pytest.mark.parametrize("n,levels", [(1, 3), (2, 1), (5, 1), (5, 2), (5, 3), (5, 9), (511, 4), (512, 9), (513, 9),
                                      (1000, 0), (1000, 1), (1000, 5), (1000, 10), (28_672, 6), (28_672, 12),
                                      (300_001, 9), (300_001, 11), (300_001, 19), (300_001, 30)])
def test_merkle_levels_equals_oracle_roots_of_aligned_runs(ctx, n, levels):
    """Node j, `levels` levels up, is the root of the aligned run of 2^levels leaves (oracle per run)."""
    leaves = inputs.uniform_bytes(32 * n, seed=500 + n + levels, device="cuda").view(n, 32)
    got = _host(ctx.merkle_levels(leaves, levels))
    host = _host(leaves)
    run = 1 << min(levels, 40)
    want = np.stack([np.frombuffer(oracle.merkle_root(host[s:s + run]), dtype=np.uint8) for s in range(0, n, run)])
    assert np.array_equal(got, want)


def test_sharded_root_emulated_ranks_on_one_gpu(ctx):
    """The multi-GPU plan with every rank's share computed in turn on this GPU: chunk digests of the rank's
    chunk range, iv_merkle_levels, nodes concatenated in rank order, iv_merkle_root == oracle root."""
    from paper_2510_23938_b200 import sharded
    chunk = 4096
    data = inputs.uniform_bytes(chunk * 2510 - 99, seed=61, device="cuda")
    n = binding.n_chunks(data.numel(), chunk)
    want = oracle.merkle_root(oracle.hash_chunks(_host(data), chunk, nthreads=oracle.host_threads()))
    for world in (1, 2, 3, 8):
        plan = sharded.plan_shards(n, world)
        parts = []
        for rank in range(world):
            lo, hi = plan.leaf_ranges[rank]
            shard = data[lo * chunk:min(hi * chunk, data.numel())]
            digests = ctx.hash_chunks(shard, chunk)
            assert digests.shape[0] == hi - lo
            if hi > lo:
                parts.append(ctx.merkle_levels(digests, plan.level))
        assert _root_bytes(ctx.merkle_root(torch.cat(parts))) == want
    # and the collective entry point with a world of one
    plan = sharded.plan_shards(n, 1)
    root = sharded.sharded_root(ctx, ctx.hash_chunks(data, chunk), plan, 0)
    assert _root_bytes(root) == want


def _oracle_tree(leaves: np.ndarray) -> np.ndarray:
    """Every level of the tree, leaves first: level l, node j = oracle root of the aligned run of 2^l leaves."""
    n = len(leaves)
    if n == 0:
        return np.frombuffer(oracle.merkle_root(b""), dtype=np.uint8).reshape(1, 32)
    levels, count, run = [leaves], n, 1
    while count > 1:
        run *= 2
        count = (count + 1) // 2
        levels.append(np.stack([np.frombuffer(oracle.merkle_root(leaves[s:s + run]), dtype=np.uint8)
                                for s in range(0, n, run)]))
    return np.concatenate(levels)


@pytest.mark.parametrize("n_chunks,chunk,last,n_dirty", [
    (1, 4096, 4096, 1), (2, 4096, 100, 2), (5, 1024, 1024, 2), (77, 512, 33, 9), (1000, 4096, 4096, 1),
    (1000, 4096, 17, 40), (2510, 4096, 4096, 300), (3000, 1024, 1024, 2000), (513, 2048, 2048, 513),
])
def test_tree_build_and_incremental_update_equal_a_full_oracle_rebuild(ctx, n_chunks, chunk, last, n_dirty):
    nbytes = (n_chunks - 1) * chunk + last
    data = inputs.uniform_bytes(nbytes, seed=n_chunks + n_dirty, device="cuda")
    leaves = ctx.hash_chunks(data, chunk)
    tree = ctx.tree_build(leaves)
    host_leaves = oracle.hash_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    assert np.array_equal(_host(tree), _oracle_tree(host_leaves))
    assert _host(tree[-1]).tobytes() == oracle.merkle_root(host_leaves)
    # change some chunks (always including the last, possibly short, one), update, compare with a rebuild
    rng = np.random.default_rng(n_chunks * 7 + n_dirty)
    dirty = rng.choice(n_chunks, size=min(n_dirty, n_chunks), replace=False)
    dirty[0] = n_chunks - 1
    dirty = np.concatenate([dirty, dirty[:3]])                      # repeats are allowed
    pos = torch.from_numpy(np.minimum(dirty * chunk + 3, nbytes - 1)).cuda()
    data[pos] ^= 0x5A
    ctx.tree_update(data, chunk, torch.from_numpy(dirty.astype(np.int64)).cuda(), tree)
    new_leaves = oracle.hash_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    assert not np.array_equal(new_leaves, host_leaves)
    assert np.array_equal(_host(tree), _oracle_tree(new_leaves))
    assert ctx.device_status() == 0


def test_tree_update_rejects_an_index_outside_the_tree_without_touching_it(ctx):
    chunk, n = 1024, 50
    data = inputs.uniform_bytes(chunk * n, seed=5, device="cuda")
    tree = ctx.tree_build(ctx.hash_chunks(data, chunk))
    before = tree.clone()
    ctx.tree_update(data, chunk, torch.tensor([n + 5], dtype=torch.int64, device="cuda"), tree)
    assert ctx.device_status() == 2
    assert torch.equal(tree, before)
    assert ctx.device_status() == 0          # reading the status clears it


# ------------------------------------------------------------------------------------------ a4

def _manifest_from_oracle(ctx, host_blob: np.ndarray, chunk: int):
    digests = oracle.hash_chunks(host_blob, chunk, nthreads=oracle.host_threads())
    root = oracle.merkle_root(digests)
    d_dig = torch.from_numpy(digests).cuda()
    return ctx.make_manifest(host_blob.size, chunk, d_dig, root), digests, root


def _verify(ctx, data, manifest, cap):
    res = binding.new_result("cuda")
    idx = torch.full((max(cap, 1),), -1, dtype=torch.int64, device="cuda")
    ctx.verify_manifest(data, manifest, res, idx if cap else None)
    torch.cuda.synchronize()
    r = binding.read_result(res)
    return r, [int(v) for v in idx[:min(cap, r["n_mismatch"])].cpu()]


def test_verify_small_configuration_with_three_tampered_copies(ctx):
    """64 MiB, 64 KiB chunks, manifest from the oracle; three copies with one flipped bit each."""
    nbytes, chunk = 64 << 20, 64 << 10
    data = inputs.uniform_bytes(nbytes, seed=1, device="cuda")
    manifest, digests, root = _manifest_from_oracle(ctx, _host(data), chunk)
    r, idx = _verify(ctx, data, manifest, 16)
    assert r == {"status": 0, "root_ok": True, "n_mismatch": 0, "root": root} and idx == []
    assert np.array_equal(_host(ctx.last_digests(1024)), digests)
    for seed in (2, 3, 4):
        off, bit = inputs.flip_position(seed, nbytes)
        bad = data.clone()
        bad[off] ^= (1 << bit)
        r, idx = _verify(ctx, bad, manifest, 16)
        o_ok, o_bad, o_idx, o_root = oracle.verify(_host(bad), chunk, digests, root, nthreads=oracle.host_threads())
        assert (r["root_ok"], r["n_mismatch"], idx, r["root"]) == (o_ok, o_bad, o_idx, o_root)
        assert idx == [off // chunk] and not r["root_ok"]


def test_batch_verification_of_the_small_configuration_and_its_three_tampered_copies(ctx):
    """The four verifications of the small configuration as ONE pass (4096 chains in one hashing launch)."""
    nbytes, chunk = 64 << 20, 64 << 10
    data = inputs.uniform_bytes(nbytes, seed=1, device="cuda")
    manifest, digests, root = _manifest_from_oracle(ctx, _host(data), chunk)
    blobs, want = [data], [(True, 0, [], root)]
    for seed in (2, 3, 4):
        off, bit = inputs.flip_position(seed, nbytes)
        bad = data.clone()
        bad[off] ^= (1 << bit)
        blobs.append(bad)
        want.append(oracle.verify(_host(bad), chunk, digests, root, nthreads=oracle.host_threads()))
        assert want[-1][2] == [off // chunk]
    results = torch.zeros((4, 48), dtype=torch.uint8, device="cuda")
    idx = torch.full((4, 8), -1, dtype=torch.int64, device="cuda")
    ctx.verify_manifest_batch(blobs, manifest, results, idx)
    torch.cuda.synchronize()
    for b, r in enumerate(binding.read_results(results)):
        got = (r["root_ok"], r["n_mismatch"], [int(v) for v in idx[b, :r["n_mismatch"]].cpu()], r["root"])
        assert got == want[b], b
    assert ctx.device_status() == 0
    # ragged size, unaligned blobs, capacity 0
    content = inputs.uniform_bytes(100_003, seed=9, device="cuda")
    small = []
    for k in (0, 1, 5):                                   # three copies at different byte alignments
        buf = torch.empty(100_003 + 16, dtype=torch.uint8, device="cuda")
        buf[k:k + 100_003] = content
        small.append(buf[k:k + 100_003])
    small[1][77_777] ^= 4
    m2, d2, r2 = _manifest_from_oracle(ctx, _host(small[0]), 1000)
    res2 = torch.zeros((3, 48), dtype=torch.uint8, device="cuda")
    ctx.verify_manifest_batch(small, m2, res2, None)
    out = binding.read_results(res2)
    assert [o["root_ok"] for o in out] == [True, False, True] and [o["n_mismatch"] for o in out] == [0, 1, 0]


def test_verify_many_mismatches_ascending_exact_count_and_truncation(ctx):
    chunk, n = 512, 5000
    data = inputs.uniform_bytes(chunk * n - 17, seed=8, device="cuda")
    manifest, digests, root = _manifest_from_oracle(ctx, _host(data), chunk)
    rng = np.random.default_rng(9)
    hit = np.sort(rng.choice(n, size=777, replace=False))
    bad = data.clone()
    bad[torch.from_numpy(hit * chunk + 5).cuda()] ^= 0x40
    want = oracle.verify(_host(bad), chunk, digests, root, nthreads=oracle.host_threads())
    r, idx = _verify(ctx, bad, manifest, n)
    assert (r["root_ok"], r["n_mismatch"], idx, r["root"]) == want
    assert idx == [int(v) for v in hit]
    r, idx = _verify(ctx, bad, manifest, 100)
    assert r["n_mismatch"] == 777 and idx == [int(v) for v in hit[:100]]
    r, idx = _verify(ctx, bad, manifest, 0)
    assert r["n_mismatch"] == 777 and idx == []
    # every chunk wrong
    allbad = data ^ 0xFF
    r, idx = _verify(ctx, allbad, manifest, n)
    assert r["n_mismatch"] == n and idx == list(range(n))


def test_verify_manifest_side_tampering_and_argument_checks(ctx):
    chunk = 1024
    data = inputs.uniform_bytes(chunk * 70 + 1, seed=12, device="cuda")
    manifest, digests, root = _manifest_from_oracle(ctx, _host(data), chunk)
    man2 = digests.copy()
    man2[33, 0] ^= 1
    m2 = ctx.make_manifest(data.numel(), chunk, torch.from_numpy(man2).cuda(), root)
    r, idx = _verify(ctx, data, m2, 8)
    assert r["root_ok"] and r["n_mismatch"] == 1 and idx == [33]
    wrong_root = bytes([root[0] ^ 0x80]) + root[1:]
    m3 = ctx.make_manifest(data.numel(), chunk, torch.from_numpy(digests).cuda(), wrong_root)
    r, idx = _verify(ctx, data, m3, 8)
    assert (not r["root_ok"]) and r["n_mismatch"] == 0 and r["root"] == root
    res = binding.new_result("cuda")
    with pytest.raises(binding.IvError):                 # manifest for a different size
        ctx.verify_manifest(data[:-1], manifest, res, None)
    bad = ctx.make_manifest(data.numel(), chunk, torch.from_numpy(digests[:-1]).cuda(), root)
    with pytest.raises(binding.IvError):                 # wrong chunk count
        ctx.verify_manifest(data, bad, res, None)


def test_verify_empty_blob(ctx):
    empty = torch.empty(0, dtype=torch.uint8, device="cuda")
    root = oracle.merkle_root(b"")
    m = ctx.make_manifest(0, 4096, empty, root)
    r, idx = _verify(ctx, empty, m, 4)
    assert r["root_ok"] and r["n_mismatch"] == 0 and r["root"] == root


# ------------------------------------------------------------------------------------------ two-level leaves

def _oracle_two_level(host: np.ndarray, chunk: int, sub: int) -> np.ndarray:
    """D_i = oracle root over the oracle digests of chunk i's pieces (the mode's definition, composed on the CPU)."""
    out = []
    for o in range(0, host.size, chunk):
        pieces = oracle.hash_chunks(host[o:o + chunk], sub)
        out.append(np.frombuffer(oracle.merkle_root(pieces), dtype=np.uint8))
    return np.stack(out) if out else np.zeros((0, 32), dtype=np.uint8)


@pytest.mark.parametrize("nbytes,chunk,sub", [
    (64 << 20, 4 << 20, 64 << 10),            # 16 chunks of 64 pieces: 1024 independent chains instead of 16
    ((8 << 20) + 12345, 1 << 20, 1 << 16),    # short last chunk whose last piece is short too
    (300_000, 4096, 1024), (300_000, 4096, 4096), (100, 4096, 512), (5 * 8192 + 1, 8192, 8192 // 4),
])
def test_two_level_leaves_equal_their_definition_and_share_the_root_with_piece_granularity(ctx, nbytes, chunk, sub):
    data = inputs.uniform_bytes(nbytes, seed=71, device="cuda")
    host = _host(data)
    got = ctx.hash_chunks_two_level(data, chunk, sub)
    want = _oracle_two_level(host, chunk, sub)
    assert np.array_equal(_host(got), want)
    # one root for both granularities
    root = _root_bytes(ctx.merkle_root(got))
    assert root == oracle.merkle_root(oracle.hash_chunks(host, sub, nthreads=oracle.host_threads()))
    # verification in this mode finds a flipped bit at its chunk
    manifest = ctx.make_manifest(nbytes, chunk, torch.from_numpy(want).cuda(), oracle.merkle_root(want))
    res = binding.new_result("cuda")
    idx = torch.zeros(4, dtype=torch.int64, device="cuda")
    ctx.verify_manifest_two_level(data, manifest, sub, res, idx)
    r = binding.read_result(res)
    assert r["root_ok"] and r["n_mismatch"] == 0 and r["root"] == root
    bad = data.clone()
    bad[nbytes - 1] ^= 1
    ctx.verify_manifest_two_level(bad, manifest, sub, res, idx)
    r = binding.read_result(res)
    assert (not r["root_ok"]) and r["n_mismatch"] == 1 and int(idx[0]) == (nbytes - 1) // chunk


def test_two_level_requires_a_power_of_two_ratio(ctx):
    data = inputs.uniform_bytes(1 << 16, seed=1, device="cuda")
    for chunk, sub in ((4096, 3000), (4096, 0), (4096, 8192), (12288, 4096)):
        with pytest.raises(binding.IvError) as e:
            ctx.hash_chunks_two_level(data, chunk, sub)
        assert e.value.code == binding.IV_ERR_INVALID_ARG


# ------------------------------------------------------------------------------------------ a5

@pytest.mark.parametrize("pinned", [True, False])
def test_streamed_verification_equals_resident(ctx, pinned):
    chunk, n = 4096, 301
    host = inputs.uniform_bytes(chunk * n - 1000, seed=21)
    if pinned:
        host = host.pin_memory()
    manifest, digests, root = _manifest_from_oracle(ctx, host.numpy(), chunk)
    for window_chunks in (1, 7, 64, 1000):
        res = binding.new_result("cuda")
        idx = torch.zeros(8, dtype=torch.int64, device="cuda")
        ctx.verify_streamed(host, window_chunks * chunk, host.numel(), manifest, res, idx)
        torch.cuda.synchronize()
        r = binding.read_result(res)
        assert r["root_ok"] and r["n_mismatch"] == 0 and r["root"] == root
        assert np.array_equal(_host(ctx.last_digests(n)), digests)
    bad = host.clone()
    bad[chunk * 200 + 9] ^= 2
    res = binding.new_result("cuda")
    idx = torch.zeros(8, dtype=torch.int64, device="cuda")
    ctx.verify_streamed(bad.pin_memory() if pinned else bad, 16 * chunk, bad.numel(), manifest, res, idx)
    torch.cuda.synchronize()
    r = binding.read_result(res)
    assert (not r["root_ok"]) and r["n_mismatch"] == 1 and int(idx[0]) == 200
    with pytest.raises(binding.IvError):                 # window not a multiple of the chunk size
        ctx.verify_streamed(host, chunk + 1, host.numel(), manifest, res, idx)


@pytest.mark.parametrize("chunk,n_chunks,short_by,window_chunks,pinned", [
    (32768, 40, 100, 16, True),             # two column parts of 16 KiB per chunk
    (65536, 64, 0, 64, True), (3 * 16384 + 4096 + 48, 21, 5, 5, False),   # four parts; three parts, odd chunk size
    (131072, 37, 1000, 8, True),            # eight column parts per chunk, five windows, short last chunk
    (1 << 20, 19, 77, 4, True),             # sixteen parts, a last chunk that ends inside a block
    (1 << 20, 19, 77, 19, False),           # one window, pageable host memory
    (5 * 65536 + 64, 11, 0, 3, True),       # a chunk size that is no multiple of 4 KiB: the last part is longer
    (200_008, 9, 199_990, 4, True),         # no multiple of 16; the short last chunk has 18 bytes
    (1 << 20, 1, 0, 1, True), (1 << 20, 1, (1 << 20) - 64, 1, True), (1 << 20, 2, (1 << 20) - 1, 2, True),
])
def test_streamed_windows_hashed_in_column_parts(ctx, chunk, n_chunks, short_by, window_chunks, pinned):
    """Chunks of 32 KiB and more with few chains per window take the column-part path of the streamed
    verification (strided copies, resumed chaining values): digests, root and the located damage equal the oracle's."""
    nbytes = chunk * n_chunks - short_by
    host = inputs.uniform_bytes(nbytes, seed=33 + n_chunks)
    manifest, digests, root = _manifest_from_oracle(ctx, host.numpy(), chunk)
    src = host.pin_memory() if pinned else host
    res = binding.new_result("cuda")
    idx = torch.zeros(8, dtype=torch.int64, device="cuda")
    for _ in range(2):                                       # twice: the window buffers and states are reused
        ctx.verify_streamed(src, window_chunks * chunk, nbytes, manifest, res, idx)
        torch.cuda.synchronize()
        r = binding.read_result(res)
        assert r == {"status": 0, "root_ok": True, "n_mismatch": 0, "root": root}
        assert np.array_equal(_host(ctx.last_digests(n_chunks)), digests)
    # one flipped bit in a middle part of a chunk and one in the very last byte
    bad = host.clone()
    hits = sorted({min(nbytes - 1, (n_chunks // 2) * chunk + chunk // 2 + 5), nbytes - 1})
    for off in hits:
        bad[off] ^= 0x40
    ctx.verify_streamed(bad.pin_memory() if pinned else bad, window_chunks * chunk, nbytes, manifest, res, idx)
    torch.cuda.synchronize()
    r = binding.read_result(res)
    want_idx = sorted({off // chunk for off in hits})
    assert (not r["root_ok"]) and r["n_mismatch"] == len(want_idx)
    assert [int(v) for v in idx[:len(want_idx)].cpu()] == want_idx
    want = oracle.hash_chunks(bad.numpy(), chunk, nthreads=oracle.host_threads())
    assert np.array_equal(_host(ctx.last_digests(n_chunks)), want) and r["root"] == oracle.merkle_root(want)
    assert ctx.device_status() == 0


# ------------------------------------------------------------------------------------------ a6

def test_hash_ragged_edge_lengths_and_alignments(ctx):
    base = inputs.uniform_bytes(200_000, seed=31, device="cuda")
    lengths, offsets = [], []
    for ln in (0, 1, 2, 3, 4, 55, 56, 57, 63, 64, 65, 119, 120, 121, 127, 128, 129, 1000, 4096, 4097):
        for o in (0, 1, 2, 3, 5, 6, 7, 9, 13, 15, 16, 17):
            lengths.append(ln)
            offsets.append(o + 37 * len(lengths))
    got = ctx.hash_ragged(base, torch.tensor(offsets, device="cuda"), torch.tensor(lengths, device="cuda"))
    want = oracle.hash_ragged(_host(base), offsets, lengths, nthreads=oracle.host_threads())
    assert np.array_equal(_host(got), want)


def test_hash_ragged_log_uniform_set_and_root(ctx):
    """The ragged configuration scaled down: 3000 tensors, log-uniform 64 B .. 256 KiB, packed at 2-byte alignment."""
    sizes = inputs.ragged_sizes(3000, 64, 256 << 10, seed=5)
    offs = inputs.packed_offsets(sizes, first=6)
    total = int(offs[-1] + sizes[-1])
    base = inputs.uniform_bytes(total + 10, seed=32, device="cuda")
    got = ctx.hash_ragged(base, torch.from_numpy(offs).cuda(), torch.from_numpy(sizes).cuda())
    want = oracle.hash_ragged(_host(base), offs, sizes, nthreads=oracle.host_threads())
    assert np.array_equal(_host(got), want)
    assert _root_bytes(ctx.merkle_root(got)) == oracle.merkle_root(want)


def test_hash_ragged_per_tensor_digests_of_a_weight_file(ctx):
    blob, table = inputs.weight_file(inputs.tiny_tensors(), seed=7, device="cuda")
    offs = np.array([o for _, o, _ in table], dtype=np.int64)
    lens = np.array([n for _, _, n in table], dtype=np.int64)
    got = ctx.hash_ragged(blob, torch.from_numpy(offs).cuda(), torch.from_numpy(lens).cuda())
    assert np.array_equal(_host(got), oracle.hash_ragged(_host(blob), offs, lens))
    # chunk digests of the same file, header included, 4 KiB chunks
    chunks = ctx.hash_chunks(blob, 4096)
    assert np.array_equal(_host(chunks), oracle.hash_chunks(_host(blob), 4096))


def test_hash_ragged_large_set_takes_the_work_queue_path(ctx):
    """More tensors than the sorted two-warp path takes (32768): the per-lane work-queue kernel."""
    n = 40_000
    rng = np.random.default_rng(41)
    sizes = rng.integers(0, 700, size=n).astype(np.int64)
    sizes[::997] = rng.integers(10_000, 60_000, size=len(sizes[::997]))
    offs = inputs.packed_offsets(sizes, first=3)
    base = inputs.uniform_bytes(int(offs[-1] + sizes[-1]) + 8, seed=33, device="cuda")
    got = ctx.hash_ragged(base, torch.from_numpy(offs).cuda(), torch.from_numpy(sizes).cuda())
    want = oracle.hash_ragged(_host(base), offs, sizes, nthreads=oracle.host_threads())
    assert np.array_equal(_host(got), want)


def test_hash_ragged_every_16_byte_misalignment_with_long_messages(ctx):
    """Messages of many blocks at each start offset 0..31: every stage hand-over of the bulk-copy ring."""
    base = inputs.uniform_bytes(64 * 70_000, seed=34, device="cuda")
    lengths, offsets = [], []
    for a in range(32):
        for ln in (64 * 8, 64 * 8 + 1, 64 * 9 - 1, 64 * 17 + 5, 64 * 24, 64 * 25 + 63, 40_000 + a):
            offsets.append(a + 100_000 * (len(offsets) % 40))
            lengths.append(ln)
    got = ctx.hash_ragged(base, torch.tensor(offsets, device="cuda"), torch.tensor(lengths, device="cuda"))
    want = oracle.hash_ragged(_host(base), offsets, lengths, nthreads=oracle.host_threads())
    assert np.array_equal(_host(got), want)
    assert ctx.device_status() == 0


def test_hash_ragged_update_in_parts_equals_one_shot_digests(ctx):
    """Multi-pass hashing: every tensor is fed in three parts (whole blocks, whole blocks, the rest) from
    different places of the buffer; the chaining values travel in the state records."""
    rng = np.random.default_rng(51)
    n = 300
    sizes = np.concatenate([rng.integers(0, 5000, size=n - 6), [0, 63, 64, 65, 200_000, 1_000_003]]).astype(np.int64)
    offs = inputs.packed_offsets(sizes, first=5)
    base = inputs.uniform_bytes(int(offs[-1] + sizes[-1]) + 16, seed=52, device="cuda")
    host = _host(base)
    want = oracle.hash_ragged(host, offs, sizes, nthreads=oracle.host_threads())
    # cut points: multiples of 64 inside each tensor
    blocks = sizes // 64
    cut1 = (blocks * rng.uniform(0, 1, size=n)).astype(np.int64) * 64
    cut2 = cut1 + ((blocks - cut1 // 64) * rng.uniform(0, 1, size=n)).astype(np.int64) * 64
    states = ctx.new_sha_states(n)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int64)).cuda()
    assert ctx.hash_ragged_update(base, dev(offs), dev(cut1), states, finish=False) is None
    ctx.hash_ragged_update(base, dev(offs + cut1), dev(cut2 - cut1), states, finish=False)
    got = ctx.hash_ragged_update(base, dev(offs + cut2), dev(sizes - cut2), states, finish=True)
    assert np.array_equal(_host(got), want)
    assert ctx.device_status() == 0
    # one-shot through the same entry point
    fresh = ctx.new_sha_states(n)
    got1 = ctx.hash_ragged_update(base, dev(offs), dev(sizes), fresh, finish=True)
    assert np.array_equal(_host(got1), want)
    # a non-final part that is not a whole number of blocks is refused (status 2)
    bad = ctx.new_sha_states(2)
    ctx.hash_ragged_update(base, dev([0, 100]), dev([64, 65]), bad, finish=False)
    assert ctx.device_status() == 2


def test_hash_ragged_empty_set(ctx):
    base = inputs.uniform_bytes(64, seed=1, device="cuda")
    e = torch.empty(0, dtype=torch.int64, device="cuda")
    assert ctx.hash_ragged(base, e, e).shape == (0, 32)


def test_streamed_windows_may_repeat_and_phase_times_are_reported(ctx):
    """A ring of two host windows read three times each: the blob is periodic; timing brackets the phases."""
    chunk, per_win = 4096, 16
    ring = [inputs.uniform_bytes(chunk * per_win, seed=40 + k).pin_memory() for k in range(2)]
    windows = [ring[w % 2] for w in range(6)]
    whole = torch.cat(windows).numpy()
    manifest, digests, root = _manifest_from_oracle(ctx, whole, chunk)
    res = binding.new_result("cuda")
    ctx.set_timing(True)
    ctx.verify_streamed(windows, chunk * per_win, whole.size, manifest, res, None)
    torch.cuda.synchronize()
    ms = ctx.phase_times(0)
    ctx.set_timing(False)
    r = binding.read_result(res)
    assert r["root_ok"] and r["n_mismatch"] == 0 and r["root"] == root
    assert all(t >= 0.0 for t in ms) and ms[0] > 0.0
    ctx.verify_manifest(torch.from_numpy(whole).cuda(), manifest, res, None)
    with pytest.raises(binding.IvError):
        ctx.phase_times(0)                       # timing was off for that call


def test_device_status_is_clean_after_all_of_the_above(ctx):
    assert ctx.device_status() == 0


def test_launch_counter_counts_kernels(ctx):
    before = ctx.kernel_launches
    data = inputs.uniform_bytes(1 << 16, seed=1, device="cuda")
    d = ctx.hash_chunks(data, 1024)
    ctx.merkle_root(d)
    assert ctx.kernel_launches == before + 2


def test_two_contexts_on_two_streams_at_once():
    """One context per stream (the header's rule): two verifications enqueued back to back on two streams
    overlap on the GPU and both come out right; a third call on the default stream runs beside them."""
    a, b = binding.Context(0), binding.Context(0)
    try:
        sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
        da = inputs.uniform_bytes((96 << 20) + 5, seed=71, device="cuda")
        db = inputs.uniform_bytes(80 << 20, seed=72, device="cuda")
        torch.cuda.synchronize()
        man_a, _, root_a = _manifest_from_oracle(a, _host(da), 1 << 20)
        man_b, _, root_b = _manifest_from_oracle(b, _host(db), 64 << 10)
        ra, rb = binding.new_result("cuda"), binding.new_result("cuda")
        ia = torch.zeros(4, dtype=torch.int64, device="cuda")
        ib = torch.zeros(4, dtype=torch.int64, device="cuda")
        db[12345] ^= 1
        torch.cuda.synchronize()
        for _ in range(3):
            a.verify_manifest(da, man_a, ra, ia, stream=sa)
            b.verify_manifest(db, man_b, rb, ib, stream=sb)
        torch.cuda.synchronize()
        r = binding.read_result(ra)
        assert r["root_ok"] and r["n_mismatch"] == 0 and r["root"] == root_a
        r = binding.read_result(rb)
        assert (not r["root_ok"]) and r["n_mismatch"] == 1 and int(ib[0]) == 12345 // (64 << 10)
        assert a.device_status() == 0 and b.device_status() == 0
    finally:
        a.close()
        b.close()
