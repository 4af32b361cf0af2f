"""Seeded random cases through the calls that sit on top of leaf hashing -- verification with tampering,
streamed verification, the retained tree and its updates, batch verification, resumable tensor digests,
Merkle roots and levels -- each result compared with the CPU oracle bit for bit.  The hand-written cases
elsewhere fix their shapes; here blob size, chunk size, tail, window size, number and place of the flipped
bits, dirty sets and the way a tensor is cut into parts come from a seeded generator.  All through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_23938_b200 import binding, inputs

pytestmark = pytest.mark.gpu

T = oracle.host_threads()


@pytest.fixture(scope="module")
def ctx():
    if not torch.cuda.is_available():
        pytest.fail("the gpu-marked tests need a CUDA device")
    c = binding.Context(0)
    yield c
    c.close()


def _host(t):
    return t.cpu().numpy()


def _shape(rng, max_bytes):
    """A chunk size, a chunk count and a blob length whose last chunk may be short."""
    kind = int(rng.integers(0, 4))
    if kind == 0:      # many chains, small chunks (migrating or pairs kernel)
        chunk = 16 * int(rng.integers(256, 1024)); n = int(rng.integers(9_500, 20_000))
    elif kind == 1:    # medium
        chunk = 16 * int(rng.integers(1024, 8_000)); n = int(rng.integers(100, 3_000))
    elif kind == 2:    # few chains, large chunks (two-warp kernel)
        chunk = 16 * int(rng.integers(4096, 60_000)); n = int(rng.integers(1, 200))
    else:              # odd chunk sizes (direct kernel)
        chunk = int(rng.integers(1, 20_000)); n = int(rng.integers(1, 2_000))
    while chunk * n > max_bytes:
        n //= 2
    n = max(n, 1)
    tail = int(rng.integers(1, chunk + 1)) if rng.random() < 0.6 else chunk
    return chunk, n, (n - 1) * chunk + tail


def _oracle_manifest(ctx, host_blob, chunk):
    digests = oracle.hash_chunks(host_blob, chunk, nthreads=T)
    root = oracle.merkle_root(digests)
    return ctx.make_manifest(host_blob.size, chunk, torch.from_numpy(digests).cuda(), root), digests, root


def _oracle_tree(leaves):
    """All levels of the tree, leaves first: level k holds the roots of the aligned runs of 2^k leaves."""
    n = leaves.shape[0]
    levels, run, count = [leaves], 1, n
    while count > 1:
        run *= 2
        count = (count + 1) // 2
        levels.append(np.stack([np.frombuffer(oracle.merkle_root(leaves[s:s + run]), dtype=np.uint8)
                                for s in range(0, n, run)]))
    return np.concatenate(levels)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_verification_with_random_tampering(ctx, seed):
    rng = np.random.default_rng(seed)
    kernels = set()
    for _ in range(12):
        chunk, n, nbytes = _shape(rng, 160 << 20)
        data = inputs.uniform_bytes(nbytes, seed=int(rng.integers(1, 1 << 30)), device="cuda")
        manifest, digests, root = _oracle_manifest(ctx, _host(data), chunk)
        k = int(rng.choice([0, 1, 3, 50]))
        pos = np.unique(rng.integers(0, nbytes, size=k)) if k else np.zeros(0, dtype=np.int64)
        if k:
            data[torch.from_numpy(pos).cuda()] ^= 0x10
        want_idx = sorted({int(p) // chunk for p in pos})
        cap = int(rng.choice([0, 2, 64]))
        res = binding.new_result("cuda")
        idx = torch.full((max(cap, 1),), -1, dtype=torch.int64, device="cuda")
        ctx.verify_manifest(data, manifest, res, idx if cap else None)
        torch.cuda.synchronize()
        r = binding.read_result(res)
        kernels.add(ctx.last_leaf_kernel)
        o_ok, o_bad, o_idx, o_root = oracle.verify(_host(data), chunk, digests, root, nthreads=T)
        assert o_idx == want_idx and o_bad == len(want_idx)         # the flips are where they were put
        what = (seed, chunk, n, nbytes, k, cap, ctx.last_leaf_kernel)
        assert (r["status"], r["root_ok"], r["n_mismatch"], r["root"]) == (0, o_ok, o_bad, o_root), what
        assert [int(v) for v in idx[:min(cap, o_bad)].cpu()] == o_idx[:cap], what
        if cap > o_bad:
            assert int(idx[o_bad]) == -1, what                      # nothing written past the list
    assert len(kernels) >= 2


@pytest.mark.parametrize("seed", [21, 22])
def test_streamed_verification_with_random_windows(ctx, seed):
    rng = np.random.default_rng(seed)
    for _ in range(10):
        chunk, n, nbytes = _shape(rng, 96 << 20)
        blob = inputs.uniform_bytes(nbytes, seed=int(rng.integers(1, 1 << 30)))
        pinned = bool(rng.random() < 0.5)
        if pinned:
            blob = blob.pin_memory()
        manifest, digests, root = _oracle_manifest(ctx, blob.numpy(), chunk)
        window_chunks = int(rng.integers(1, max(2, n // 2 + 2)))
        res = binding.new_result("cuda")
        idx = torch.full((8,), -1, dtype=torch.int64, device="cuda")
        ctx.verify_streamed(blob, window_chunks * chunk, nbytes, manifest, res, idx)
        torch.cuda.synchronize()
        what = (seed, chunk, n, nbytes, window_chunks, pinned, ctx.last_leaf_kernel)
        assert binding.read_result(res) == {"status": 0, "root_ok": True, "n_mismatch": 0, "root": root}, what
        assert np.array_equal(_host(ctx.last_digests(n)), digests), what
        assert int(idx[0]) == -1, what


@pytest.mark.parametrize("seed", [31, 32])
def test_retained_tree_with_random_dirty_sets(ctx, seed):
    rng = np.random.default_rng(seed)
    for _ in range(8):
        chunk, n, nbytes = _shape(rng, 64 << 20)
        if n > 3000:
            n, nbytes = 3000, 3000 * chunk
        data = inputs.uniform_bytes(nbytes, seed=int(rng.integers(1, 1 << 30)), device="cuda")
        tree = ctx.tree_build(ctx.hash_chunks(data, chunk))
        before = oracle.hash_chunks(_host(data), chunk, nthreads=T)
        assert np.array_equal(_host(tree), _oracle_tree(before)), (seed, chunk, n)
        n_dirty = int(rng.integers(1, n + 1))
        dirty = rng.choice(n, size=n_dirty, replace=False)
        pos = np.minimum(dirty * chunk + int(rng.integers(0, chunk)), nbytes - 1)
        data[torch.from_numpy(pos).cuda()] ^= 0x21
        ctx.tree_update(data, chunk, torch.from_numpy(dirty.astype(np.int64)).cuda(), tree)
        after = oracle.hash_chunks(_host(data), chunk, nthreads=T)
        assert np.array_equal(_host(tree), _oracle_tree(after)), (seed, chunk, n, n_dirty)
        assert ctx.device_status() == 0


@pytest.mark.parametrize("seed", [41, 42])
def test_batch_verification_with_random_tampering(ctx, seed):
    rng = np.random.default_rng(seed)
    for _ in range(8):
        chunk = 16 * int(rng.integers(64, 8192))
        n = int(rng.integers(1, 400))
        n_blobs = int(rng.integers(1, 9))
        nbytes = (n - 1) * chunk + (int(rng.integers(1, chunk + 1)) if rng.random() < 0.5 else chunk)
        while nbytes * n_blobs > (256 << 20) and n_blobs > 1:
            n_blobs -= 1
        base = inputs.uniform_bytes(nbytes, seed=int(rng.integers(1, 1 << 30)), device="cuda")
        manifest, digests, root = _oracle_manifest(ctx, _host(base), chunk)
        blobs = []
        for _b in range(n_blobs):
            copy = base.clone()
            k = int(rng.choice([0, 1, 4]))
            if k:
                copy[torch.from_numpy(np.unique(rng.integers(0, nbytes, size=k))).cuda()] ^= 0x02
            blobs.append(copy)
        results = torch.zeros((n_blobs, 48), dtype=torch.uint8, device="cuda")
        idx = torch.full((n_blobs, 8), -1, dtype=torch.int64, device="cuda")
        ctx.verify_manifest_batch(blobs, manifest, results, idx)
        torch.cuda.synchronize()
        got = binding.read_results(results)
        for b in range(n_blobs):
            o_ok, o_bad, o_idx, o_root = oracle.verify(_host(blobs[b]), chunk, digests, root, nthreads=T)
            what = (seed, chunk, n, n_blobs, b)
            assert (got[b]["root_ok"], got[b]["n_mismatch"], got[b]["root"]) == (o_ok, o_bad, o_root), what
            assert [int(v) for v in idx[b, :min(8, o_bad)].cpu()] == o_idx[:8], what
        assert ctx.device_status() == 0


@pytest.mark.parametrize("seed", [51, 52])
def test_tensor_digests_one_shot_and_in_random_parts(ctx, seed):
    rng = np.random.default_rng(seed)
    for _ in range(8):
        n = int(rng.choice([1, 7, 33, 200, 1500]))
        total = int(rng.integers(1 << 16, 48 << 20))
        base = inputs.uniform_bytes(total, seed=int(rng.integers(1, 1 << 30)), device="cuda")
        mode = int(rng.integers(0, 3))
        if mode == 0:       # log-uniform lengths
            lens = np.exp(rng.uniform(0, np.log(max(total // 4, 2)), size=n)).astype(np.int64)
        elif mode == 1:     # empty tensors and lengths around the padding borders
            lens = rng.choice([0, 1, 55, 56, 63, 64, 65, 119, 120, 127, 128, 4095, 4096, 4097], size=n).astype(np.int64)
        else:               # equal, long
            lens = np.full(n, max(total // n - 16, 1), dtype=np.int64)
        lens = np.minimum(lens, total)
        offs = np.array([int(rng.integers(0, total - int(ln) + 1)) for ln in lens], dtype=np.int64)   # any alignment; may overlap
        want = oracle.hash_ragged(_host(base), offs, lens, nthreads=T)
        got = ctx.hash_ragged(base, torch.from_numpy(offs).cuda(), torch.from_numpy(lens).cuda())
        assert np.array_equal(_host(got), want), (seed, n, total, mode)
        # the same digests from two to four calls; every part but the last is a whole number of 64-byte blocks
        parts = int(rng.integers(2, 5))
        states = ctx.new_sha_states(n)
        done = np.zeros(n, dtype=np.int64)
        out = None
        for p in range(parts):
            last = p + 1 == parts
            part = lens - done if last else (rng.integers(0, 1 << 30, size=n) % ((lens - done) // 64 + 1)) * 64
            out = ctx.hash_ragged_update(base, torch.from_numpy(offs + done).cuda(),
                                         torch.from_numpy(part.astype(np.int64)).cuda(), states, last)
            done = done + part
        assert np.array_equal(_host(out), want), (seed, n, total, mode, parts)
        assert ctx.device_status() == 0


@pytest.mark.parametrize("seed", [61])
def test_roots_and_levels_of_random_leaf_counts(ctx, seed):
    rng = np.random.default_rng(seed)
    out = torch.zeros(32, dtype=torch.uint8, device="cuda")
    for _ in range(30):
        n = int(rng.choice([1, 2, 3, int(rng.integers(1, 2000)), int(rng.integers(2000, 600_000))]))
        leaves = inputs.uniform_bytes(32 * n, seed=int(rng.integers(1, 1 << 30)), device="cuda").view(n, 32)
        host_leaves = _host(leaves)
        want = oracle.merkle_root(host_leaves)
        assert _host(ctx.merkle_root(leaves)).tobytes() == want, n
        assert _host(ctx.merkle_root_rfc6962(leaves)).tobytes() == oracle.merkle_root_rfc6962(host_leaves), n
        k = int(rng.integers(0, 12))
        nodes = _host(ctx.merkle_levels(leaves, k))
        run = 1 << k
        assert nodes.shape[0] == -(-n // run)
        for j in rng.choice(nodes.shape[0], size=min(nodes.shape[0], 16), replace=False):
            assert nodes[j].tobytes() == oracle.merkle_root(host_leaves[j * run:(j + 1) * run]), (n, k, j)
        if n <= binding.NOALLOC_MAX_LEAVES:
            binding.merkle_root_noalloc(leaves, out)
            assert _host(out).tobytes() == want, n
