"""Stand-ins for a memory checker, which this pool does not offer: guard bytes around every output the
library writes, and the bounded-wait failure path run end to end.

Guard bytes.  Every output of a call (digests, roots, result records, index lists, tree arrays, hashing
states) lies inside a larger device buffer filled with a sentinel; after the call the margins on both sides
must be untouched and the output must equal the oracle's.  The shapes walk through every leaf-hashing
kernel and launch shape the dispatcher can pick.

Timeout.  A kernel whose wait runs out must return, set the device status to 1 and leave the context
usable: `iv_selftest_wait_timeout` waits, with the library's own wait routine and a short limit, on a
barrier nobody arrives at.  Nothing spins for ever and nothing traps."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2510_23938_b200 import binding, inputs

pytestmark = pytest.mark.gpu

SENTINEL = 0xA5
MARGIN = 512          # bytes on each side; keeps 16-byte alignment of the guarded view


class Guarded:
    """`nbytes` bytes of device memory between two sentinel-filled margins."""

    def __init__(self, nbytes: int, fill: int = 0):
        self.nbytes = nbytes
        self.raw = torch.full((2 * MARGIN + nbytes,), SENTINEL, dtype=torch.uint8, device="cuda")
        self.view = self.raw[MARGIN:MARGIN + nbytes]
        self.view.fill_(fill)

    def as_(self, dtype=torch.uint8, shape=None) -> torch.Tensor:
        t = self.view.view(dtype)
        return t if shape is None else t.view(shape)

    def check(self, what=""):
        torch.cuda.synchronize()
        lo, hi = self.raw[:MARGIN], self.raw[MARGIN + self.nbytes:]
        assert bool((lo == SENTINEL).all()), f"bytes BEFORE the output were written {what}"
        assert bool((hi == SENTINEL).all()), f"bytes AFTER the output were written {what}"


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available(), "the gpu-marked tests need a CUDA device"
    c = binding.Context(0)
    yield c
    c.close()


def _host(t):
    return t.cpu().numpy()


# kernel and (for the many-chain kernel) launch shape each blob shape must land in on a 148-SM GPU
LEAF_SHAPES = [
    (100 * 1000 + 7, 100, "hash_chunks_kernel", ""),                       # tiny chunks, ragged tail
    (100 * (64 << 10) + 4097, 64 << 10, "hash_chunks_split_kernel", ""),    # few chains
    (9_600 * 4096 + 100, 4096, "hash_chunks_pairs_kernel", ""),             # 300 groups
    (16_000 * 4096 + 64, 4096, "hash_chunks_sliced_kernel", "4 workers per SM"),
    (32_000 * 4096, 4096, "hash_chunks_sliced_kernel", "8 workers per SM"),
    (57_000 * 4096 + 5, 4096, "hash_chunks_sliced_kernel", "12 workers per SM"),
]


@pytest.mark.parametrize("nbytes,chunk,kernel,instance", LEAF_SHAPES)
def test_leaf_kernels_write_only_their_digests(ctx, nbytes, chunk, kernel, instance):
    data = inputs.uniform_bytes(nbytes, seed=11, device="cuda")
    host = _host(data)
    n = binding.n_chunks(nbytes, chunk)
    g = Guarded(32 * n)
    got = ctx.hash_chunks(data, chunk, out=g.as_(shape=(n, 32)))
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    if sms == 148:
        assert (ctx.last_leaf_kernel, ctx.last_leaf_instance) == (kernel, instance)
    g.check(kernel)
    assert np.array_equal(_host(got), oracle.hash_chunks(host, chunk, nthreads=oracle.host_threads()))
    # the same shape in the RFC 6962 mode (the prefixed instances of the same kernels)
    g2 = Guarded(32 * n)
    got2 = ctx.hash_chunks_rfc6962(data, chunk, out=g2.as_(shape=(n, 32)))
    if sms == 148 and kernel != "hash_chunks_kernel":
        assert (ctx.last_leaf_kernel, ctx.last_leaf_instance) == (kernel, instance)
    g2.check(kernel + " (prefixed)")
    assert np.array_equal(_host(got2), oracle.hash_chunks_rfc6962(host, chunk, nthreads=oracle.host_threads()))
    # and with SHA-384 digests
    g3 = Guarded(48 * n)
    got3 = ctx.hash_chunks_sha384(data, chunk, out=g3.as_(shape=(n, 48)))
    g3.check("sha384")
    assert np.array_equal(_host(got3), oracle.hash_chunks_sha384(host, chunk, nthreads=oracle.host_threads()))
    assert ctx.device_status() == 0


def test_tensor_kernels_write_only_their_digests(ctx):
    rng = np.random.default_rng(12)
    for n, hi, kernel in ((300, 50_000, "hash_chunks_split_kernel (tensors)"), (33_000, 600, "hash_ragged_kernel")):
        sizes = rng.integers(0, hi, size=n).astype(np.int64)
        offs = inputs.packed_offsets(sizes, first=3)
        base = inputs.uniform_bytes(int(offs[-1] + sizes[-1]) + 8, seed=13, device="cuda")
        g = Guarded(32 * n)
        got = ctx.hash_ragged(base, torch.from_numpy(offs).cuda(), torch.from_numpy(sizes).cuda(), out=g.as_(shape=(n, 32)))
        assert ctx.last_leaf_kernel == kernel
        g.check(kernel)
        assert np.array_equal(_host(got), oracle.hash_ragged(_host(base), offs, sizes, nthreads=oracle.host_threads()))


def test_resumable_hashing_writes_only_states_and_digests(ctx):
    n = 70
    rng = np.random.default_rng(14)
    sizes = rng.integers(0, 9000, size=n).astype(np.int64)
    offs = inputs.packed_offsets(sizes, first=1)
    base = inputs.uniform_bytes(int(offs[-1] + sizes[-1]) + 8, seed=15, device="cuda")
    cut = (sizes // 64 // 2) * 64
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int64)).cuda()
    gs = Guarded(ctypes.sizeof(ctypes.c_uint32) * 8 * n + 16 * n)           # n records of 48 bytes, zero-filled
    assert gs.nbytes == binding.Context.SHA_STATE_BYTES * n
    gd = Guarded(32 * n)
    states = gs.as_(shape=(n, 48))
    ctx.hash_ragged_update(base, dev(offs), dev(cut), states, finish=False)
    gs.check("states, first part")
    got = ctx.hash_ragged_update(base, dev(offs + cut), dev(sizes - cut), states, finish=True, out=gd.as_(shape=(n, 32)))
    gs.check("states, last part")
    gd.check("digests")
    assert np.array_equal(_host(got), oracle.hash_ragged(_host(base), offs, sizes, nthreads=oracle.host_threads()))


@pytest.mark.parametrize("n", [1, 2, 511, 513, 1000, 70_000, 300_001])
def test_merkle_passes_write_only_their_outputs(ctx, n):
    leaves = inputs.uniform_bytes(32 * n, seed=20 + n, device="cuda").view(n, 32)
    host = _host(leaves)
    want = oracle.merkle_root(host)
    g = Guarded(32, fill=0x11)
    ctx.merkle_root(leaves, out=g.as_())
    g.check("root")
    assert _host(g.view).tobytes() == want
    for levels in (1, 9, 10):
        n_out = n
        for _ in range(levels):
            n_out = (n_out + 1) // 2 if n_out > 1 else n_out
        gl = Guarded(32 * n_out)
        got = ctx.merkle_levels(leaves, levels, out=gl.as_(shape=(n_out, 32)))
        gl.check(f"levels {levels}")
        run = 1 << levels
        sample = sorted({0, n_out - 1, n_out // 2})
        for j in sample:
            assert _host(got[j]).tobytes() == oracle.merkle_root(host[j * run:(j + 1) * run]), (levels, j)
    records = ctx.tree_records(n)
    gt = Guarded(32 * records)
    tree = ctx.tree_build(leaves, out=gt.as_(shape=(records, 32)))
    gt.check("tree")
    assert _host(tree[-1]).tobytes() == want and np.array_equal(_host(tree[:n]), host)
    # the other trees
    g6 = Guarded(32)
    ctx.merkle_root_rfc6962(leaves, out=g6.as_())
    g6.check("rfc6962 root")
    assert _host(g6.view).tobytes() == oracle.merkle_root_rfc6962(host)
    n48 = (32 * n) // 48
    if n48:
        leaves48 = leaves.reshape(-1)[:48 * n48].view(n48, 48)
        g4 = Guarded(48)
        ctx.merkle_root_sha384(leaves48, out=g4.as_())
        g4.check("sha384 root")
        assert _host(g4.view).tobytes() == oracle.merkle_root_sha384(_host(leaves48))


def test_tree_update_writes_only_the_tree(ctx):
    chunk, n = 4096, 1000
    data = inputs.uniform_bytes(chunk * n - 17, seed=31, device="cuda")
    records = ctx.tree_records(n)
    gt = Guarded(32 * records)
    tree = ctx.tree_build(ctx.hash_chunks(data, chunk), out=gt.as_(shape=(records, 32)))
    dirty = torch.tensor([0, 999, 500, 1, 998, 500], dtype=torch.int64, device="cuda")
    data[dirty * chunk + 5] ^= 0x40
    ctx.tree_update(data, chunk, dirty, tree)
    gt.check("tree after update")
    want = oracle.hash_chunks(_host(data), chunk, nthreads=oracle.host_threads())
    assert np.array_equal(_host(tree[:n]), want) and _host(tree[-1]).tobytes() == oracle.merkle_root(want)
    assert ctx.device_status() == 0


def _tampered(nbytes, chunk, seed, flips):
    data = inputs.uniform_bytes(nbytes, seed=seed, device="cuda")
    host = _host(data)
    digests = oracle.hash_chunks(host, chunk, nthreads=oracle.host_threads())
    root = oracle.merkle_root(digests)
    rng = np.random.default_rng(seed)
    hit = sorted(int(v) for v in rng.choice(len(digests), size=flips, replace=False))
    for c in hit:
        data[min(c * chunk + 9, nbytes - 1)] ^= 0x02
    return data, digests, root, hit


@pytest.mark.parametrize("mode", ["default", "two_level", "rfc6962", "streamed", "batch", "sha384"])
def test_verification_writes_only_its_result_and_index_list(ctx, mode):
    """Six mismatches into an index list of four: the list is truncated, the count is not, and neither the
    48-byte (64-byte) result record nor the list spills over."""
    chunk, nbytes, cap = 8192, 700 * 8192 + 333, 4
    data, digests, root, hit = _tampered(nbytes, chunk, seed=40, flips=6)
    # manifests of the variants come from the oracle's variant functions over the UNTAMPERED bytes
    clean = data.clone()
    for c in hit:
        clean[min(c * chunk + 9, nbytes - 1)] ^= 0x02
    host_clean = _host(clean)
    gi = Guarded(8 * cap, fill=0xFF)
    idx = gi.as_(torch.int64)
    if mode == "sha384":
        d384 = oracle.hash_chunks_sha384(host_clean, chunk, nthreads=oracle.host_threads())
        r = ctx.verify_manifest_sha384(data, nbytes, chunk, torch.from_numpy(d384).cuda(), oracle.merkle_root_sha384(d384), idx)
        gi.check("index list (sha384)")
        assert (not r["root_ok"]) and r["n_mismatch"] == 6 and [int(v) for v in idx.cpu()] == hit[:cap]
        return
    gr = Guarded(48, fill=0xEE)
    res = gr.as_()
    if mode == "default":
        m = ctx.make_manifest(nbytes, chunk, torch.from_numpy(digests).cuda(), root)
        ctx.verify_manifest(data, m, res, idx)
    elif mode == "two_level":
        sub = 2048
        pieces = oracle.hash_chunks(host_clean, sub, nthreads=oracle.host_threads())
        per = chunk // sub
        d2 = np.stack([np.frombuffer(oracle.merkle_root(pieces[i * per:(i + 1) * per]), dtype=np.uint8)
                       for i in range(len(digests))])
        m = ctx.make_manifest(nbytes, chunk, torch.from_numpy(d2.copy()).cuda(), oracle.merkle_root(d2))
        ctx.verify_manifest_two_level(data, m, sub, res, idx)
    elif mode == "rfc6962":
        d6 = oracle.hash_chunks_rfc6962(host_clean, chunk, nthreads=oracle.host_threads())
        m = ctx.make_manifest(nbytes, chunk, torch.from_numpy(d6).cuda(), oracle.merkle_root_rfc6962(d6))
        ctx.verify_manifest_rfc6962(data, m, res, idx)
    elif mode == "streamed":
        m = ctx.make_manifest(nbytes, chunk, torch.from_numpy(digests).cuda(), root)
        ctx.verify_streamed(data.cpu().pin_memory(), 64 * chunk, nbytes, m, res, idx)
    elif mode == "batch":
        m = ctx.make_manifest(nbytes, chunk, torch.from_numpy(digests).cuda(), root)
        grb = Guarded(48 * 3, fill=0xEE)
        gib = Guarded(8 * cap * 3, fill=0xFF)
        ctx.verify_manifest_batch([clean, data, clean], m, grb.as_(shape=(3, 48)), gib.as_(torch.int64, (3, cap)))
        grb.check("batch results")
        gib.check("batch index lists")
        rs = binding.read_results(grb.as_(shape=(3, 48)))
        assert [x["n_mismatch"] for x in rs] == [0, 6, 0] and [x["root_ok"] for x in rs] == [True, False, True]
        assert [int(v) for v in gib.as_(torch.int64, (3, cap))[1].cpu()] == hit[:cap]
        return
    gr.check(f"result record ({mode})")
    gi.check(f"index list ({mode})")
    r = binding.read_result(res)
    assert r["status"] == 0 and (not r["root_ok"]) and r["n_mismatch"] == 6
    assert [int(v) for v in idx.cpu()] == hit[:cap]


def test_a_wait_that_runs_out_sets_the_status_and_returns(ctx):
    assert ctx.device_status() == 0
    limit = 2_000_000                                  # about a millisecond of SM clocks
    waited = ctx.selftest_wait_timeout(limit)
    assert limit <= waited < 100 * limit               # it gave up, and promptly
    assert ctx.device_status() == 1                    # IVK_DEV_TIMEOUT reaches the host ...
    assert ctx.device_status() == 0                    # ... and reading it clears it
    # a verification enqueued behind a timed-out kernel reports the status in its result record too
    data = inputs.uniform_bytes(64 * 4096, seed=50, device="cuda")
    digests = oracle.hash_chunks(_host(data), 4096)
    m = ctx.make_manifest(data.numel(), 4096, torch.from_numpy(digests).cuda(), oracle.merkle_root(digests))
    res = binding.new_result("cuda")
    ctx.selftest_wait_timeout(limit)
    ctx.verify_manifest(data, m, res, None)
    r = binding.read_result(res)
    assert r["status"] == 1 and r["root_ok"] and r["n_mismatch"] == 0
    assert ctx.device_status() == 1
    # and the context is as good as new
    ctx.verify_manifest(data, m, res, None)
    r = binding.read_result(res)
    assert r["status"] == 0 and r["root_ok"] and r["n_mismatch"] == 0 and ctx.device_status() == 0
    with pytest.raises(binding.IvError):
        ctx.selftest_wait_timeout(0)
