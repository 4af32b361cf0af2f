"""Parity at the full sizes of the named configurations, in the launch configuration bench.py times.

The blobs are built by bench.py's own workload builder and hashed through the same entry points the
benchmark calls.  Every configuration is checked completely: the blob goes to the host window by window through a
pinned staging buffer, the oracle hashes every chunk (every tensor) on the host cores, and every digest,
the root, and the count and indices of seeded bit flips are compared bit for bit.  Manifests are built
from the ORACLE's digests and root, never from the library's own output.  At the largest size the RFC 6962
and SHA-384 variants are checked completely too; SHA-512 (the same kernel as SHA-384) is sampled."""
import numpy as np
import pytest
import torch

import bench
import oracle
from paper_2510_23938_b200 import binding, inputs

pytestmark = pytest.mark.gpu

GIB = 1 << 30


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available(), "the gpu-marked tests need a CUDA device"
    c = binding.Context(0)
    yield c
    c.close()


def _need(nbytes):
    free, _ = torch.cuda.mem_get_info(0)
    if free < nbytes:
        pytest.skip(f"needs {nbytes / GIB:.0f} GiB of free device memory, {free / GIB:.0f} GiB available")


def _host(t):
    return t.cpu().numpy()


def _oracle_digests_of_device_blob(data: torch.Tensor, chunk: int, piece: int = 1 * GIB) -> np.ndarray:
    """Oracle chunk digests of a device blob, brought to the host piece by piece (piece a multiple of chunk)."""
    piece -= piece % chunk
    out = []
    for off in range(0, data.numel(), piece):
        out.append(oracle.hash_chunks(_host(data[off:off + piece]), chunk, nthreads=oracle.host_threads()))
    return np.concatenate(out)


class _Stager:
    """Device bytes -> a numpy view of a reused pinned host buffer (valid until the next call)."""

    def __init__(self, capacity: int):
        self.buf = torch.empty(capacity, dtype=torch.uint8, pin_memory=True)

    def __call__(self, t: torch.Tensor) -> np.ndarray:
        n = t.numel()
        self.buf[:n].copy_(t)
        torch.cuda.synchronize()
        return self.buf[:n].numpy()


def _oracle_tensor_digests(data: torch.Tensor, offs: np.ndarray, lens: np.ndarray, stage: _Stager) -> np.ndarray:
    """Oracle digests of tensors laid out in ascending offset order, over consecutive runs of tensors that fit
    the staging buffer."""
    cap, n = stage.buf.numel(), len(lens)
    want = np.zeros((n, 32), dtype=np.uint8)
    threads = oracle.host_threads()
    k = 0
    while k < n:
        j = k + 1
        while j < n and int(offs[j] + lens[j] - offs[k]) <= cap:
            j += 1
        lo, hi = int(offs[k]), int(offs[j - 1] + lens[j - 1])
        assert hi - lo <= cap
        want[k:j] = oracle.hash_ragged(stage(data[lo:hi]), offs[k:j] - lo, lens[k:j], nthreads=threads)
        k = j
    return want


@pytest.mark.parametrize("cfg_id", [2, 3])
def test_weight_file_configurations_completely(ctx, cfg_id):
    _need((4 if cfg_id == 2 else 20) * GIB)
    wl = bench.build_workload(cfg_id, torch.device("cuda", 0), seed=1000)
    data, chunk = wl["data"], wl["chunk"]
    n = binding.n_chunks(data.numel(), chunk)
    assert n == (2501 if cfg_id == 2 else 3830)
    want = _oracle_digests_of_device_blob(data, chunk)
    want_root = oracle.merkle_root(want)
    got = ctx.hash_chunks(data, chunk)
    assert ctx.last_leaf_kernel == "hash_chunks_split_kernel"
    assert np.array_equal(_host(got), want)
    assert _host(ctx.merkle_root(got)).tobytes() == want_root
    # verification against the oracle's manifest: clean, then one flipped bit in the last (short) chunk
    manifest = ctx.make_manifest(data.numel(), chunk, torch.from_numpy(want).cuda(), want_root)
    res = binding.new_result("cuda")
    idx = torch.zeros(4, dtype=torch.int64, device="cuda")
    ctx.verify_manifest(data, manifest, res, idx)
    r = binding.read_result(res)
    assert r["root_ok"] and r["n_mismatch"] == 0 and r["root"] == want_root
    data[data.numel() - 2] ^= 0x10
    ctx.verify_manifest(data, manifest, res, idx)
    r = binding.read_result(res)
    assert (not r["root_ok"]) and r["n_mismatch"] == 1 and int(idx[0]) == n - 1
    data[data.numel() - 2] ^= 0x10
    # per-tensor digests of the same file: every tensor against the oracle
    table = wl["table"]
    offs = np.array([o for _, o, _ in table], dtype=np.int64)
    lens = np.array([ln for _, _, ln in table], dtype=np.int64)
    tens = ctx.hash_ragged(data, torch.from_numpy(offs).cuda(), torch.from_numpy(lens).cuda())
    assert ctx.device_status() == 0
    want_t = _oracle_tensor_digests(data, offs, lens, _Stager(2 * GIB))
    bad = np.nonzero((_host(tens) != want_t).any(axis=1))[0]
    assert bad.size == 0, [table[k][0] for k in bad[:8]]
    del data, wl
    torch.cuda.empty_cache()


def test_largest_configuration_completely(ctx):
    """112 GiB, 4 MiB chunks: the launch the benchmark times (migrating kernel, tiled copies, six workers
    per SM on the two progress-ordered queues), every one of its 28,672 digests against the oracle."""
    _need(125 * GIB)
    wl = bench.build_workload(4, torch.device("cuda", 0), seed=1000)
    data, chunk = wl["data"], wl["chunk"]
    nbytes = data.numel()
    n = binding.n_chunks(nbytes, chunk)
    assert n == 28_672
    got = ctx.hash_chunks(data, chunk)
    assert ctx.last_leaf_kernel == "hash_chunks_sliced_kernel" and ctx.device_status() == 0
    assert ctx.last_leaf_instance == "6 workers per SM"
    host_got = _host(got)

    # the oracle over the whole blob, one 4 GiB window at a time: SHA-256 chunk digests, and the RFC 6962 leaf hashes
    # and SHA-384 digests of the same chunks for the variants' legs below
    window = 4 * GIB
    stage = _Stager(window)
    threads = oracle.host_threads()
    parts, parts6962, parts384 = [], [], []
    for off in range(0, nbytes, window):
        host = stage(data[off:off + window])
        parts.append(oracle.hash_chunks(host, chunk, nthreads=threads))
        parts6962.append(oracle.hash_chunks_rfc6962(host, chunk, nthreads=threads))
        parts384.append(oracle.hash_chunks_sha384(host, chunk, nthreads=threads))
    want, want6962, want384 = np.concatenate(parts), np.concatenate(parts6962), np.concatenate(parts384)
    del parts, parts6962, parts384
    assert want.shape == (n, 32)
    bad = np.nonzero((host_got != want).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} digests differ from the oracle, first at chunk {bad[:8]}"
    want_root = oracle.merkle_root(want)
    assert _host(ctx.merkle_root(got)).tobytes() == want_root
    assert _host(ctx.merkle_root(ctx.merkle_levels(got, 9))).tobytes() == want_root
    assert _host(ctx.tree_build(got)[-1]).tobytes() == want_root

    # verification against the ORACLE's manifest: clean, then three seeded flipped bits
    manifest = ctx.make_manifest(nbytes, chunk, torch.from_numpy(want).cuda(), want_root)
    res = binding.new_result("cuda")
    idx = torch.full((8,), -1, dtype=torch.int64, device="cuda")
    ctx.verify_manifest(data, manifest, res, idx)
    assert ctx.last_leaf_kernel == "hash_chunks_sliced_kernel"
    r = binding.read_result(res)
    assert r["status"] == 0 and r["root_ok"] and r["n_mismatch"] == 0 and r["root"] == want_root
    flips = [inputs.flip_position(seed, nbytes) for seed in (2, 3, 4)]
    for off, bit in flips:
        data[off] ^= (1 << bit)
    touched = sorted({off // chunk for off, _ in flips})
    tampered = want.copy()
    for c in touched:
        d = oracle.sha256(stage(data[c * chunk:(c + 1) * chunk]))
        assert d != want[c].tobytes()
        tampered[c] = np.frombuffer(d, dtype=np.uint8)
    ctx.verify_manifest(data, manifest, res, idx)
    r = binding.read_result(res)
    assert r["status"] == 0 and (not r["root_ok"]) and r["n_mismatch"] == len(touched)
    assert [int(v) for v in idx[:len(touched)].cpu()] == touched
    assert r["root"] == oracle.merkle_root(tampered)
    assert np.array_equal(_host(ctx.last_digests(n)), tampered)
    for off, bit in flips:
        data[off] ^= (1 << bit)

    # the same launch shape in the RFC 6962 mode (prefixed instance of the migrating kernel) and with SHA-384 and
    # SHA-512 digests (the two-warp kernel on the slice FIFO, 256 slices per chunk): every digest; SHA-512 sampled
    got6962 = ctx.hash_chunks_rfc6962(data, chunk)
    assert ctx.last_leaf_kernel == "hash_chunks_sliced_kernel" and ctx.device_status() == 0
    bad = np.nonzero((_host(got6962) != want6962).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} RFC 6962 leaf hashes differ from the oracle, first at chunk {bad[:8]}"
    assert _host(ctx.merkle_root_rfc6962(got6962)).tobytes() == oracle.merkle_root_rfc6962(want6962)
    del got6962
    got384 = ctx.hash_chunks_sha384(data, chunk)
    assert ctx.last_leaf_kernel == "hash_sha512_pairs_kernel" and ctx.device_status() == 0
    bad = np.nonzero((_host(got384) != want384).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} SHA-384 digests differ from the oracle, first at chunk {bad[:8]}"
    assert _host(ctx.merkle_root_sha384(got384)).tobytes() == oracle.merkle_root_sha384(want384)
    del got384
    rng = np.random.default_rng(4)
    sample = sorted(set([0, 1, 31, 32, 1023, 1024, n - 33, n - 32, n - 1] + [int(v) for v in rng.integers(0, n, size=12)]))
    got512 = _host(ctx.hash_chunks_sha512(data, chunk))
    assert ctx.device_status() == 0
    for i in sample:
        assert got512[i].tobytes() == oracle.sha512(stage(data[i * chunk:(i + 1) * chunk])), i
    del got512

    # streamed from pinned host windows (a ring of two 4 GiB windows read as windows 0 and 1 of the blob),
    # against the oracle's digests of those windows
    ring = [torch.empty(window, dtype=torch.uint8, pin_memory=True) for _ in range(2)]
    for w in range(2):
        ring[w].copy_(data[w * window:(w + 1) * window])
    per = window // chunk
    sub_manifest = ctx.make_manifest(2 * window, chunk, torch.from_numpy(want[:2 * per].copy()).cuda(),
                                     oracle.merkle_root(want[:2 * per]))
    ctx.verify_streamed(ring, window, 2 * window, sub_manifest, res, idx)
    r = binding.read_result(res)
    assert r["status"] == 0 and r["root_ok"] and r["n_mismatch"] == 0
    del data, wl, ring, stage
    torch.cuda.empty_cache()


@pytest.mark.parametrize("groups,chunk,instance", [(750, 2 << 20, "5 workers per SM"), (900, 1 << 20, "6 workers per SM"),
                                                   (1_040, 1 << 20, "7 workers per SM")])
def test_progress_ordered_queues_with_64_and_128_slices_per_chunk(ctx, groups, chunk, instance):
    """The launch shapes whose workers differ in speed (six or seven per SM, tasks from the two progress-ordered
    queues) with 64 or 128 slices per chunk: 28 to 47 GiB in chunks of 1 or 2 MiB, every digest and the root against
    the oracle, the last shape in the RFC 6962 mode as well."""
    n = groups * 32 - 5
    nbytes = n * chunk - 12_344                       # short last chunk beside the main launch
    torch.cuda.empty_cache()
    _need(nbytes + 4 * GIB)
    data = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    for off in range(0, nbytes, GIB):
        inputs.fill_bf16_normal(data[off:off + GIB], 77, first_elem=off // 2)
    want = _oracle_digests_of_device_blob(data, chunk)
    got = ctx.hash_chunks(data, chunk)
    assert (ctx.last_leaf_kernel, ctx.last_leaf_instance) == ("hash_chunks_sliced_kernel", instance)
    assert ctx.device_status() == 0
    assert np.array_equal(_host(got), want)
    assert _host(ctx.merkle_root(got)).tobytes() == oracle.merkle_root(want)
    if groups != 1_040:
        return                                        # the prefixed instance is held against the oracle on the other shape
    got6962 = ctx.hash_chunks_rfc6962(data, chunk)
    assert (ctx.last_leaf_kernel, ctx.last_leaf_instance) == ("hash_chunks_sliced_kernel", instance)
    want6962 = np.concatenate([oracle.hash_chunks_rfc6962(_host(data[o:o + GIB]), chunk, nthreads=oracle.host_threads())
                               for o in range(0, nbytes, GIB)])
    assert np.array_equal(_host(got6962), want6962) and ctx.device_status() == 0


def test_ragged_configuration_completely(ctx):
    """10,000 tensors, log-uniform 4 KiB .. 64 MiB, packed at 2-byte alignment (about 69 GB): every tensor
    digest and the root over them against the oracle."""
    _need(75 * GIB)
    wl = bench.build_workload(5, torch.device("cuda", 0), seed=1000)
    data, offs, lens = wl["data"], wl["offsets"], wl["lengths"]
    assert len(lens) == 10_000 and 60e9 < lens.sum() < 80e9
    got = ctx.hash_ragged(data, torch.from_numpy(offs).cuda(), torch.from_numpy(lens).cuda())
    assert ctx.last_leaf_kernel.startswith("hash_chunks_split_kernel") and ctx.device_status() == 0
    host_got = _host(got)
    stage = _Stager(4 * GIB)
    want = _oracle_tensor_digests(data, offs, lens, stage)
    bad = np.nonzero((host_got != want).any(axis=1))[0]
    assert bad.size == 0, f"{bad.size} tensor digests differ from the oracle, first at {bad[:8]}"
    # the root over the tensor digests in index order
    assert _host(ctx.merkle_root(got)).tobytes() == oracle.merkle_root(want)
    del data, wl, stage
    torch.cuda.empty_cache()
