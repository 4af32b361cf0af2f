"""Pins for the CPU oracle: it is checked against things other than itself.

 * the constants and example digests printed in FIPS 180-4 (tests/golden/),
 * Python's hashlib (an unrelated library SHA-256) on seeded random messages of
   every length around the padding boundaries,
 * the Merkle closed forms for 1..5 leaves, the perfect-tree special case and
   the equality of the level-by-level and the recursive definitions,
 * chunking special cases (one chunk, short last chunk, window-split invariance),
 * brute force: every single-bit flip of a tiny blob is detected at exactly the
   chunk that holds the bit.
"""
import hashlib
import os

import numpy as np
import pytest

import oracle


def _words(line):
    return bytes.fromhex("".join(line.split()))


def _read_vectors(path):
    lines = [ln.strip() for ln in open(path) if ln.strip() and not ln.startswith("#")]
    out = []
    for spec, digest in zip(lines[0::2], lines[1::2]):
        if spec == "empty":
            msg = b""
        elif spec.startswith("ascii:"):
            msg = spec[len("ascii:"):].encode("ascii")
        elif spec.startswith("repeat:"):
            _, count, text = spec.split(":", 2)
            msg = text.encode("ascii") * int(count)
        else:  # pragma: no cover
            raise ValueError(spec)
        out.append((spec, msg, _words(digest)))
    return out


# --------------------------------------------------------------------------- constants

def test_constants_match_fips_tables(golden_dir):
    """K and H0 derived from prime roots equal the tables typed from FIPS 180-4 4.2.2 / 5.3.3."""
    text = [ln.strip() for ln in open(os.path.join(golden_dir, "fips180_4_sha256_constants.txt"))
            if ln.strip() and not ln.startswith("#")]
    k_lines = text[text.index("K") + 1:text.index("H0")]
    h_lines = text[text.index("H0") + 1:]
    k_gold = [int(w, 16) for ln in k_lines for w in ln.split()]
    h_gold = [int(w, 16) for ln in h_lines for w in ln.split()]
    assert len(k_gold) == 64 and len(h_gold) == 8
    k, h0 = oracle.constants()
    assert [int(v) for v in k] == k_gold
    assert [int(v) for v in h0] == h_gold
    assert k_gold[0] == 0x428A2F98 and k_gold[63] == 0xC67178F2
    assert h_gold[0] == 0x6A09E667 and h_gold[7] == 0x5BE0CD19


# --------------------------------------------------------------------------- SHA-256

def test_fips_example_digests(golden_dir):
    vectors = _read_vectors(os.path.join(golden_dir, "fips180_4_sha256_vectors.txt"))
    assert len(vectors) == 4
    for spec, msg, digest in vectors:
        assert oracle.sha256(msg) == digest, spec


def test_sha256_equals_hashlib_every_length_0_to_300():
    rng = np.random.default_rng(1234)
    blob = rng.integers(0, 256, size=400, dtype=np.uint8).tobytes()
    for n in range(0, 301):
        assert oracle.sha256(blob[:n]) == hashlib.sha256(blob[:n]).digest(), n


@pytest.mark.parametrize("n", [55, 56, 57, 63, 64, 65, 119, 120, 121, 127, 128, 129,
                               4095, 4096, 65536, (1 << 20) - 1, 1 << 20, (1 << 20) + 1])
def test_sha256_equals_hashlib_boundaries(n):
    rng = np.random.default_rng(n)
    msg = rng.integers(0, 256, size=n, dtype=np.uint8).tobytes()
    assert oracle.sha256(msg) == hashlib.sha256(msg).digest()


def test_sha256_is_sensitive_to_every_input_bit_of_a_two_block_message():
    """A dropped word or a wrong index in the schedule would leave some bit without effect."""
    base = bytes(range(70))
    ref = oracle.sha256(base)
    seen = {ref}
    for bit in range(70 * 8):
        m = bytearray(base)
        m[bit // 8] ^= 1 << (bit % 8)
        d = oracle.sha256(bytes(m))
        assert d == hashlib.sha256(bytes(m)).digest()
        seen.add(d)
    assert len(seen) == 70 * 8 + 1


# --------------------------------------------------------------------------- Merkle

def _leaves(n, seed=0):
    return b"".join(hashlib.sha256(bytes([seed & 0xFF, i & 0xFF, i >> 8])).digest()
                    for i in range(n))


def _H(b):
    return hashlib.sha256(b).digest()


def test_merkle_golden_roots_1_to_5(golden_dir):
    rows = [ln.split() for ln in open(os.path.join(golden_dir, "merkle_single_byte_leaves.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert [int(r[0]) for r in rows] == [1, 2, 3, 4, 5]
    leaves = [_H(bytes([i])) for i in range(5)]
    for n_str, root_hex in rows:
        n = int(n_str)
        assert oracle.merkle_root(b"".join(leaves[:n])).hex() == root_hex
        assert oracle.merkle_root(b"".join(leaves[:n]), recursive=True).hex() == root_hex


def test_merkle_closed_forms_with_hashlib():
    d = [_H(b"leaf-%d" % i) for i in range(5)]
    assert oracle.merkle_root(d[0]) == d[0]
    assert oracle.merkle_root(d[0] + d[1]) == _H(d[0] + d[1])
    assert oracle.merkle_root(b"".join(d[:3])) == _H(_H(d[0] + d[1]) + d[2])
    assert oracle.merkle_root(b"".join(d[:4])) == _H(_H(d[0] + d[1]) + _H(d[2] + d[3]))
    assert oracle.merkle_root(b"".join(d[:5])) == _H(_H(_H(d[0] + d[1]) + _H(d[2] + d[3])) + d[4])


def test_merkle_zero_leaves_is_empty_string_digest():
    assert oracle.merkle_root(b"") == hashlib.sha256(b"").digest()


def test_merkle_perfect_tree_equals_textbook_reduction():
    for k in range(0, 8):
        n = 1 << k
        level = [_leaves(n, 7)[32 * i:32 * i + 32] for i in range(n)]
        flat = b"".join(level)
        while len(level) > 1:
            level = [_H(level[i] + level[i + 1]) for i in range(0, len(level), 2)]
        assert oracle.merkle_root(flat) == level[0]


def test_merkle_iterative_equals_recursive_split_1_to_300():
    flat = _leaves(300, 3)
    for n in range(1, 301):
        assert oracle.merkle_root(flat[:32 * n]) == oracle.merkle_root(flat[:32 * n], recursive=True), n


def test_merkle_aligned_power_of_two_runs_are_tree_nodes():
    """Replacing an aligned run of 2^k leaves by its own root one level up gives the same root."""
    n = 77
    flat = _leaves(n, 9)
    run = 8
    nodes = b"".join(oracle.merkle_root(flat[32 * s:32 * min(s + run, n)]) for s in range(0, n, run))
    assert oracle.merkle_root(nodes) == oracle.merkle_root(flat)


def test_merkle_root_depends_on_leaf_order_and_every_leaf():
    flat = bytearray(_leaves(9, 5))
    ref = oracle.merkle_root(bytes(flat))
    swapped = bytearray(flat)
    swapped[0:32], swapped[32:64] = flat[32:64], flat[0:32]
    assert oracle.merkle_root(bytes(swapped)) != ref
    for i in range(9):
        m = bytearray(flat)
        m[32 * i + 31] ^= 1
        assert oracle.merkle_root(bytes(m)) != ref


# --------------------------------------------------------------------------- chunking

def test_chunk_digests_equal_hashlib_per_chunk_with_short_last_chunk():
    rng = np.random.default_rng(5)
    blob = rng.integers(0, 256, size=10_000, dtype=np.uint8).tobytes()
    for c in (1, 63, 64, 65, 1000, 4096, 9999, 10_000, 10_001, 1 << 20):
        got = oracle.hash_chunks(blob, c)
        n = -(-len(blob) // c)
        assert got.shape == (n, 32)
        for i in range(n):
            assert got[i].tobytes() == hashlib.sha256(blob[i * c:(i + 1) * c]).digest(), (c, i)


def test_single_chunk_root_is_plain_digest_and_empty_blob_has_no_chunks():
    blob = bytes(range(200))
    d = oracle.hash_chunks(blob, 4096)
    assert d.shape == (1, 32)
    assert oracle.merkle_root(d) == hashlib.sha256(blob).digest()
    assert oracle.hash_chunks(b"", 64).shape == (0, 32)


def test_window_split_invariance_and_threads():
    rng = np.random.default_rng(6)
    blob = rng.integers(0, 256, size=64 * 37 + 11, dtype=np.uint8).tobytes()
    c = 64
    whole = oracle.hash_chunks(blob, c)
    for window in (c, 3 * c, 16 * c):
        parts = [oracle.hash_chunks(blob[o:o + window], c) for o in range(0, len(blob), window)]
        assert np.array_equal(np.concatenate(parts), whole)
    assert np.array_equal(oracle.hash_chunks(blob, c, nthreads=4), whole)


# --------------------------------------------------------------------------- verify

def _manifest(blob, c):
    digests = np.frombuffer(b"".join(hashlib.sha256(blob[o:o + c]).digest()
                                     for o in range(0, len(blob), c)), dtype=np.uint8)
    return digests, oracle.merkle_root(digests)


@pytest.mark.parametrize("n_chunks,c,last", [(4, 64, 64), (5, 100, 37), (7, 200, 1), (6, 65, 65)])
def test_every_single_bit_flip_is_found_at_its_chunk(n_chunks, c, last):
    rng = np.random.default_rng(n_chunks * 1000 + c)
    size = (n_chunks - 1) * c + last
    blob = rng.integers(0, 256, size=size, dtype=np.uint8).tobytes()
    digests, root = _manifest(blob, c)
    ok, bad, idx, got_root = oracle.verify(blob, c, digests, root)
    assert ok and bad == 0 and idx == [] and got_root == root
    for bit in range(size * 8):
        m = bytearray(blob)
        m[bit // 8] ^= 1 << (bit % 8)
        ok, bad, idx, got_root = oracle.verify(bytes(m), c, digests, root)
        assert not ok and bad == 1 and idx == [bit // 8 // c], bit
        assert got_root != root


def test_manifest_side_tampering_and_truncated_index_list():
    rng = np.random.default_rng(11)
    c = 128
    blob = rng.integers(0, 256, size=c * 9 + 5, dtype=np.uint8).tobytes()
    digests, root = _manifest(blob, c)
    man = digests.copy()
    man[32 * 3] ^= 0x80                      # manifest digest 3 altered, manifest root intact
    ok, bad, idx, _ = oracle.verify(blob, c, man, root)
    assert ok and bad == 1 and idx == [3]
    bad_root = bytes([root[0] ^ 1]) + root[1:]
    ok, bad, idx, _ = oracle.verify(blob, c, digests, bad_root)
    assert (not ok) and bad == 0 and idx == []
    m = bytearray(blob)
    for chunk in (1, 4, 6, 9):
        m[chunk * c] ^= 0xFF
    ok, bad, idx, _ = oracle.verify(bytes(m), c, digests, root, idx_cap=2)
    assert (not ok) and bad == 4 and idx == [1, 4]      # count exact, list truncated, ascending
    ok, bad, idx, _ = oracle.verify(bytes(m), c, digests, root)
    assert idx == [1, 4, 6, 9]


# --------------------------------------------------------------------------- ragged

def test_ragged_equals_hashlib_any_offset_and_length():
    rng = np.random.default_rng(21)
    base = rng.integers(0, 256, size=20_000, dtype=np.uint8).tobytes()
    lengths = [0, 1, 55, 56, 64, 4096, 63, 65, 119, 120, 1000, 3, 0, 777]
    offsets = [0, 1, 2, 3, 5, 7, 9, 11, 13, 15, 16, 17, 19_999, 6000]
    got = oracle.hash_ragged(base, offsets, lengths)
    for k, (o, n) in enumerate(zip(offsets, lengths)):
        assert got[k].tobytes() == hashlib.sha256(base[o:o + n]).digest(), k
    assert np.array_equal(oracle.hash_ragged(base, offsets, lengths, nthreads=3), got)
    # the root over tensor digests is order sensitive
    swapped = got.copy()
    swapped[[1, 2]] = swapped[[2, 1]]
    assert oracle.merkle_root(swapped) != oracle.merkle_root(got)
