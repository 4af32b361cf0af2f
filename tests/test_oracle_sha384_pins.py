"""Pins for the oracle's SHA-384 variant: FIPS example digests, spot values of the derived constants,
hashlib on every length around the 128-byte padding boundaries, tree closed forms, tamper detection."""
import hashlib
import os

import numpy as np
import pytest

import oracle
from test_oracle_pins import _read_vectors


def test_constants_spot_values_from_fips_180_4():
    """First and last round constant (section 4.2.3) and the SHA-384 initial value (section 5.3.4)."""
    k, h0 = oracle.constants512()
    assert int(k[0]) == 0x428A2F98D728AE22 and int(k[1]) == 0x7137449123EF65CD
    assert int(k[79]) == 0x6C44198C4A475817
    assert int(h0[0]) == 0xCBBB9D5DC1059ED8 and int(h0[7]) == 0x47B5481DBEFA4FA4
    # the high halves of the first 64 SHA-512 constants are the SHA-256 constants (same cube roots)
    k256, _ = oracle.constants()
    assert [int(v) >> 32 for v in k[:64]] == [int(v) for v in k256]


def test_fips_example_digests(golden_dir):
    vectors = _read_vectors(os.path.join(golden_dir, "fips180_4_sha384_vectors.txt"))
    assert len(vectors) == 4
    for spec, msg, digest in vectors:
        assert oracle.sha384(msg) == digest, spec


def test_sha384_equals_hashlib_every_length_0_to_400():
    rng = np.random.default_rng(384)
    blob = rng.integers(0, 256, size=500, dtype=np.uint8).tobytes()
    for n in range(0, 401):
        assert oracle.sha384(blob[:n]) == hashlib.sha384(blob[:n]).digest(), n


@pytest.mark.parametrize("n", [111, 112, 113, 127, 128, 129, 239, 240, 241, 255, 256, 257, 65536, (1 << 20) + 1])
def test_sha384_equals_hashlib_boundaries(n):
    msg = np.random.default_rng(n).integers(0, 256, size=n, dtype=np.uint8).tobytes()
    assert oracle.sha384(msg) == hashlib.sha384(msg).digest()


def test_chunk_digests_and_tree_closed_forms():
    rng = np.random.default_rng(5)
    blob = rng.integers(0, 256, size=10_000, dtype=np.uint8).tobytes()
    H = lambda b: hashlib.sha384(b).digest()
    for c in (1, 127, 128, 129, 1000, 4096, 10_000, 10_001):
        got = oracle.hash_chunks_sha384(blob, c)
        for i in range(-(-len(blob) // c)):
            assert got[i].tobytes() == H(blob[i * c:(i + 1) * c]), (c, i)
    d = [H(b"leaf-%d" % i) for i in range(5)]
    assert oracle.merkle_root_sha384(b"") == H(b"")
    assert oracle.merkle_root_sha384(d[0]) == d[0]
    assert oracle.merkle_root_sha384(d[0] + d[1]) == H(d[0] + d[1])
    assert oracle.merkle_root_sha384(b"".join(d[:3])) == H(H(d[0] + d[1]) + d[2])
    assert oracle.merkle_root_sha384(b"".join(d[:4])) == H(H(d[0] + d[1]) + H(d[2] + d[3]))
    assert oracle.merkle_root_sha384(b"".join(d[:5])) == H(H(H(d[0] + d[1]) + H(d[2] + d[3])) + d[4])
    assert np.array_equal(oracle.hash_chunks_sha384(blob, 100, nthreads=4), oracle.hash_chunks_sha384(blob, 100))


def test_every_bit_of_a_two_block_message_matters():
    base = bytes(range(140))
    seen = {oracle.sha384(base)}
    for bit in range(140 * 8):
        m = bytearray(base)
        m[bit // 8] ^= 1 << (bit % 8)
        seen.add(oracle.sha384(bytes(m)))
    assert len(seen) == 140 * 8 + 1
