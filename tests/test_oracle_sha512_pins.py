"""Pins for the oracle's SHA-512 variant: the FIPS 180-4 example digests, the initial value as printed in
section 5.3.5, hashlib on every length around the 128-byte padding boundaries, tree closed forms."""
import hashlib
import os

import numpy as np
import pytest

import oracle
from test_oracle_pins import _read_vectors


def test_initial_value_as_printed_in_fips_180_4_section_5_3_5():
    h0 = [int(v) for v in oracle.h0_sha512()]
    assert h0 == [0x6A09E667F3BCC908, 0xBB67AE8584CAA73B, 0x3C6EF372FE94F82B, 0xA54FF53A5F1D36F1,
                  0x510E527FADE682D1, 0x9B05688C2B3E6C1F, 0x1F83D9ABFB41BD6B, 0x5BE0CD19137E2179]
    # the high halves are the SHA-256 initial value (the same square roots, section 5.3.3)
    _, h256 = oracle.constants()
    assert [v >> 32 for v in h0] == [int(v) for v in h256]


def test_fips_example_digests(golden_dir):
    vectors = _read_vectors(os.path.join(golden_dir, "fips180_4_sha512_vectors.txt"))
    assert len(vectors) == 4
    for spec, msg, digest in vectors:
        assert len(digest) == 64
        assert oracle.sha512(msg) == digest, spec


def test_sha512_equals_hashlib_every_length_0_to_400():
    rng = np.random.default_rng(512)
    blob = rng.integers(0, 256, size=500, dtype=np.uint8).tobytes()
    for n in range(0, 401):
        assert oracle.sha512(blob[:n]) == hashlib.sha512(blob[:n]).digest(), n


@pytest.mark.parametrize("n", [111, 112, 113, 127, 128, 129, 239, 240, 241, 255, 256, 257, 65536, (1 << 20) + 1])
def test_sha512_equals_hashlib_boundaries(n):
    msg = np.random.default_rng(n).integers(0, 256, size=n, dtype=np.uint8).tobytes()
    assert oracle.sha512(msg) == hashlib.sha512(msg).digest()


def test_sha384_is_not_a_truncation_of_sha512():
    """Different initial values (sections 5.3.4 and 5.3.5): the first 48 bytes differ."""
    assert oracle.sha512(b"abc")[:48] != oracle.sha384(b"abc")


def test_chunk_digests_and_tree_closed_forms():
    rng = np.random.default_rng(6)
    blob = rng.integers(0, 256, size=10_000, dtype=np.uint8).tobytes()
    H = lambda b: hashlib.sha512(b).digest()
    for c in (1, 127, 128, 129, 1000, 4096, 10_000, 10_001):
        got = oracle.hash_chunks_sha512(blob, c)
        for i in range(-(-len(blob) // c)):
            assert got[i].tobytes() == H(blob[i * c:(i + 1) * c]), (c, i)
    d = [H(b"leaf-%d" % i) for i in range(5)]
    assert oracle.merkle_root_sha512(b"") == H(b"")
    assert oracle.merkle_root_sha512(d[0]) == d[0]
    assert oracle.merkle_root_sha512(d[0] + d[1]) == H(d[0] + d[1])
    assert oracle.merkle_root_sha512(b"".join(d[:3])) == H(H(d[0] + d[1]) + d[2])
    assert oracle.merkle_root_sha512(b"".join(d[:4])) == H(H(d[0] + d[1]) + H(d[2] + d[3]))
    assert oracle.merkle_root_sha512(b"".join(d[:5])) == H(H(H(d[0] + d[1]) + H(d[2] + d[3])) + d[4])
    assert np.array_equal(oracle.hash_chunks_sha512(blob, 100, nthreads=4), oracle.hash_chunks_sha512(blob, 100))


def test_every_bit_of_a_two_block_message_matters():
    base = bytes(range(140))
    seen = {oracle.sha512(base)}
    for bit in range(140 * 8):
        m = bytearray(base)
        m[bit // 8] ^= 1 << (bit % 8)
        seen.add(oracle.sha512(bytes(m)))
    assert len(seen) == 140 * 8 + 1
