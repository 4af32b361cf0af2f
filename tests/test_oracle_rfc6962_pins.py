"""Pins of the oracle's RFC 6962 mode (section 2.1 of the RFC, which the paper cites for its tree).

The RFC prints no numeric examples, so the pins are: hashlib on the same prefixed bytes (another
SHA-256), the tree folded bottom-up in Python (the oracle recurses top-down), the relation to the
unprefixed tree, and the property the prefixes exist for."""
import hashlib

import numpy as np
import pytest

import oracle
from paper_2510_23938_b200 import inputs


def _levelwise_root(leaf_hashes):
    """Bottom-up fold, odd node promoted: the same tree as the RFC's split at the largest power of two."""
    level = list(leaf_hashes)
    if not level:
        return hashlib.sha256(b"").digest()
    while len(level) > 1:
        nxt = [hashlib.sha256(b"\x01" + level[i] + level[i + 1]).digest() for i in range(0, len(level) - 1, 2)]
        if len(level) % 2:
            nxt.append(level[-1])
        level = nxt
    return level[0]


@pytest.mark.parametrize("nbytes,chunk", [(1, 1), (55, 64), (56, 64), (63, 64), (64, 64), (65, 64), (1000, 7),
                                          (4096 * 5 + 63, 4096), (100_003, 1001)])
def test_leaf_hashes_are_sha256_of_zero_byte_then_chunk(nbytes, chunk):
    data = inputs.uniform_bytes(nbytes, seed=62).numpy()
    got = oracle.hash_chunks_rfc6962(data, chunk)
    raw = data.tobytes()
    want = [hashlib.sha256(b"\x00" + raw[o:o + chunk]).digest() for o in range(0, nbytes, chunk)]
    assert [bytes(r) for r in got] == want


def test_threaded_leaves_equal_single_threaded():
    data = inputs.uniform_bytes(300_000, seed=63).numpy()
    assert np.array_equal(oracle.hash_chunks_rfc6962(data, 1000, nthreads=4), oracle.hash_chunks_rfc6962(data, 1000))


@pytest.mark.parametrize("n", list(range(0, 20)) + [31, 32, 33, 100, 257])
def test_root_equals_bottom_up_fold_with_hashlib(n):
    leaves = inputs.uniform_bytes(32 * n, seed=64 + n).numpy().reshape(n, 32)
    assert oracle.merkle_root_rfc6962(leaves) == _levelwise_root([bytes(r) for r in leaves])


def test_small_trees_written_out():
    h = lambda b: hashlib.sha256(b).digest()
    d = [bytes([i]) * 3 for i in range(3)]
    leaves = [h(b"\x00" + x) for x in d]
    data = np.frombuffer(b"".join(d), dtype=np.uint8)
    assert [bytes(r) for r in oracle.hash_chunks_rfc6962(data, 3)] == leaves
    arr = np.frombuffer(b"".join(leaves), dtype=np.uint8)
    assert oracle.merkle_root_rfc6962(arr[:0]) == h(b"")
    assert oracle.merkle_root_rfc6962(arr[:32]) == leaves[0]
    assert oracle.merkle_root_rfc6962(arr[:64]) == h(b"\x01" + leaves[0] + leaves[1])
    assert oracle.merkle_root_rfc6962(arr) == h(b"\x01" + h(b"\x01" + leaves[0] + leaves[1]) + leaves[2])


def test_prefixes_separate_a_leaf_from_a_node_with_the_same_bytes():
    # Without prefixes a 64-byte chunk equal to left || right hashes to that pair's parent; with them it cannot.
    pair = inputs.uniform_bytes(64, seed=65).numpy()
    assert oracle.sha256(pair) == oracle.merkle_root(pair)                      # the unprefixed tree collides
    leaf = bytes(oracle.hash_chunks_rfc6962(pair, 64)[0])
    node = oracle.merkle_root_rfc6962(pair)
    assert leaf != node
    assert leaf == hashlib.sha256(b"\x00" + pair.tobytes()).digest()
    assert node == hashlib.sha256(b"\x01" + pair.tobytes()).digest()


def test_mode_differs_from_the_default_tree_on_the_same_data():
    data = inputs.uniform_bytes(8192, seed=66).numpy()
    a = oracle.merkle_root(oracle.hash_chunks(data, 1024))
    b = oracle.merkle_root_rfc6962(oracle.hash_chunks_rfc6962(data, 1024))
    assert a != b
