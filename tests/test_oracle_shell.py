"""Pins for the oracle's storage-shell arithmetic: key hash and payload checksum (CPU only)."""
import numpy as np

import oracle

M64 = (1 << 64) - 1


def test_fnv1a_published_vectors():
    # test vectors of the FNV-1a 64-bit reference suite
    assert oracle.fnv1a(b"") == 0xcbf29ce484222325
    assert oracle.fnv1a(b"a") == 0xaf63dc4c8601ec8c
    assert oracle.fnv1a(b"foobar") == 0x85944171f73967e8


def test_key_hash_is_fnv1a_of_little_endian_token_ids():
    rng = np.random.default_rng(1)
    for n in (0, 1, 5, 1000):
        toks = rng.integers(-2 ** 31, 2 ** 31 - 1, n).astype(np.int32)
        h = 0xcbf29ce484222325                                     # written out again with Python integers
        for b in toks.astype("<i4").tobytes():
            h = ((h ^ b) * 0x100000001b3) & M64
        assert oracle.key_hash(toks) == h == oracle.fnv1a(toks.astype("<i4").tobytes())
    assert oracle.key_hash([1, 2]) != oracle.key_hash([2, 1])


def test_checksum_by_hand_and_properties():
    K = 0x9E3779B9
    # two words 1 and 2: (1 ^ K) * 1 + (2 ^ K) * 3
    two = np.array([1, 0, 0, 0, 2, 0, 0, 0], dtype=np.uint8)
    assert oracle.checksum(two) == ((1 ^ K) * 1 + (2 ^ K) * 3) & M64
    assert oracle.checksum(np.zeros(0, dtype=np.uint8)) == 0
    assert oracle.checksum(np.zeros(8, dtype=np.uint8)) == (K * 1 + K * 3) & M64     # zeros still count, by position
    rng = np.random.default_rng(2)
    buf = rng.integers(0, 256, 4 * 1000, dtype=np.uint8)
    w = buf.view("<u4").astype(object)
    want = sum((int(x) ^ K) * ((2 * i + 1) & 0xffffffff) for i, x in enumerate(w)) & M64
    assert oracle.checksum(buf) == want
    # sensitive to a flipped bit, to swapped words, to truncation
    b2 = buf.copy(); b2[1234] ^= 0x10
    assert oracle.checksum(b2) != want
    b3 = buf.copy(); b3[0:4], b3[4:8] = buf[4:8].copy(), buf[0:4].copy()
    assert oracle.checksum(b3) != want
    assert oracle.checksum(buf[:-4]) != want
    # additive over a split when the second half's positions are accounted for: C(a|b) = C(a) + shifted C(b)
    a, b = buf[:2000], buf[2000:]
    wb = b.view("<u4").astype(object)
    shifted = sum((int(x) ^ K) * ((2 * (i + 500) + 1) & 0xffffffff) for i, x in enumerate(wb)) & M64
    assert (oracle.checksum(a) + shifted) & M64 == want
