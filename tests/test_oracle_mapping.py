"""Pins for the oracle's gather / scatter / block mapping (CPU only).

The oracle's loops are checked against formulations that share nothing with them: numpy advanced
indexing, plain slices, and algebraic invariants.
"""
import numpy as np
import pytest

import oracle
from paper_2409_13761_b200 import synth


def rand_pool(rng, L, H, D, bs, nb):
    return rng.integers(0, 1 << 16, size=(L, 2, nb, bs, H, D), dtype=np.uint16)


def fancy_store_raw(pool, table, off, T):
    """chunk[l][kv][t][h][d] = pool[l][kv][table[p // bs]][p % bs][h][d], p = off + t, by advanced indexing."""
    bs = pool.shape[3]
    p = off + np.arange(T)
    return pool[:, :, table[p // bs], p % bs]          # [L][2][T][H][D]


@pytest.mark.parametrize("bs", [1, 2, 3, 16])
@pytest.mark.parametrize("L,H,D", [(1, 1, 64), (2, 2, 64), (2, 3, 8)])
def test_store_raw_equals_advanced_indexing_all_offsets(bs, L, H, D):
    rng = np.random.default_rng(7 + bs)
    nb = 12
    pool = rand_pool(rng, L, H, D, bs, nb)
    n_table = 6
    table = rng.permutation(nb)[:n_table].astype(np.int32)
    span = n_table * bs
    for off in range(0, span):
        for T in sorted({0, 1, 2, bs, bs + 1, min(40, span - off), span - off}):
            if T < 0 or off + T > span:
                continue
            got = oracle.store(pool, table, off, T, oracle.RAW_BF16).view(np.uint16)
            want = fancy_store_raw(pool, table, off, T).reshape(-1)
            assert np.array_equal(got, want), (bs, off, T)


def test_store_allows_repeated_source_blocks():
    rng = np.random.default_rng(3)
    pool = rand_pool(rng, 2, 2, 64, 4, 5)
    table = np.array([3, 3, 0, 3], dtype=np.int32)
    got = oracle.store(pool, table, 2, 13, oracle.RAW_BF16).view(np.uint16)
    assert np.array_equal(got, fancy_store_raw(pool, table, 2, 13).reshape(-1))


def test_contiguous_table_is_a_slice():
    """Identity table, offset 0: the chunk is pool[l][kv] flattened and cut at T tokens."""
    rng = np.random.default_rng(11)
    L, H, D, bs, nb = 2, 2, 64, 16, 8
    pool = rand_pool(rng, L, H, D, bs, nb)
    table = np.arange(nb, dtype=np.int32)
    for T in (1, 16, 37, nb * bs):
        got = oracle.store(pool, table, 0, T, oracle.RAW_BF16).view(np.uint16).reshape(L, 2, T, H, D)
        want = pool.reshape(L, 2, nb * bs, H, D)[:, :, :T]
        assert np.array_equal(got, want)


def special_bit_patterns():
    # +-0, subnormals, smallest/largest normals, +-inf, quiet and signalling NaNs with payloads
    return np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x007f, 0x0080, 0x7f7f, 0xff7f, 0x7f80, 0xff80,
                     0x7fc0, 0xffc0, 0x7f81, 0x7fff, 0xffff, 0x3f80, 0xbf80, 0x1234, 0xfedc],
                    dtype=np.uint16)


def test_store_then_retrieve_is_identity_on_raw_bits():
    rng = np.random.default_rng(5)
    L, H, D, bs, nb = 2, 2, 64, 4, 16
    pool = rand_pool(rng, L, H, D, bs, nb)
    sp = special_bit_patterns()
    pool.reshape(-1)[: sp.size * 50] = np.tile(sp, 50)          # every class, many places
    src = rng.permutation(nb)[:5].astype(np.int32)
    dst = np.setdiff1d(np.arange(nb), src)[:5].astype(np.int32)
    rng.shuffle(dst)
    off, T = 3, 15
    chunk = oracle.store(pool, src, off, T, oracle.RAW_BF16)
    out = pool.copy()
    oracle.retrieve(out, dst, off, T, oracle.RAW_BF16, chunk)
    p = off + np.arange(T)
    assert np.array_equal(out[:, :, dst[p // bs], p % bs], pool[:, :, src[p // bs], p % bs])
    # and storing it again from the new place gives the same bytes
    assert np.array_equal(oracle.store(out, dst, off, T, oracle.RAW_BF16), chunk)


@pytest.mark.parametrize("codec", [oracle.RAW_BF16, oracle.INT8_G64])
def test_placement_invariance(codec):
    """The same logical tokens stored from two different physical placements give identical chunks."""
    rng = np.random.default_rng(9)
    shape = synth.TOY.with_(n_blocks=32, block_size=4)
    k, v = synth.make_pool(shape, seed=1)
    pool = synth.pool_to_numpy(k, v)
    t1 = rng.permutation(32)[:6].astype(np.int32)
    t2 = np.setdiff1d(np.arange(32), t1)[:6].astype(np.int32)
    rng.shuffle(t2)
    pool2 = pool.copy()
    pool2[:, :, t2] = pool[:, :, t1]
    for off, T in ((0, 24), (1, 20), (5, 7)):
        assert np.array_equal(oracle.store(pool, t1, off, T, codec), oracle.store(pool2, t2, off, T, codec))
    # a shifted window of the same tokens: offset changes, bytes do not
    t3 = np.concatenate(([31 if 31 not in t1 else 30], t1)).astype(np.int32)
    assert np.array_equal(oracle.store(pool, t1, 2, 9, codec), oracle.store(pool, t3, 2 + 4, 9, codec))


@pytest.mark.parametrize("codec", [oracle.RAW_BF16, oracle.INT8_G64])
def test_retrieve_writes_only_addressed_slots(codec):
    rng = np.random.default_rng(13)
    shape = synth.TOY.with_(n_blocks=16, block_size=4)
    k, v = synth.make_pool(shape, seed=2)
    pool = synth.pool_to_numpy(k, v)
    table = rng.permutation(16)[:4].astype(np.int32)
    off, T = 3, 9
    chunk = oracle.store(pool, table, off, T, codec)
    SENT = np.uint16(0x7fa5)
    out = np.full_like(pool, SENT)
    dst = rng.permutation(16)[:4].astype(np.int32)
    oracle.retrieve(out, dst, off, T, codec, chunk)
    written = np.zeros(pool.shape[2:4], dtype=bool)
    p = off + np.arange(T)
    written[dst[p // 4], p % 4] = True
    assert np.all(out[:, :, ~written] == SENT)
    assert not np.any(out[:, :, written] == SENT)


def test_bad_arguments_are_refused():
    rng = np.random.default_rng(1)
    pool = rand_pool(rng, 1, 1, 64, 4, 4)
    table = np.array([0, 1], dtype=np.int32)
    with pytest.raises(ValueError):
        oracle.store(pool, table, 0, 9, oracle.RAW_BF16)            # beyond the table
    with pytest.raises(ValueError):
        oracle.store(pool, np.array([0, 4], dtype=np.int32), 0, 8, oracle.RAW_BF16)   # block id outside pool
    with pytest.raises(ValueError):
        oracle.store(pool, table, -1, 2, oracle.RAW_BF16)
    assert oracle.chunk_bytes(1, 1, 32, 4, oracle.INT8_G64) == 0    # head_dim not a multiple of 64
    assert oracle.chunk_bytes(2, 2, 64, 256, oracle.RAW_BF16) == 256 * 1024
    assert oracle.chunk_bytes(2, 2, 64, 256, oracle.INT8_G64) == 256 * 544
    assert oracle.chunk_bytes(32, 8, 128, 1, oracle.INT8_G64) == 68 * 1024
    assert oracle.chunk_bytes(80, 8, 128, 1, oracle.RAW_BF16) == 320 * 1024
