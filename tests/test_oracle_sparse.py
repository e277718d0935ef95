"""Pins for the oracle's token lists: keep-lists in store / retrieve, select-lists in compose (CPU only)."""
import numpy as np
import pytest

import oracle
from paper_2409_13761_b200 import synth

CODECS = [oracle.RAW_BF16, oracle.INT8_G64, oracle.INT4_G64]


def make(seed, bs=4, nb=24):
    shape = synth.TOY.with_(block_size=bs, n_blocks=nb)
    k, v = synth.make_pool(shape, seed=seed)
    return shape, synth.pool_to_numpy(k, v)


def chunk_rows(chunk, L, T, H, D, codec):
    """Per-token view of a chunk: (codes/raw rows [L][2][T][row bytes], scale rows [L][2][T][bytes] or None)."""
    n = L * 2 * T * H * D
    if codec == oracle.RAW_BF16:
        return chunk.reshape(L, 2, T, H * D * 2), None
    nc = n // 2 if codec == oracle.INT4_G64 else n
    return chunk[:nc].reshape(L, 2, T, -1), chunk[nc:].reshape(L, 2, T, -1)


@pytest.mark.parametrize("codec", CODECS)
def test_keep_list_store_is_the_dense_chunk_restricted_to_the_kept_tokens(codec):
    shape, pool = make(3)
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    rng = np.random.default_rng(codec)
    table = rng.permutation(24)[:8].astype(np.int32)
    off, span = 3, 27
    dense = oracle.store(pool, table, off, span, codec)
    drows, dscales = chunk_rows(dense, L, span, H, D, codec)
    for keep in ([0], [26], [1, 2, 3, 9, 10, 26], list(range(span)), sorted(rng.choice(span, 11, replace=False).tolist())):
        keep = np.array(keep, dtype=np.int32)
        got = oracle.store(pool, table, off, len(keep), codec, keep=keep)
        rows, scales = chunk_rows(got, L, len(keep), H, D, codec)
        assert np.array_equal(rows, drows[:, :, keep])
        if scales is not None:
            assert np.array_equal(scales, dscales[:, :, keep])
    assert np.array_equal(oracle.store(pool, table, off, span, codec, keep=np.arange(span)), dense)
    # raw: directly against advanced indexing of the pool
    if codec == oracle.RAW_BF16:
        keep = np.array([0, 5, 6, 20], dtype=np.int32)
        p = off + keep
        want = pool[:, :, table[p // 4], p % 4]
        assert np.array_equal(oracle.store(pool, table, off, 4, codec, keep=keep).view(np.uint16).reshape(want.shape), want)


@pytest.mark.parametrize("codec", CODECS)
def test_keep_list_retrieve_writes_exactly_the_kept_positions(codec):
    shape, pool = make(4)
    rng = np.random.default_rng(10 + codec)
    src = rng.permutation(24)[:6].astype(np.int32)
    dst = np.setdiff1d(np.arange(24), src)[:6].astype(np.int32)
    off, span = 1, 20
    keep = np.array(sorted(rng.choice(span, 9, replace=False).tolist()), dtype=np.int32)
    chunk = oracle.store(pool, src, off, len(keep), codec, keep=keep)
    SENT = np.uint16(0x7fa5)
    out = np.full_like(pool, SENT)
    oracle.retrieve(out, dst, off + 2, len(keep), codec, chunk, keep=keep)
    # the same values a dense retrieve of the dense chunk puts there
    ref = np.full_like(pool, SENT)
    oracle.retrieve(ref, dst, off + 2, span, codec, oracle.store(pool, src, off, span, codec))
    p = off + 2 + keep
    assert np.array_equal(out[:, :, dst[p // 4], p % 4], ref[:, :, dst[p // 4], p % 4])
    mask = np.ones(out.shape[2:4], dtype=bool)
    mask[dst[p // 4], p % 4] = False
    assert np.all(out[:, :, mask] == SENT) and not np.any(out[:, :, ~mask] == SENT)


@pytest.mark.parametrize("codec", CODECS)
def test_select_list_compose_is_dense_compose_on_the_selected_positions(codec):
    shape, pool = make(5, bs=4, nb=40)
    rng = np.random.default_rng(20 + codec)
    perm = rng.permutation(40).astype(np.int32)
    T1, T2 = 13, 9
    c1 = oracle.store(pool, perm[:4], 1, T1, codec)
    c2 = oracle.store(pool, perm[4:7], 0, T2, codec)
    table = perm[10:18]
    parts = [(c1, T1, codec, 0, 2), (c2, T2, codec, 50, 17)]          # deltas 2 and -33
    sel1 = np.array([0, 3, 4, 12], dtype=np.int32)
    before = pool.copy()
    dense = pool.copy()
    kd, md = oracle.compose(dense, table, parts, 10000.0, want_ref=True)
    got = pool.copy()
    ks, ms = oracle.compose(got, table, parts, 10000.0, want_ref=True, select=[sel1, None])
    pos = np.arange(len(table) * 4)
    chosen = np.zeros(len(pos), dtype=bool)
    chosen[2 + sel1] = True
    chosen[17:17 + T2] = True
    blk, slot = table[pos // 4], pos % 4
    assert np.array_equal(got[:, :, blk[chosen], slot[chosen]], dense[:, :, blk[chosen], slot[chosen]])
    assert np.array_equal(got[:, :, blk[~chosen], slot[~chosen]], before[:, :, blk[~chosen], slot[~chosen]])
    assert np.array_equal(ks[:, chosen], kd[:, chosen]) and np.all(np.isnan(ks[:, ~chosen]))
    assert np.array_equal(ms[:, chosen], md[:, chosen])
    others = np.setdiff1d(np.arange(40), table)
    assert np.array_equal(got[:, :, others], before[:, :, others])
    # an empty selection delivers nothing
    nothing = pool.copy()
    oracle.compose(nothing, table, parts[:1], 10000.0, select=[np.zeros(0, dtype=np.int32)])
    assert np.array_equal(nothing, before)


def test_bad_lists_are_refused():
    shape, pool = make(6)
    table = np.arange(4, dtype=np.int32)
    for keep in ([2, 2], [3, 1], [-1, 2], [0, 16]):                       # repeats, decreasing, negative, past the table
        with pytest.raises(ValueError):
            oracle.store(pool, table, 0, 2, oracle.RAW_BF16, keep=np.array(keep, dtype=np.int32))
    with pytest.raises(ValueError):
        oracle.store(pool, table, 0, 3, oracle.RAW_BF16, keep=np.array([0, 1], dtype=np.int32))   # count mismatch
    c = oracle.store(pool, table, 0, 5, oracle.RAW_BF16)
    with pytest.raises(ValueError):                                        # selected token beyond the part
        oracle.compose(pool.copy(), table, [(c, 5, oracle.RAW_BF16, 0, 0)], 1e4, select=[np.array([1, 5], dtype=np.int32)])
