"""GPU parity for token lists: keep-list store / retrieve and select-list compose against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np, check_rotated_keys

pytestmark = pytest.mark.gpu
RAW, INT8, INT4 = oracle.RAW_BF16, oracle.INT8_G64, oracle.INT4_G64


def dev_list(dev, a):
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).to(dev.dev)
    dev._keep.append(t)
    return t


@pytest.mark.parametrize("codec", [RAW, INT8, INT4])
@pytest.mark.parametrize("shape", [synth.TOY.with_(n_blocks=64, block_size=16),
                                   synth.TOY.with_(n_layers=3, n_kv_heads=8, head_dim=128, block_size=8, n_blocks=96)],
                         ids=["toy", "H8D128"])
def test_keep_list_store_and_retrieve(shape, codec):
    dev = Device(shape, seed=23)
    try:
        K = dev.K
        bs = shape.block_size
        rng = np.random.default_rng(codec + 7)
        host = dev.pool_np()
        perm = rng.permutation(shape.n_blocks).astype(np.int32)
        span = 6 * bs
        cases = [(perm[0:6], 0, np.arange(span)),                                         # everything
                 (perm[6:12], 0, np.sort(rng.choice(span, span // 2, replace=False))),    # random half
                 (perm[12:18], 3, np.array([0, 1, 2, span - 4])),                         # few, offset start
                 (perm[18:24], 1, np.array([5]))]                                         # a single token
        ops, keeps, bufs = [], [], []
        for tab, off, keep in cases:
            b = dev.chunk_buf(len(keep), codec)
            bufs.append(b)
            ops.append(dev.op(dev.table(tab), off, b, len(keep), codec))
            keeps.append(dev_list(dev, keep).data_ptr())
        pinned = dev.chunk_buf(len(cases[1][2]), codec, pinned=True)                      # one chunk to host memory
        ops.append(dev.op(dev.table(cases[1][0]), cases[1][1], pinned, len(cases[1][2]), codec))
        keeps.append(keeps[1])
        K.kdn_store_sparse(dev.ctx, dev.pool_id, ops, keeps, dev.stream.cuda_stream)
        assert dev.sync() == 0
        wants = [oracle.store(host, tab, off, len(keep), codec, keep=keep) for tab, off, keep in cases]
        for b, w in zip(bufs, wants):
            assert np.array_equal(to_np(b), w)
        assert np.array_equal(to_np(pinned), wants[1])
        assert np.array_equal(dev.pool_np(), host)
        # retrieve into other blocks, shifted by one position; only the listed slots may change
        ref = host.copy()
        rops = []
        for i, ((tab, off, keep), b, w) in enumerate(zip(cases, bufs, wants)):
            dtab = perm[30 + 7 * i:30 + 7 * i + 7]
            src_buf = pinned if i == 1 else b
            rops.append(dev.op(dev.table(dtab), off + 1, src_buf, len(keep), codec))
            oracle.retrieve(ref, dtab, off + 1, len(keep), codec, w, keep=keep)
        K.kdn_retrieve_sparse(dev.ctx, dev.pool_id, rops, keeps[:4], dev.stream.cuda_stream)
        assert dev.sync() == 0
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [RAW, INT8, INT4])
def test_select_list_compose(codec):
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=128, block_size=8, n_blocks=80, rope_theta=500000.0)
    dev = Device(shape, seed=29)
    try:
        K = dev.K
        rng = np.random.default_rng(codec + 40)
        host = dev.pool_np()
        perm = rng.permutation(80).astype(np.int32)
        Ts, base, dst = [40, 24, 16], [0, 1000, 7], [2, 44, 70]
        srcs = [perm[0:5], perm[5:8], perm[8:10]]
        bufs, ochunks = [], []
        sops = []
        for tab, T in zip(srcs, Ts):
            b = dev.chunk_buf(T, codec)
            bufs.append(b)
            sops.append(dev.op(dev.table(tab), 0, b, T, codec))
            ochunks.append(oracle.store(host, tab, 0, T, codec))
        dev.store(sops)
        assert dev.sync() == 0
        req_tab = perm[20:31]                                                              # 88 positions
        sels = [np.sort(rng.choice(40, 13, replace=False)), None, np.array([0, 15])]
        dsel = [(dev_list(dev, s).data_ptr(), len(s)) if s is not None else None for s in sels]
        parts = [dev.chunk(b, T, codec, bp) for b, T, bp in zip(bufs, Ts, base)]
        dtab = dev.table(req_tab)
        K.kdn_compose_select(dev.ctx, dev.pool_id, [K.ComposeReq(dtab.data_ptr(), len(req_tab), parts, dst, shape.rope_theta)],
                             [dsel], dev.stream.cuda_stream)
        assert dev.sync() == 0
        ref = host.copy()
        kref, kmag = oracle.compose(ref, req_tab, [(oc, T, codec, bp, dp) for oc, T, bp, dp in zip(ochunks, Ts, base, dst)],
                                    shape.rope_theta, want_ref=True, select=sels)
        got = dev.pool_np()
        rot = np.zeros(got.shape, dtype=bool)
        written = ~np.isnan(kref[0, :, 0, 0])
        pos = np.flatnonzero(written)
        rot[:, 0, req_tab[pos // 8], pos % 8] = True
        assert np.array_equal(got[~rot], ref[~rot])                                       # values, unlisted slots, other blocks
        gk = got[:, 0, req_tab[pos // 8], pos % 8]
        rk = ref[:, 0, req_tab[pos // 8], pos % 8]
        check_rotated_keys(gk, kref[:, pos], kmag[:, pos], rk)
        assert len(pos) == 13 + 24 + 2
    finally:
        dev.close()


def test_list_entries_outside_the_table_are_reported_not_faulted():
    shape = synth.TOY.with_(n_blocks=16, block_size=16)
    dev = Device(shape, seed=2)
    try:
        K = dev.K
        host = dev.pool_np()
        tab = np.array([3, 9], dtype=np.int32)                            # 32 positions
        keep = np.array([0, 5, 40, 31], dtype=np.int32)                   # 40 is outside
        buf = dev.chunk_buf(4, RAW, fill=0xA5)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(tab), 0, buf, 4, RAW)], [dev_list(dev, keep).data_ptr()],
                           dev.stream.cuda_stream)
        assert dev.sync() == K.KDN_E_RANGE
        got = to_np(buf).view(np.uint16).reshape(2, 2, 4, 2, 64)
        # the entry outside the table is never stored; the rows that share its tile (neighbours in the list) are either
        # stored correctly or left alone, nothing else
        assert np.all(got[:, :, 2] == 0xA5A5)
        for j, want in ((0, host[:, :, 3, 0]), (1, host[:, :, 3, 5]), (3, host[:, :, 9, 15])):
            assert np.array_equal(got[:, :, j], want) or np.all(got[:, :, j] == 0xA5A5)
        with pytest.raises(K.KdnError):                                   # more listed tokens than positions
            K.kdn_store_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(tab), 30, buf, 4, RAW)], [dev_list(dev, keep).data_ptr()],
                               dev.stream.cuda_stream)
        assert dev.sync() == 0
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [INT8, INT4])
def test_coded_keep_lists_take_several_rows_per_tile(codec):
    """Coded keep-list launches put several listed rows in a tile (two of 1024 elements, up to four shorter ones) and move rows that are neighbours in the pool with
    one copy: lists with runs of every length, over a contiguous and over a scattered block table (runs that cross a
    block boundary stay one copy only where the blocks are neighbours too), list lengths that leave a ragged last tile,
    and a mixed batch with a raw op."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=8, head_dim=128, block_size=8, n_blocks=128)
    dev = Device(shape, seed=61)
    try:
        K = dev.K
        bs = shape.block_size
        rng = np.random.default_rng(codec)
        host = dev.pool_np()
        span = 10 * bs
        contiguous = (np.arange(10) + 50).astype(np.int32)
        scattered = rng.permutation(50)[:10].astype(np.int32)
        runs = np.array([0, 1, 2, 3, 5, 6, 8, 10, 11, 12, 13, 14, 15, 16, 17, 20, 23, 24, 30, 31, 32, 33, 34, 41, 47, 48, 49, 50, 51, 52, 79])
        lists = [runs, np.arange(span), np.sort(rng.choice(span, 37, replace=False)), np.array([7, 8]), np.arange(3) * 9]
        ops, keeps, wants, bufs = [], [], [], []
        for tab in (contiguous, scattered):
            for keep in lists:
                c = codec
                b = dev.chunk_buf(len(keep), c)
                ops.append(dev.op(dev.table(tab), 0, b, len(keep), c))
                keeps.append(dev_list(dev, keep).data_ptr())
                wants.append(oracle.store(host, tab, 0, len(keep), c, keep=keep))
                bufs.append(b)
        raw_keep = np.array([1, 2, 3, 40])
        rb = dev.chunk_buf(4, RAW)
        ops.append(dev.op(dev.table(scattered), 0, rb, 4, RAW))
        keeps.append(dev_list(dev, raw_keep).data_ptr())
        wants.append(oracle.store(host, scattered, 0, 4, RAW, keep=raw_keep))
        bufs.append(rb)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, ops, keeps, dev.stream.cuda_stream)
        assert dev.sync() == 0
        assert K.kdn_last_launch(dev.ctx)["tile_bytes"] == 2 * 1024 * 2            # two rows of 1024 elements
        for b, w in zip(bufs, wants):
            assert np.array_equal(to_np(b), w)
        # retrieve each chunk into its own destination blocks: neighbouring blocks for the first, scattered for the rest
        ref = host.copy()
        all_keeps = lists + lists + [raw_keep]
        free = rng.permutation(np.setdiff1d(np.arange(128), np.arange(60, 70)))
        for i, (b, w, keep) in enumerate(zip(bufs, wants, all_keeps)):
            dtab = (np.arange(10) + 60).astype(np.int32) if i == 0 else free[(i % 11) * 10:(i % 11) * 10 + 10].astype(np.int32)
            c = RAW if i == len(bufs) - 1 else codec
            K.kdn_retrieve_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(dtab), 0, b, len(keep), c)], [keeps[i]], dev.stream.cuda_stream)
            oracle.retrieve(ref, dtab, 0, len(keep), c, w, keep=keep)
        assert dev.sync() == 0
        assert np.array_equal(dev.pool_np(), ref)
        # a listed position outside the table: reported; the tile that holds it is skipped, the other tiles are written
        keep_bad = np.array([0, 1, 2, 3, 4, 5, 6, 200], dtype=np.int32)
        b = dev.chunk_buf(8, codec, fill=0xA5)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(contiguous), 0, b, 8, codec)], [dev_list(dev, keep_bad).data_ptr()],
                           dev.stream.cuda_stream)
        assert dev.sync() == K.KDN_E_RANGE
        L, R = shape.n_layers, shape.n_kv_heads * shape.head_dim
        rows_per_tile = K.kdn_last_launch(dev.ctx)["tile_bytes"] // 2 // R
        n_ok = 7 // rows_per_tile * rows_per_tile                                   # the tiles before the one with the bad entry
        good = oracle.store(ref, contiguous, 0, n_ok, codec, keep=keep_bad[:n_ok])      # ref: the pool as the retrieves left it
        got = to_np(b)
        per_tok = R // 2 if codec == INT4 else R
        codes = got[:L * 2 * 8 * per_tok].reshape(L * 2, 8, per_tok)
        gcodes = good[:L * 2 * n_ok * per_tok].reshape(L * 2, n_ok, per_tok)
        assert np.array_equal(codes[:, :n_ok], gcodes) and np.all(codes[:, n_ok:] == 0xA5)
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [RAW, INT8, INT4])
@pytest.mark.parametrize("heads,head_dim", [(1, 64), (2, 64), (1, 128)])
def test_keep_lists_over_short_rows_take_up_to_16_rows_per_tile(codec, heads, head_dim):
    """Rows of 64 to 128 elements (one or two KV heads per GPU): a tile takes up to 16 listed rows, the row indices
    travel in shared memory, and the launch runs on the kernels built for that.  Lists with runs of every length up to
    beyond 16 (a run longer than a tile is cut at the tile), ragged last tiles, contiguous and scattered block tables."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=heads, head_dim=head_dim, block_size=8, n_blocks=128)
    dev = Device(shape, seed=71)
    try:
        K = dev.K
        rng = np.random.default_rng(7 + codec)
        host = dev.pool_np()
        span = 20 * 8
        contiguous = (np.arange(20) + 40).astype(np.int32)
        scattered = np.setdiff1d(rng.permutation(128), np.arange(60, 100))[:20].astype(np.int32)
        runs = np.concatenate([np.arange(0, 40), [42, 44, 45, 50], np.arange(60, 77), [100, 101, 159]])
        lists = [runs, np.arange(span), np.sort(rng.choice(span, 53, replace=False)), np.array([5]), np.arange(17) * 9]
        ops, keeps, wants, bufs = [], [], [], []
        for tab in (contiguous, scattered):
            for keep in lists:
                b = dev.chunk_buf(len(keep), codec)
                ops.append(dev.op(dev.table(tab), 0, b, len(keep), codec))
                keeps.append(dev_list(dev, keep).data_ptr())
                wants.append(oracle.store(host, tab, 0, len(keep), codec, keep=keep))
                bufs.append(b)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, ops, keeps, dev.stream.cuda_stream)
        assert dev.sync() == 0
        info = K.kdn_last_launch(dev.ctx)
        R = heads * head_dim
        assert info["tile_bytes"] == min(16, 2048 // R) * R * 2 and "rows" in info["kernel"]
        for b, w in zip(bufs, wants):
            assert np.array_equal(to_np(b), w)
        ref = host.copy()
        free = rng.permutation(np.arange(60, 100))
        for i, (b, w, keep) in enumerate(zip(bufs, wants, lists + lists)):
            dtab = (np.arange(20) + 60).astype(np.int32) if i % 2 == 0 else free[:20].astype(np.int32)
            K.kdn_retrieve_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(dtab), 0, b, len(keep), codec)], [keeps[i]], dev.stream.cuda_stream)
            assert "rows" in K.kdn_last_launch(dev.ctx)["kernel"]
            oracle.retrieve(ref, dtab, 0, len(keep), codec, w, keep=keep)
            assert dev.sync() == 0
            assert np.array_equal(dev.pool_np(), ref), i
        # an entry outside the table: reported, and nothing but listed rows is ever written
        keep_bad = np.concatenate([np.arange(30), [500]]).astype(np.int32)
        b = dev.chunk_buf(31, codec, fill=0xA5)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(contiguous), 0, b, 31, codec)], [dev_list(dev, keep_bad).data_ptr()],
                           dev.stream.cuda_stream)
        assert dev.sync() == K.KDN_E_RANGE
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()
