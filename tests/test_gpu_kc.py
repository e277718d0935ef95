"""GPU parity for the per-channel key codecs (keys grouped along tokens): the CUDA library against the CPU oracle."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np, check_rotated_keys, kdn

pytestmark = pytest.mark.gpu
RAW, INT8 = oracle.RAW_BF16, oracle.INT8_G64
KC = [oracle.INT8_KC64, oracle.INT4_KC64]

SHAPES = [
    synth.TOY.with_(n_layers=3, n_blocks=96, block_size=16),                                   # 128-element rows
    synth.TOY.with_(n_layers=2, n_kv_heads=8, head_dim=128, block_size=16, n_blocks=96),       # 8B-sized rows (1024)
    synth.TOY.with_(n_layers=2, n_kv_heads=3, head_dim=192, block_size=32, n_blocks=48),
    synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=4, n_blocks=300),
]


def gather(pool_np, table, pos):
    bs = pool_np.shape[3]
    pos = np.asarray(pos)
    return pool_np[:, :, table[pos // bs], pos % bs]


@pytest.mark.parametrize("codec", KC, ids=["int8kc", "int4kc"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "H%dD%dbs%d" % (s.n_kv_heads, s.head_dim, s.block_size))
def test_store_retrieve_compose_against_the_oracle(shape, codec):
    """One batched store mixing the codec with raw and int8 chunks, chunk lengths that end inside a 64-token group and
    inside a block; then retrieve into other blocks; then compose with a position shift."""
    dev = Device(shape, seed=41)
    try:
        K, bs = dev.K, shape.block_size
        host = dev.pool_np()
        rng = np.random.default_rng(6)
        perm = rng.permutation(shape.n_blocks).astype(np.int32)
        span = -(-200 // bs)                                            # blocks that hold 200 tokens
        # (offset in blocks, tokens, codec): a short group, several groups with a ragged tail, exactly one group
        cases = [(0, 200, codec), (1, 7, codec), (0, 64, codec), (2, 130, RAW), (0, 100, INT8), (1, 65, codec)]
        tabs, bufs, ops, want = [], [], [], []
        nxt = 0
        for ob, T, cd in cases:
            tab = perm[nxt:nxt + span + 2]
            nxt += span + 2
            if nxt + span + 2 > shape.n_blocks:
                nxt = 0                                                  # source blocks may repeat between ops
            b = dev.chunk_buf(T, cd)
            tabs.append(tab); bufs.append(b)
            ops.append(dev.op(dev.table(tab), ob * bs, b, T, cd))
            want.append(oracle.store(host, tab, ob * bs, T, cd))
        dev.store(ops)
        assert dev.sync() == 0
        for i, (b, w) in enumerate(zip(bufs, want)):
            assert np.array_equal(to_np(b), w), "store: chunk %d (%s)" % (i, cases[i],)
        assert np.array_equal(dev.pool_np(), host)                      # store writes no pool block

        # retrieve the first two chunks into blocks of their own
        dst0, dst1 = perm[-(span + 1):], perm[-(2 * span + 3):-(span + 2)]
        rops = [dev.op(dev.table(dst0), bs, bufs[0], 200, codec), dev.op(dev.table(dst1), 0, bufs[1], 7, codec)]
        ref = host.copy()
        oracle.retrieve(ref, dst0, bs, 200, codec, want[0])
        oracle.retrieve(ref, dst1, 0, 7, codec, want[1])
        dev.retrieve(rops)
        assert dev.sync() == 0
        assert np.array_equal(dev.pool_np(), ref)

        # compose chunk 0 (base 0) at position 2*bs and chunk 5 (base 1000) right behind it, rounded up to a block
        host2 = dev.pool_np()
        req = perm[:2 * span + 6]
        d0 = 2 * bs
        d5 = d0 + -(-200 // bs) * bs
        d2 = d5 + -(-65 // bs) * bs
        parts = [dev.chunk(bufs[0], 200, codec, 0), dev.chunk(bufs[5], 65, codec, 1000), dev.chunk(bufs[2], 64, codec, d2)]
        dstp = [d0, d5, d2]                                              # the third part keeps its position: no rotation
        dev.compose([K.ComposeReq(dev.table(req).data_ptr(), len(req), parts, dstp, 500000.0)])
        assert dev.sync() == 0
        ref2 = host2.copy()
        kref, kmag = oracle.compose(ref2, req, [(want[0], 200, codec, 0, d0), (want[5], 65, codec, 1000, d5), (want[2], 64, codec, d2, d2)],
                                    500000.0, want_ref=True)
        got = dev.pool_np()
        rot = np.zeros(got.shape, dtype=bool)
        for T, dp in ((200, d0), (65, d5)):
            p = dp + np.arange(T)
            rot[:, 0, req[p // bs], p % bs] = True
        assert np.array_equal(got[~rot], ref2[~rot])
        for T, dp in ((200, d0), (65, d5)):
            p = dp + np.arange(T)
            check_rotated_keys(gather(got, req, p)[:, 0], kref[:, dp:dp + T], kmag[:, dp:dp + T], gather(ref2, req, p)[:, 0])
    finally:
        dev.close()


@pytest.mark.parametrize("codec", KC, ids=["int8kc", "int4kc"])
def test_many_ops_host_memory_files_and_layer_steps(tmp_path, codec):
    """More ops than travel as kernel parameters; chunks in page-locked host memory and in a file through small staging
    slabs; layer-wise retrieve."""
    shape = synth.TOY.with_(n_layers=4, n_blocks=128, block_size=16)
    dev = Device(shape, seed=42)
    try:
        K, bs = dev.K, shape.block_size
        K.kdn_set_staging_bytes(dev.ctx, 64 * 1024)
        host = dev.pool_np()
        perm = np.random.default_rng(2).permutation(shape.n_blocks).astype(np.int32)
        # 40 device-resident stores in one call
        ops, bufs, want = [], [], []
        for i in range(40):
            tab = perm[(3 * i) % 120:(3 * i) % 120 + 7]
            T = 1 + (37 * i) % 90
            b = dev.chunk_buf(T, codec)
            bufs.append(b)
            ops.append(dev.op(dev.table(tab), bs * (i % 2), b, T, codec))
            want.append(oracle.store(host, tab, bs * (i % 2), T, codec))
        dev.store(ops)
        assert dev.sync() == 0
        for b, w in zip(bufs, want):
            assert np.array_equal(to_np(b), w)
        # a chunk stored to page-locked host memory and to a file, then brought back from both
        tab, T = perm[:12], 150
        w = oracle.store(host, tab, 0, T, codec)
        hb = dev.chunk_buf(T, codec, pinned=True)
        dev.store([dev.op(dev.table(tab), 0, hb, T, codec)])
        fd = os.open(tmp_path / "kc.bin", os.O_RDWR | os.O_CREAT, 0o600)
        try:
            fop = K.XferOp(dev.table(tab).data_ptr(), len(tab), 0, K.Chunk(0, len(w), T, codec))
            K.kdn_store_file(dev.ctx, dev.pool_id, [fop], [fd], [5], dev.stream.cuda_stream)
            assert dev.sync() == 0
            assert np.array_equal(hb.numpy(), w)
            assert np.array_equal(np.fromfile(tmp_path / "kc.bin", dtype=np.uint8)[5:], w)
            d1, d2, d3 = perm[20:32], perm[40:52], perm[60:72]
            ref = host.copy()
            for d in (d1, d2, d3):
                oracle.retrieve(ref, d, bs, T, codec, w)
            dev.retrieve([dev.op(dev.table(d1), bs, hb, T, codec)])
            K.kdn_retrieve_file(dev.ctx, dev.pool_id, [K.XferOp(dev.table(d2).data_ptr(), len(d2), bs, K.Chunk(0, len(w), T, codec))],
                                [fd], [5], dev.stream.cuda_stream)
            db = dev.chunk_buf(T, codec)
            db.copy_(torch.from_numpy(w))
            K.kdn_retrieve_layerwise(dev.ctx, dev.pool_id, [dev.op(dev.table(d3), bs, db, T, codec)], 3, dev.stream.cuda_stream)
            assert dev.sync() == 0
            assert np.array_equal(dev.pool_np(), ref)
        finally:
            os.close(fd)
    finally:
        dev.close()


def test_what_the_codecs_do_not_support_is_refused():
    K = kdn()
    for shape, off in ((synth.TOY.with_(n_blocks=16, block_size=16), 3), (synth.TOY.with_(n_blocks=16, block_size=3), 0),
                       (synth.TOY.with_(n_blocks=16, block_size=128), 0)):
        dev = Device(shape, seed=1)
        try:
            for codec in KC:
                b = dev.chunk_buf(5, codec)
                tab = dev.table(np.arange(4, dtype=np.int32))
                for call in (dev.store, dev.retrieve):
                    with pytest.raises(K.KdnError) as e:
                        call([dev.op(tab, off, b, 5, codec)])
                    assert e.value.status == K.KDN_E_UNSUPPORTED
        finally:
            dev.close()


@pytest.mark.parametrize("shape", SHAPES[:3], ids=["H%dD%dbs%d" % (s.n_kv_heads, s.head_dim, s.block_size) for s in SHAPES[:3]])
@pytest.mark.parametrize("codec", KC, ids=["int8kc", "int4kc"])
def test_select_list_compose_against_the_oracle(shape, codec):
    """kdn_compose_select with per-channel key chunks: two parts, one with a select-list and a position shift (keys
    re-rotated), one delivered whole; listed positions as the oracle has them, every other position untouched."""
    bs = shape.block_size
    rng = np.random.default_rng(37 + codec)
    perm = rng.permutation(shape.n_blocks).astype(np.int32)
    T = 130
    nb = -(-T // bs)
    dev = Device(shape, seed=79)
    try:
        K = dev.K
        pool = dev.pool_np()
        srcs = [perm[:nb], perm[nb:2 * nb]]
        bufs = [dev.chunk_buf(T, codec) for _ in srcs]
        dev.store([dev.op(dev.table(t), 0, b, T, codec) for t, b in zip(srcs, bufs)])
        assert dev.sync() == 0
        wants = [oracle.store(pool, t, 0, T, codec) for t in srcs]
        d0, d1 = 0, -(-T // 64) * 64                                       # block-aligned destinations (64 is a multiple of block_size)
        rt = perm[2 * nb:2 * nb + -(-(d1 + T) // bs)]
        sel = np.sort(rng.choice(T, 41, replace=False)).astype(np.int32)
        d_sel = dev.table(sel)
        before = dev.pool_np()
        K.kdn_compose_select(dev.ctx, dev.pool_id,
                             [K.ComposeReq(dev.table(rt).data_ptr(), len(rt), [dev.chunk(bufs[0], T, codec, 9), dev.chunk(bufs[1], T, codec, d1)],
                                           [d0, d1], shape.rope_theta)],
                             [[(d_sel.data_ptr(), len(sel)), None]], dev.stream.cuda_stream)
        assert dev.sync() == 0
        ref = before.copy()
        kref, kmag = oracle.compose(ref, rt, [(wants[0], T, codec, 9, d0), (wants[1], T, codec, d1, d1)], shape.rope_theta,
                                    want_ref=True, select=[sel, None])
        got = dev.pool_np()
        p = d0 + sel
        rot = np.zeros(got.shape, dtype=bool)
        rot[:, 0, rt[p // bs], p % bs] = True
        assert np.array_equal(got[~rot], ref[~rot])
        check_rotated_keys(got[:, 0, rt[p // bs], p % bs], kref[:, p], kmag[:, p], ref[:, 0, rt[p // bs], p % bs],
                           min_equal=0.995 if got[:, 0, rt[p // bs], p % bs].size >= 8192 else 0.95)
    finally:
        dev.close()


@pytest.mark.parametrize("shape", SHAPES, ids=["H%dD%dbs%d" % (s.n_kv_heads, s.head_dim, s.block_size) for s in SHAPES])
@pytest.mark.parametrize("codec", KC, ids=["int8kc", "int4kc"])
def test_keep_list_chunks_against_the_oracle(shape, codec):
    """Keep-lists with the per-channel key codecs: a key group is 64 consecutive listed tokens, wherever they sit in the
    request (no alignment rule).  Store bytes, retrieve into other blocks (device and page-locked host chunk), a dense
    compose of a sparsely stored chunk, and a list entry outside the table."""
    bs = shape.block_size
    rng = np.random.default_rng(31 + codec)
    perm = rng.permutation(shape.n_blocks).astype(np.int32)
    span, off = 200, 5
    nb = -(-(off + span) // bs)
    src, dst = perm[:nb], perm[nb:2 * nb]
    dev = Device(shape, seed=77)
    try:
        K = dev.K
        pool = dev.pool_np()
        lists = [np.sort(rng.choice(span, 100, replace=False)), np.arange(span), np.array([7]), np.arange(0, span, 3), np.arange(64) + 5]
        ops, keeps, wants, bufs = [], [], [], []
        for keep in lists:
            keep = keep.astype(np.int32)
            b = dev.chunk_buf(len(keep), codec)
            ops.append(dev.op(dev.table(src), off, b, len(keep), codec))
            keeps.append(dev.table(keep).data_ptr())
            wants.append(oracle.store(pool, src, off, len(keep), codec, keep=keep))
            bufs.append(b)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, ops, keeps, dev.stream.cuda_stream)
        assert dev.sync() == 0
        for b, w, keep in zip(bufs, wants, lists):
            assert np.array_equal(to_np(b), w), len(keep)
        assert np.array_equal(dev.pool_np(), pool)
        ref = pool.copy()
        for i, (b, w, keep) in enumerate(zip(bufs, wants, lists)):
            src_buf = b
            if i % 2 == 1:
                src_buf = dev.chunk_buf(len(keep), codec, pinned=True)
                src_buf.copy_(b.cpu())
            K.kdn_retrieve_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(dst), off, src_buf, len(keep), codec)], [keeps[i]], dev.stream.cuda_stream)
            assert dev.sync() == 0
            oracle.retrieve(ref, dst, off, len(keep), codec, w, keep=keep.astype(np.int32))
            assert np.array_equal(dev.pool_np(), ref), i
        # a sparsely stored chunk is an ordinary chunk of its own tokens: a dense retrieve at a block start places them side by side
        if 64 % bs == 0:
            T = len(lists[0])
            dt = perm[2 * nb:2 * nb + -(-T // bs)]
            dev.retrieve([dev.op(dev.table(dt), 0, bufs[0], T, codec)])
            assert dev.sync() == 0
            oracle.retrieve(ref, dt, 0, T, codec, wants[0])
            assert np.array_equal(dev.pool_np(), ref)
        bad = np.array([0, 1, 2, nb * bs], dtype=np.int32)
        b = dev.chunk_buf(4, codec)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(src), 0, b, 4, codec)], [dev.table(bad).data_ptr()], dev.stream.cuda_stream)
        assert dev.sync() == K.KDN_E_RANGE
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


@pytest.mark.parametrize("codec", KC, ids=["int8kc", "int4kc"])
def test_a_wait_that_runs_out_in_the_key_plane_store(codec):
    """The key-plane kernel's wait for its tile is bounded too: KDN_E_TIMEOUT, no write outside the chunk, the pool
    untouched, and the context bit-exact again once the default bound is back."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=4, head_dim=64, block_size=16, n_blocks=96)
    dev = Device(shape, seed=9)
    try:
        K = dev.K
        host = dev.pool_np()
        tab = np.random.default_rng(6).permutation(96)[:20].astype(np.int32)
        T = 300
        guard = 4096
        n = K.kdn_chunk_bytes(dev.desc, T, codec)
        arena = torch.full((n + 2 * guard,), 0x5C, dtype=torch.uint8, device=dev.dev)
        buf = arena[guard:guard + n]
        K.kdn_set_wait_limit_ns(dev.ctx, 40)
        dev.store([dev.op(dev.table(tab), 0, buf, T, codec)])
        assert dev.sync() in (0, K.KDN_E_TIMEOUT)                         # (0: every CTA found its rows landed in time)
        assert np.array_equal(dev.pool_np(), host)
        a = to_np(arena)
        assert np.all(a[:guard] == 0x5C) and np.all(a[-guard:] == 0x5C)
        K.kdn_set_wait_limit_ns(dev.ctx, 0)
        dev.store([dev.op(dev.table(tab), 0, buf, T, codec)])
        assert dev.sync() == 0
        assert np.array_equal(to_np(buf), oracle.store(host, tab, 0, T, codec))
    finally:
        dev.close()
