"""GPU parity of the token-delta Rice codecs (codecs 5 and 6) against the CPU oracle, through the C ABI.

store: the bytes a chunk uses are bit-identical to the oracle's chunk, and nothing past them is written;
retrieve: the pool is bit-identical to the oracle's; compose: values and unrotated keys bit-identical, re-rotated
keys within the rotation tolerance.  Inputs are uncorrelated and token-correlated (so that both coding modes occur),
with zero, constant, extreme and saw-tooth channels planted (flushed scales, the shortest and the longest
sub-streams, the escape code)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np, check_rotated_keys

pytestmark = pytest.mark.gpu
RAW, INT8 = oracle.RAW_BF16, oracle.INT8_G64
TD8, TD4 = oracle.INT8_TD64, oracle.INT4_TD64

SHAPES = [
    synth.TOY,                                                                                  # rows of 128: one slice
    synth.TOY.with_(n_layers=2, n_kv_heads=8, head_dim=128, block_size=16, n_blocks=96),        # rows of 1024: four slices
    synth.TOY.with_(n_layers=1, n_kv_heads=3, head_dim=192, block_size=32, n_blocks=40),        # rows of 576: slices of 144
    synth.TOY.with_(n_layers=3, n_kv_heads=1, head_dim=64, block_size=4, n_blocks=128),         # rows of 64, tiny blocks
]
IDS = ["H%dD%dbs%d" % (s.n_kv_heads, s.head_dim, s.block_size) for s in SHAPES]


def bf16_bits(x):
    return (np.asarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)


def make_pool_np(shape, table, off, T, rho, seed):
    """A pool whose request positions off .. off+T-1 (through `table`) hold token-correlated values with planted
    special channels; the rest is the ordinary uncorrelated fill."""
    k, v = synth.make_pool(shape, "cpu", seed=seed)
    x = synth.correlated_tokens(shape, T, rho, seed + 1)
    xb = x.view(torch.int16).numpy().view(np.uint16).copy()                 # [L][2][T][H][D]
    big = bf16_bits([3.0])[0]
    xb[0, 0, :, 0, 0] = 0                                                    # an all-zero channel: scale 0
    xb[0, 1, :, 0, 1] = bf16_bits([1e-40])[0]                                # a subnormal channel: flushed
    xb[0, 0, :, 0, 2] = big                                                  # constant: delta mode, one bit a token
    xb[0, 1, :, 0, 3] = np.where(np.arange(T) % 2 == 0, big, big | 0x8000)   # +max, -max: the longest sub-streams
    xb[0, 0, :, 0, 4] = np.where(np.arange(T) % 64 == 0, big, 0)             # one spike per group
    xb[0, 0, 1::3, 0, 5] = 0x8000                                            # negative zeros among ordinary values
    synth.place_tokens(k, v, table, off, torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16))
    return synth.pool_to_numpy(k, v)


def used_bytes(K, desc, buf, T, codec):
    lay = K.kdn_td_layout(desc, T, codec)
    head = to_np(buf[:8 * (lay["segments"] + 1)]).view(np.uint64)
    return int(head[lay["segments"]]), lay


@pytest.mark.parametrize("shape", SHAPES, ids=IDS)
@pytest.mark.parametrize("codec", [TD8, TD4], ids=["int8td", "int4td"])
@pytest.mark.parametrize("rho", [0.0, 0.97])
def test_store_retrieve_compose_against_the_oracle(shape, codec, rho):
    bs = shape.block_size
    rng = np.random.default_rng(17)
    perm = rng.permutation(shape.n_blocks).astype(np.int32)
    cases = [(150, 0), (64, bs), (37, 2 * bs)]                              # ragged last group, one full group, a short one
    nb_src = max(-(-(off + T) // bs) for T, off in cases)
    src = perm[:nb_src]
    pool = make_pool_np(shape, src, 0, nb_src * bs, rho, seed=31)
    dev = Device(shape, pool_np=pool)
    try:
        K = dev.K
        for T, off in cases:
            want = oracle.store(pool, src, off, T, codec)
            buf = dev.chunk_buf(T, codec)
            dev.store([dev.op(dev.table(src), off, buf, T, codec)])
            assert dev.sync() == 0
            used, lay = used_bytes(K, dev.desc, buf, T, codec)
            assert lay["capacity"] == buf.numel() == want.size
            assert used == oracle.td_used_bytes(want, shape.n_layers, shape.n_kv_heads, shape.head_dim, T, codec)
            got = to_np(buf)
            assert np.array_equal(got[:used], want[:used])
            assert np.all(got[used:] == 0xA5)                                # nothing past the bytes in use is written
            # retrieve into other blocks
            nb = -(-(off + T) // bs)
            dst = perm[nb_src:nb_src + nb]
            before = dev.pool_np()
            dev.retrieve([dev.op(dev.table(dst), off, buf, T, codec)])
            assert dev.sync() == 0
            ref = before.copy()
            oracle.retrieve(ref, dst, off, T, codec, want)
            assert np.array_equal(dev.pool_np(), ref)
            # compose at another block-aligned position, keys re-rotated (chunks of different base positions)
            if shape.head_dim % 16 == 0 and (shape.n_kv_heads * shape.head_dim <= 512 or 256 % shape.head_dim == 0):
                rt = perm[nb_src + nb:nb_src + nb + nb + 2]
                dpos = 2 * bs
                before = dev.pool_np()
                dev.compose([K.ComposeReq(dev.table(rt).data_ptr(), len(rt), [dev.chunk(buf, T, codec, 7)], [dpos], shape.rope_theta)])
                assert dev.sync() == 0
                ref = before.copy()
                kref, kmag = oracle.compose(ref, rt, [(want, T, codec, 7, dpos)], shape.rope_theta, want_ref=True)
                got_pool = dev.pool_np()
                p = dpos + np.arange(T)
                rot = np.zeros(got_pool.shape, dtype=bool)
                rot[:, 0, rt[p // bs], p % bs] = True
                assert np.array_equal(got_pool[~rot], ref[~rot])
                check_rotated_keys(got_pool[:, 0, rt[p // bs], p % bs], kref[:, dpos:dpos + T], kmag[:, dpos:dpos + T],
                                   ref[:, 0, rt[p // bs], p % bs])
    finally:
        dev.close()


def test_mixed_batch_and_many_ops():
    """One call carrying token-delta chunks of both widths next to raw and int8 chunks, more ops than one launch holds."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=512)
    dev = Device(shape, seed=23)
    try:
        K = dev.K
        host = dev.pool_np()
        rng = np.random.default_rng(5)
        n = 45
        codecs = [(TD8, TD4, RAW, INT8)[i % 4] for i in range(n)]
        Ts = [int(rng.integers(1, 130)) for _ in range(n)]
        tabs = [rng.permutation(512)[:9].astype(np.int32) for _ in range(n)]
        bufs = [dev.chunk_buf(T, c) for T, c in zip(Ts, codecs)]
        dev.store([dev.op(dev.table(t), 0, b, T, c) for t, b, T, c in zip(tabs, bufs, Ts, codecs)])
        assert dev.sync() == 0
        wants = []
        for t, b, T, c in zip(tabs, bufs, Ts, codecs):
            want = oracle.store(host, t, 0, T, c)
            wants.append(want)
            got = to_np(b)
            if c in (TD8, TD4):
                used = oracle.td_used_bytes(want, 2, 2, 64, T, c)
                assert np.array_equal(got[:used], want[:used])
            else:
                assert np.array_equal(got, want)
        # retrieve all of them into disjoint destinations in one call
        dst = rng.permutation(512).astype(np.int32)[:n * 9].reshape(n, 9)
        dev.retrieve([dev.op(dev.table(d), 0, b, T, c) for d, b, T, c in zip(dst, bufs, Ts, codecs)])
        assert dev.sync() == 0
        ref = host.copy()
        for d, w, T, c in zip(dst, wants, Ts, codecs):
            oracle.retrieve(ref, d, 0, T, c, w)
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


def test_layerwise_retrieve_of_a_token_delta_chunk():
    shape = synth.TOY.with_(n_layers=5, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=64)
    dev = Device(shape, seed=29)
    try:
        K = dev.K
        host = dev.pool_np()
        perm = np.random.default_rng(2).permutation(64).astype(np.int32)
        T = 100
        buf = dev.chunk_buf(T, TD4)
        dev.store([dev.op(dev.table(perm[:7]), 0, buf, T, TD4)])
        assert dev.sync() == 0
        K.kdn_retrieve_layerwise(dev.ctx, dev.pool_id, [dev.op(dev.table(perm[10:17]), 0, buf, T, TD4)], 2, dev.stream.cuda_stream)
        assert dev.sync() == 0
        ref = host.copy()
        oracle.retrieve(ref, perm[10:17], 0, T, TD4, oracle.store(host, perm[:7], 0, T, TD4))
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


def test_refusals_and_damaged_chunks():
    shape = synth.TOY.with_(n_layers=1, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=64)
    dev = Device(shape, seed=3)
    try:
        K = dev.K
        tab = dev.table(np.arange(8, dtype=np.int32))
        T = 64
        buf = dev.chunk_buf(T, TD8)
        for bad in (lambda: dev.store([dev.op(tab, 3, buf, T, TD8)]),                       # first token not at a block start
                    lambda: dev.store([dev.op(tab, 0, dev.chunk_buf(T, TD8, pinned=True), T, TD8)])):  # store into host memory
            with pytest.raises(K.KdnError) as e:
                bad()
            assert e.value.status == K.KDN_E_UNSUPPORTED
        st = K.kdn_compose_static(0, dev.desc, [K.ComposeReq(tab.data_ptr(), 8, [dev.chunk(buf, T, TD8)], [0], 1e4)], dev.stream.cuda_stream)
        assert st == K.KDN_E_UNSUPPORTED
        assert K.kdn_chunk_bytes(K.pool_desc(1, 2, 80, 16, 64), T, TD8) == 0            # head_dim not a multiple of 64
        # a damaged chunk is reported, never followed: lengths that cannot be, and an offset outside the chunk
        dev.store([dev.op(tab, 0, buf, T, TD8)])
        assert dev.sync() == 0
        host = dev.pool_np()
        lay = K.kdn_td_layout(dev.desc, T, TD8)
        good = buf.clone()
        buf[lay["lens_offset"]:lay["lens_offset"] + 128] = 255
        dev.retrieve([dev.op(dev.table(np.arange(8, dtype=np.int32) + 20), 0, buf, T, TD8)])
        assert dev.sync() == K.KDN_E_RANGE
        buf.copy_(good)
        buf[:8].copy_(torch.from_numpy(np.array([lay["capacity"] + 4096], dtype=np.uint64).view(np.uint8)).to(dev.dev))
        dev.retrieve([dev.op(dev.table(np.arange(8, dtype=np.int32) + 20), 0, buf, T, TD8)])
        assert dev.sync() == K.KDN_E_RANGE
        buf.copy_(good)
        dev.retrieve([dev.op(dev.table(np.arange(8, dtype=np.int32) + 40), 0, buf, T, TD8)])
        assert dev.sync() == 0
        ref = host.copy()
        oracle.retrieve(ref, np.arange(8, dtype=np.int32) + 40, 0, T, TD8, oracle.store(host, np.arange(8, dtype=np.int32), 0, T, TD8))
        got = dev.pool_np()
        assert np.array_equal(got[:, :, 40:], ref[:, :, 40:]) and np.array_equal(got[:, :, :20], ref[:, :, :20])
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [TD8, TD4], ids=["int8td", "int4td"])
def test_retrieve_and_compose_from_page_locked_host_chunks(codec):
    """Delivery of compressed chunks (the point of coding them): token-delta chunks kept in page-locked host memory are
    retrieved and composed; only the bytes each chunk uses cross the host link, through staging slabs that hold a few
    chunks at a time, in a call that also carries device-resident chunks."""
    shape = synth.TOY.with_(n_layers=3, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=512)
    perm = np.random.default_rng(12).permutation(512).astype(np.int32)
    pool = make_pool_np(shape, perm[:40], 0, 640, 0.9, seed=77)
    dev = Device(shape, pool_np=pool)
    try:
        K = dev.K
        Ts = [200, 64, 130, 37, 256]
        srcs, off = [], 0
        for T in Ts:
            nb = -(-T // 16)
            srcs.append(perm[off:off + nb])
            off += nb
        wants = [oracle.store(pool, t, 0, T, codec) for t, T in zip(srcs, Ts)]
        dbufs = [dev.chunk_buf(T, codec) for T in Ts]
        dev.store([dev.op(dev.table(t), 0, b, T, codec) for t, b, T in zip(srcs, dbufs, Ts)])
        assert dev.sync() == 0
        hbufs = []
        for b, w, T in zip(dbufs, wants, Ts):
            used = oracle.td_used_bytes(w, 3, 2, 64, T, codec)
            h = dev.chunk_buf(T, codec, pinned=True, fill=0x5A)
            h[:used].copy_(b[:used])                                   # only the bytes in use are kept
            hbufs.append(h)
        torch.cuda.synchronize()
        K.kdn_set_staging_bytes(dev.ctx, 512 * 1024)                      # two or three of the chunks at a time
        dsts = [perm[60 + 20 * i:60 + 20 * i + 17] for i in range(len(Ts))]
        ops = [dev.op(dev.table(d), 0, (hbufs[i] if i != 2 else dbufs[i]), T, codec) for i, (d, T) in enumerate(zip(dsts, Ts))]
        dev.retrieve(ops)
        assert dev.sync() == 0
        ref = pool.copy()
        for d, w, T in zip(dsts, wants, Ts):
            oracle.retrieve(ref, d, 0, T, codec, w)
        assert np.array_equal(dev.pool_np(), ref)
        # compose two host-resident parts into one request, the second one re-rotated
        rt = perm[200:230]
        dev.compose([K.ComposeReq(dev.table(rt).data_ptr(), 30, [dev.chunk(hbufs[0], 200, codec, 0), dev.chunk(hbufs[4], 256, codec, 0)],
                                  [0, 208], shape.rope_theta)])
        assert dev.sync() == 0
        kref, kmag = oracle.compose(ref, rt, [(wants[0], 200, codec, 0, 0), (wants[4], 256, codec, 0, 208)], shape.rope_theta, want_ref=True)
        got = dev.pool_np()
        p = 208 + np.arange(256)
        rot = np.zeros(got.shape, dtype=bool)
        rot[:, 0, rt[p // 16], p % 16] = True
        assert np.array_equal(got[~rot], ref[~rot])
        check_rotated_keys(got[:, 0, rt[p // 16], p % 16], kref[:, 208:464], kmag[:, 208:464], ref[:, 0, rt[p // 16], p % 16])
        # layer-wise delivery of a host-resident chunk (every step brings the chunk's bytes over again: correct, not fast)
        before = dev.pool_np()
        lw = perm[232:249]
        K.kdn_retrieve_layerwise(dev.ctx, dev.pool_id, [dev.op(dev.table(lw), 0, hbufs[3], Ts[3], codec)], 2, dev.stream.cuda_stream)
        assert dev.sync() == 0
        oracle.retrieve(before, lw, 0, Ts[3], codec, wants[3])
        assert np.array_equal(dev.pool_np(), before)
        # chunks in files: only the bytes in use need be there; all five in one file at odd offsets, retrieved in one call
        import tempfile
        with tempfile.TemporaryFile() as tf:
            offs, cur = [], 24
            for h, w, T in zip(hbufs, wants, Ts):
                used = oracle.td_used_bytes(w, 3, 2, 64, T, codec)
                offs.append(cur)
                os.pwrite(tf.fileno(), h[:used].numpy().tobytes(), cur)
                cur += used + 40
            fdst = [perm[250 + 20 * i:250 + 20 * i + 17] for i in range(len(Ts))]
            fops = [dev.op(dev.table(d), 0, dbufs[i], T, codec) for i, (d, T) in enumerate(zip(fdst, Ts))]   # (the data address is ignored)
            before = dev.pool_np()
            K.kdn_retrieve_file(dev.ctx, dev.pool_id, fops, [tf.fileno()] * len(Ts), offs, dev.stream.cuda_stream)
            assert dev.sync() == 0
            for d, w, T in zip(fdst, wants, Ts):
                oracle.retrieve(before, d, 0, T, codec, w)
            assert np.array_equal(dev.pool_np(), before)
            with pytest.raises(K.KdnError) as e:                          # storing into a file: the size is not known beforehand
                K.kdn_store_file(dev.ctx, dev.pool_id, [fops[0]], [tf.fileno()], [0], dev.stream.cuda_stream)
            assert e.value.status == K.KDN_E_UNSUPPORTED
            with pytest.raises(K.KdnError) as e:                          # no offset table a store can have written at this place
                K.kdn_retrieve_file(dev.ctx, dev.pool_id, [fops[0]], [tf.fileno()], [offs[0] + 8], dev.stream.cuda_stream)
            assert e.value.status == K.KDN_E_SHAPE
        # a host buffer no store has written is refused, not followed
        junk = dev.chunk_buf(64, codec, pinned=True, fill=0xFF)
        with pytest.raises(K.KdnError) as e:
            dev.retrieve([dev.op(dev.table(dsts[0]), 0, junk, 64, codec)])
        assert e.value.status == K.KDN_E_SHAPE
    finally:
        dev.close()


@pytest.mark.parametrize("shape", SHAPES, ids=IDS)
@pytest.mark.parametrize("codec", [TD8, TD4], ids=["int8td", "int4td"])
def test_keep_list_chunks_against_the_oracle(shape, codec):
    """Keep-lists with the token-delta codecs: the chunk codes the listed tokens (groups of 64 chunk tokens, differences
    along the listed tokens), wherever they sit in the request -- no alignment rule.  Store bytes, retrieve into other
    blocks (device and page-locked host chunk), and a list entry outside the table."""
    bs = shape.block_size
    rng = np.random.default_rng(23 + codec)
    perm = rng.permutation(shape.n_blocks).astype(np.int32)
    span, off = 200, 3
    nb = -(-(off + span) // bs)
    src, dst = perm[:nb], perm[nb:2 * nb]
    pool = make_pool_np(shape, src, off, span, 0.95, seed=41)
    dev = Device(shape, pool_np=pool)
    try:
        K = dev.K
        lists = [np.sort(rng.choice(span, 100, replace=False)), np.arange(span), np.array([7]), np.arange(0, span, 3), np.arange(64) + 5]
        ops, keeps, wants, bufs = [], [], [], []
        for keep in lists:
            keep = keep.astype(np.int32)
            b = dev.chunk_buf(len(keep), codec)
            d_keep = dev.table(keep)
            ops.append(dev.op(dev.table(src), off, b, len(keep), codec))
            keeps.append(d_keep.data_ptr())
            wants.append(oracle.store(pool, src, off, len(keep), codec, keep=keep))
            bufs.append(b)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, ops, keeps, dev.stream.cuda_stream)
        assert dev.sync() == 0
        for b, w, keep in zip(bufs, wants, lists):
            used = oracle.td_used_bytes(w, shape.n_layers, shape.n_kv_heads, shape.head_dim, len(keep), codec)
            got = to_np(b)
            assert np.array_equal(got[:used], w[:used]) and np.all(got[used:] == 0xA5), len(keep)
        assert np.array_equal(dev.pool_np(), pool)
        ref = pool.copy()
        for i, (b, w, keep) in enumerate(zip(bufs, wants, lists)):
            src_buf = b
            if i % 2 == 1:                                                       # every other chunk from page-locked host memory
                src_buf = dev.chunk_buf(len(keep), codec, pinned=True)
                src_buf.copy_(b.cpu())
            K.kdn_retrieve_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(dst), off, src_buf, len(keep), codec)], [keeps[i]], dev.stream.cuda_stream)
            assert dev.sync() == 0
            oracle.retrieve(ref, dst, off, len(keep), codec, w, keep=keep.astype(np.int32))
            assert np.array_equal(dev.pool_np(), ref), i
        bad = np.array([0, 1, 2, nb * bs], dtype=np.int32)                        # the last entry points past the table
        b = dev.chunk_buf(4, codec)
        K.kdn_store_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(src), 0, b, 4, codec)], [dev.table(bad).data_ptr()], dev.stream.cuda_stream)
        assert dev.sync() == K.KDN_E_RANGE
        K.kdn_retrieve_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(dst), 0, bufs[2], 1, codec)], [dev.table(np.array([nb * bs + 5], dtype=np.int32)).data_ptr()],
                              dev.stream.cuda_stream)
        assert dev.sync() == K.KDN_E_RANGE
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


@pytest.mark.parametrize("shape", [SHAPES[0], SHAPES[1], SHAPES[3]], ids=[IDS[0], IDS[1], IDS[3]])   # (rows of 576 are too wide to rotate)
@pytest.mark.parametrize("codec", [TD8, TD4], ids=["int8td", "int4td"])
def test_select_list_compose_against_the_oracle(shape, codec):
    """kdn_compose_select with token-delta chunks: the decoder still decodes whole groups, but only the listed rows leave
    it, and a group without a listed token is not decoded at all.  One part with a list that skips the middle group and
    a position shift (keys re-rotated), one from page-locked host memory delivered whole, one with a single listed token."""
    shape = shape.with_(n_blocks=max(shape.n_blocks, 256))
    bs = shape.block_size
    rng = np.random.default_rng(43 + codec)
    perm = rng.permutation(shape.n_blocks).astype(np.int32)
    T = 170                                                               # three groups: 64 + 64 + 42
    nb = -(-T // bs)
    span = -(-T // 64) * 64
    pool = make_pool_np(shape, perm[:nb], 0, T, 0.9, seed=47)
    dev = Device(shape, pool_np=pool)
    try:
        K = dev.K
        buf = dev.chunk_buf(T, codec)
        dev.store([dev.op(dev.table(perm[:nb]), 0, buf, T, codec)])
        assert dev.sync() == 0
        want = oracle.store(pool, perm[:nb], 0, T, codec)
        hbuf = dev.chunk_buf(T, codec, pinned=True)
        hbuf.copy_(buf.cpu())
        rt = perm[nb:nb + 3 * span // bs + 1]
        sel_a = np.concatenate([np.sort(rng.choice(64, 20, replace=False)), 128 + np.sort(rng.choice(42, 11, replace=False))]).astype(np.int32)
        sel_c = np.array([65], dtype=np.int32)
        d_a, d_c = dev.table(sel_a), dev.table(sel_c)
        before = dev.pool_np()
        K.kdn_compose_select(dev.ctx, dev.pool_id,
                             [K.ComposeReq(dev.table(rt).data_ptr(), len(rt),
                                           [dev.chunk(buf, T, codec, 7), dev.chunk(hbuf, T, codec, span), dev.chunk(buf, T, codec, 0)],
                                           [0, span, 2 * span], shape.rope_theta)],
                             [[(d_a.data_ptr(), len(sel_a)), None, (d_c.data_ptr(), 1)]], dev.stream.cuda_stream)
        assert dev.sync() == 0
        ref = before.copy()
        kref, kmag = oracle.compose(ref, rt, [(want, T, codec, 7, 0), (want, T, codec, span, span), (want, T, codec, 0, 2 * span)],
                                    shape.rope_theta, want_ref=True, select=[sel_a, None, sel_c])
        got = dev.pool_np()
        p = np.concatenate([sel_a, 2 * span + sel_c])                      # the re-rotated positions
        rot = np.zeros(got.shape, dtype=bool)
        rot[:, 0, rt[p // bs], p % bs] = True
        assert np.array_equal(got[~rot], ref[~rot])
        g = got[:, 0, rt[p // bs], p % bs]
        check_rotated_keys(g, kref[:, p], kmag[:, p], ref[:, 0, rt[p // bs], p % bs], min_equal=0.995 if g.size >= 8192 else 0.95)
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [TD8, TD4], ids=["int8td", "int4td"])
def test_a_wait_that_runs_out_in_the_token_delta_kernels(codec):
    """The waits of the planner, the encoder and the decoder are bounded like those of the tile pipeline.  With the
    bound below the latency of a memory access a CTA whose bytes have not landed gives up: KDN_E_TIMEOUT (or, when every
    CTA found its bytes in time, a correct result), nothing written outside the chunk (a planner CTA that gives up
    leaves zero lengths behind, and the encoder trusts no length), the pool untouched by a store; with the default bound
    back the same context is bit-exact again."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=4, head_dim=64, block_size=16, n_blocks=96)
    dev = Device(shape, seed=9)
    try:
        K = dev.K
        host = dev.pool_np()
        tab = np.random.default_rng(6).permutation(96)[:20].astype(np.int32)
        T = 300
        guard = 4096
        whole = dev.chunk_buf(T, codec)                                       # (reference size)
        arena = torch.full((whole.numel() + 2 * guard,), 0x5C, dtype=torch.uint8, device=dev.dev)
        buf = arena[guard:guard + whole.numel()]
        want = oracle.store(host, tab, 0, T, codec)
        used = oracle.td_used_bytes(want, shape.n_layers, shape.n_kv_heads, shape.head_dim, T, codec)
        K.kdn_set_wait_limit_ns(dev.ctx, 40)
        dev.store([dev.op(dev.table(tab), 0, buf, T, codec)])
        st = dev.sync()
        # (a CTA of the store kernels fills its tables before it looks for its rows, so they may all have landed by then)
        assert st in (0, K.KDN_E_TIMEOUT)
        assert np.array_equal(dev.pool_np(), host)
        a = to_np(arena)
        assert np.all(a[:guard] == 0x5C) and np.all(a[-guard:] == 0x5C)       # nothing left the chunk
        assert st != 0 or np.array_equal(a[guard:guard + used], want[:used])
        K.kdn_set_wait_limit_ns(dev.ctx, 0)
        dev.store([dev.op(dev.table(tab), 0, buf, T, codec)])
        assert dev.sync() == 0
        assert np.array_equal(to_np(buf)[:used], want[:used])
        dst = np.random.default_rng(7).permutation(96)[:20].astype(np.int32)
        K.kdn_set_wait_limit_ns(dev.ctx, 40)
        dev.retrieve([dev.op(dev.table(dst), 0, buf, T, codec)])
        assert dev.sync() in (0, K.KDN_E_TIMEOUT)
        K.kdn_set_wait_limit_ns(dev.ctx, 0)
        dev.retrieve([dev.op(dev.table(dst), 0, buf, T, codec)])
        assert dev.sync() == 0
        ref = host.copy()
        oracle.retrieve(ref, dst, 0, T, codec, want)
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [TD8, TD4], ids=["int8td", "int4td"])
def test_a_block_id_outside_the_pool_in_a_store_is_reported_and_nothing_leaves_the_chunk(codec):
    """The planner CTAs of the slices that meet the bad table entry give up and leave zero lengths behind; the other
    slices of the same segments are still placed consistently: KDN_E_RANGE, no byte outside the chunk, the pool as it was."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=4, head_dim=64, block_size=16, n_blocks=96)
    dev = Device(shape, seed=10)
    try:
        K = dev.K
        host = dev.pool_np()
        tab = np.random.default_rng(8).permutation(96)[:20].astype(np.int32)
        bad = tab.copy()
        bad[7] = 96 + 5                                                       # tokens 112 .. 127: the second group
        T, guard = 300, 4096
        n = K.kdn_chunk_bytes(dev.desc, T, codec)
        arena = torch.full((n + 2 * guard,), 0xFF, dtype=torch.uint8, device=dev.dev)   # 0xFF: lengths no sub-stream can have
        buf = arena[guard:guard + n]
        dev.store([dev.op(dev.table(bad), 0, buf, T, codec)])
        assert dev.sync() == K.KDN_E_RANGE
        a = to_np(arena)
        assert np.all(a[:guard] == 0xFF) and np.all(a[-guard:] == 0xFF)
        assert np.array_equal(dev.pool_np(), host)
        dev.store([dev.op(dev.table(tab), 0, buf, T, codec)])
        assert dev.sync() == 0
        want = oracle.store(host, tab, 0, T, codec)
        used = oracle.td_used_bytes(want, shape.n_layers, shape.n_kv_heads, shape.head_dim, T, codec)
        assert np.array_equal(to_np(buf)[:used], want[:used])
    finally:
        dev.close()
