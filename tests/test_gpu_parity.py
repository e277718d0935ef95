"""GPU parity: the CUDA library against the CPU oracle, element by element, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np, bits_to_f64, check_rotated_keys

pytestmark = pytest.mark.gpu

RAW, INT8, INT4 = oracle.RAW_BF16, oracle.INT8_G64, oracle.INT4_G64


def gather_positions(pool_np, table, pos):
    bs = pool_np.shape[3]
    pos = np.asarray(pos)
    return pool_np[:, :, table[pos // bs], pos % bs]


# ----------------------------------------------------------------------------------- toy config --

def test_toy_config_store_retrieve_compose():
    """2 layers, 2 KV heads, head_dim 64, block_size 16, 64 blocks; chunk A of 256 tokens at a seeded random
    table; store, retrieve elsewhere, then compose A at 0 with a second chunk B shifted to 256, theta 1e4."""
    shape = synth.TOY
    dev = Device(shape)
    try:
        rng = np.random.default_rng(synth.SEED_TABLES)
        perm = rng.permutation(shape.n_blocks).astype(np.int32)
        tA, tR, tB, tC = perm[0:16], perm[16:32], perm[32:48], np.concatenate([perm[16:32], perm[48:64]])
        host = dev.pool_np()
        for codec in (RAW, INT8, INT4):
            ref = host.copy()
            # store A and B in one batched call
            bufA, bufB = dev.chunk_buf(256, codec), dev.chunk_buf(256, codec)
            dA, dB = dev.table(tA), dev.table(tB)
            dev.store([dev.op(dA, 0, bufA, 256, codec), dev.op(dB, 0, bufB, 256, codec)])
            assert dev.sync() == 0
            oA, oB = oracle.store(ref, tA, 0, 256, codec), oracle.store(ref, tB, 0, 256, codec)
            assert np.array_equal(to_np(bufA), oA)
            assert np.array_equal(to_np(bufB), oB)
            assert np.array_equal(dev.pool_np(), ref)                      # store does not write the pool
            # retrieve A into 16 other blocks
            dev.retrieve([dev.op(dev.table(tR), 0, bufA, 256, codec)])
            assert dev.sync() == 0
            oracle.retrieve(ref, tR, 0, 256, codec, oA)
            assert np.array_equal(dev.pool_np(), ref)
            if codec == RAW:                                               # store o retrieve = identity
                assert np.array_equal(ref[:, :, tR], ref[:, :, tA])
            # compose [A@0 (delta 0), B@256 (delta 256)] into the 32 blocks holding neither source
            K = dev.K
            parts = [dev.chunk(bufA, 256, codec, 0), dev.chunk(bufB, 256, codec, 0)]
            dC = dev.table(tC)
            dev.compose([K.ComposeReq(dC.data_ptr(), 32, parts, [0, 256], shape.rope_theta)])
            assert dev.sync() == 0
            kref, kmag = oracle.compose(ref, tC, [(oA, 256, codec, 0, 0), (oB, 256, codec, 0, 256)],
                                        shape.rope_theta, want_ref=True)
            got = dev.pool_np()
            # everything except B's re-rotated keys is bit-exact
            mask = np.ones(got.shape, dtype=bool)
            p = 256 + np.arange(256)
            mask[:, 0, tC[p // 16], p % 16] = False
            assert np.array_equal(got[mask], ref[mask])
            gk = gather_positions(got, tC, p)[:, 0]
            ok = gather_positions(ref, tC, p)[:, 0]
            check_rotated_keys(gk, kref[:, 256:512], kmag[:, 256:512], ok)
            # restore the pool for the next codec
            for l in range(shape.n_layers):
                dev.k[l].copy_(torch.from_numpy(host[l, 0].view(np.int16)).view(torch.bfloat16))
                dev.v[l].copy_(torch.from_numpy(host[l, 1].view(np.int16)).view(torch.bfloat16))
    finally:
        dev.close()


# ------------------------------------------------------------------------------------ edge cases --

EDGE_SHAPES = [
    synth.TOY.with_(n_blocks=72, block_size=16),
    synth.TOY.with_(n_blocks=96, block_size=3),
    synth.TOY.with_(n_blocks=200, block_size=1),
    synth.TOY.with_(n_layers=3, n_kv_heads=8, head_dim=128, block_size=32, n_blocks=72),
    synth.TOY.with_(n_layers=1, n_kv_heads=1, head_dim=256, block_size=16, n_blocks=72),
    synth.TOY.with_(n_layers=2, n_kv_heads=3, head_dim=192, block_size=8, n_blocks=72),
]


@pytest.mark.parametrize("shape", EDGE_SHAPES, ids=lambda s: "L%dH%dD%dbs%d" % (s.n_layers, s.n_kv_heads, s.head_dim, s.block_size))
def test_unaligned_ragged_batched_mixed_codecs(shape):
    """One batched call mixing codecs, offsets that start and end mid-block, a 1-token chunk, an empty chunk."""
    dev = Device(shape, seed=77)
    try:
        bs, nb = shape.block_size, shape.n_blocks
        rng = np.random.default_rng(5)
        host = dev.pool_np()
        free = list(rng.permutation(nb))
        cases = []                                       # (src table, off, T, codec)
        span = 6 * bs
        for off, T, codec in [(0, span, RAW), (1 % span, max(1, span - 2), INT8), (bs // 2, 1, INT8), (span - 1, 1, RAW),
                              (2 % span, max(1, span // 2), RAW), (0, 0, INT8), (bs - 1 if bs > 1 else 0, bs + 1, INT8),
                              (3 % span, max(1, span - 5), INT4), (bs // 2, 1, INT4)]:
            tab = np.array([free[i] for i in rng.integers(0, len(free), 6)], dtype=np.int32)   # repeats allowed as a source
            cases.append((tab, off, T, codec))
        bufs, ops = [], []
        for tab, off, T, codec in cases:
            b = dev.chunk_buf(T, codec)
            bufs.append(b)
            ops.append(dev.op(dev.table(tab), off, b, T, codec))
        dev.store(ops)
        assert dev.sync() == 0
        chunks = []
        for (tab, off, T, codec), b in zip(cases, bufs):
            want = oracle.store(host, tab, off, T, codec)
            assert np.array_equal(to_np(b), want), (off, T, codec)
            chunks.append(want)
        assert np.array_equal(dev.pool_np(), host)
        # retrieve all of them into pairwise distinct fresh blocks, in one call, at other offsets
        ref = host.copy()
        ops, used = [], 0
        dst_free = rng.permutation(nb)
        for (tab, off, T, codec), b in zip(cases, bufs):
            off2 = (off + 1) % bs if T else 0
            n_tb = -(-(off2 + T) // bs) if T else 0
            dtab = dst_free[used:used + n_tb].astype(np.int32)
            used += n_tb
            if T:
                ops.append(dev.op(dev.table(dtab), off2, b, T, codec))
                oracle.retrieve(ref, dtab, off2, T, codec, oracle.store(host, tab, off, T, codec))
        dev.retrieve(ops)
        assert dev.sync() == 0
        assert np.array_equal(dev.pool_np(), ref)        # addressed slots right, every other byte untouched
    finally:
        dev.close()


FUSION_WITNESS_ABSMAX = [21.25, 38.5, 46.0, 84.0, 23.0, 25.75,          # for 127/a (int8) ...
                         16.125, 17.25, 19.0, 20.0]                     # ... and for 7/a (int4)


def special_pool(shape):
    """Pool whose groups hit the codec's special cases: zeros, -0, subnormal scales, ties, big outliers, NaN-free."""
    rng = np.random.default_rng(99)
    k, v = synth.make_pool(shape, seed=5)
    pool = synth.pool_to_numpy(k, v)
    flat = pool.reshape(-1, 64)
    n = flat.shape[0]
    f = lambda x: (np.asarray(x, dtype=np.float32).view(np.uint32) >> 16).astype(np.uint16)
    flat[0::11] = 0                                                       # all-zero groups
    flat[1::11] = 0x8000                                                  # all minus zero
    g = np.zeros(64, dtype=np.float32); g[0] = 2.0 ** -120; g[1] = -2.0 ** -121
    flat[2::11] = f(g)                                                    # scale would be subnormal -> flushed
    g = np.zeros(64, dtype=np.float32); g[0] = 127.0; g[1:8] = [0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 63.5]
    flat[3::11] = f(g)                                                    # exact ties
    g = rng.standard_normal(64).astype(np.float32); g[7] = 3.0e4
    flat[4::11] = f((g.view(np.uint32) & 0xffff0000).view(np.float32))    # one huge outlier
    g = (rng.standard_normal(64) * 2.0 ** -110).astype(np.float32)
    flat[5::11] = f((g.view(np.uint32) & 0xffff0000).view(np.float32))    # tiny but normal
    g = np.full(64, 2.0 ** 120, dtype=np.float32); g[::2] *= -1
    flat[6::11] = f(g)                                                    # huge magnitudes
    # products that round TO a tie: x = a/2 with fl(127/a) below 127/a, so fl(x * inv) = 63.5 -> 64 while
    # a single-rounding fused multiply-add would give 63 (see tests/test_oracle_codec.py)
    for k, a in enumerate(FUSION_WITNESS_ABSMAX):
        g = np.zeros(64, dtype=np.float32); g[0] = a; g[1] = a / 2; g[2] = -a / 2; g[33] = -a; g[40] = a / 2
        flat[7 + 11 * k::11 * len(FUSION_WITNESS_ABSMAX)] = f(g)
    return pool


@pytest.mark.parametrize("INT8", [INT8, INT4], ids=["int8", "int4"])
def test_codec_special_groups_bit_exact(INT8):
    shape = synth.TOY.with_(n_blocks=32, block_size=8)
    pool = special_pool(shape)
    dev = Device(shape, pool_np=pool)
    try:
        tab = np.random.default_rng(1).permutation(32)[:12].astype(np.int32)
        T = 12 * 8 - 5
        buf = dev.chunk_buf(T, INT8)
        dev.store([dev.op(dev.table(tab), 3, buf, T, INT8)])
        assert dev.sync() == 0
        want = oracle.store(pool, tab, 3, T, INT8)
        assert np.array_equal(to_np(buf), want)
        dst = np.setdiff1d(np.arange(32), tab)[:12].astype(np.int32)
        dev.retrieve([dev.op(dev.table(dst), 1, buf, T, INT8)])
        assert dev.sync() == 0
        ref = pool.copy()
        oracle.retrieve(ref, dst, 1, T, INT8, want)
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


def test_raw_copy_preserves_every_bit_pattern():
    shape = synth.TOY.with_(n_blocks=16, block_size=16)
    pool = np.arange(2 * 2 * 16 * 16 * 2 * 64, dtype=np.uint32).astype(np.uint16).reshape(2, 2, 16, 16, 2, 64)  # all 65536 patterns
    dev = Device(shape, pool_np=pool)
    try:
        src = np.arange(8, dtype=np.int32)
        dst = np.arange(8, 16, dtype=np.int32)[::-1].copy()
        buf = dev.chunk_buf(128, RAW)
        dev.store([dev.op(dev.table(src), 0, buf, 128, RAW)])
        dev.retrieve([dev.op(dev.table(dst), 0, buf, 128, RAW)])
        assert dev.sync() == 0
        got = dev.pool_np()
        assert np.array_equal(got[:, :, dst], pool[:, :, src])
        assert np.array_equal(got[:, :, src], pool[:, :, src])
        assert np.array_equal(to_np(buf), oracle.store(pool, src, 0, 128, RAW))
    finally:
        dev.close()


@pytest.mark.parametrize("D,codec", [(64, RAW), (64, INT8), (128, RAW), (128, INT8), (256, INT8), (192, INT8), (192, RAW), (80, RAW),
                                     (64, INT4), (128, INT4), (192, INT4)])
def test_compose_unaligned_parts_negative_and_large_deltas(D, codec):
    H = 2 if D != 80 else 1
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=H, head_dim=D, block_size=8, n_blocks=64, rope_theta=500000.0)
    dev = Device(shape, seed=31)
    try:
        rng = np.random.default_rng(8)
        host = dev.pool_np()
        perm = rng.permutation(64).astype(np.int32)
        src_tabs = [perm[0:4], perm[4:8], perm[8:13], perm[13:15]]
        Ts = [29, 17, 32, 9]
        base = [0, 131072, 5, 40]
        dst = [3, 32, 49, 90]                           # deltas 3, -131040, 44, 50; gaps between parts stay untouched
        req_tab = perm[20:33]                           # 13 blocks = 104 positions
        bufs, ochunks, ops = [], [], []
        for tab, T in zip(src_tabs, Ts):
            b = dev.chunk_buf(T, codec)
            bufs.append(b)
            ops.append(dev.op(dev.table(tab), 1, b, T, codec))
            ochunks.append(oracle.store(host, tab, 1, T, codec))
        dev.store(ops)
        assert dev.sync() == 0
        for b, oc in zip(bufs, ochunks):
            assert np.array_equal(to_np(b), oc)
        K = dev.K
        parts = [dev.chunk(b, T, codec, bp) for b, T, bp in zip(bufs, Ts, base)]
        dtab = dev.table(req_tab)
        dev.compose([K.ComposeReq(dtab.data_ptr(), len(req_tab), parts, dst, shape.rope_theta)])
        assert dev.sync() == 0
        ref = host.copy()
        kref, kmag = oracle.compose(ref, req_tab, [(oc, T, codec, bp, dp) for oc, T, bp, dp in zip(ochunks, Ts, base, dst)],
                                    shape.rope_theta, want_ref=True)
        got = dev.pool_np()
        rot = np.zeros(got.shape, dtype=bool)
        for T, dp in zip(Ts, dst):
            p = dp + np.arange(T)
            rot[:, 0, req_tab[p // 8], p % 8] = True
        assert np.array_equal(got[~rot], ref[~rot])
        for T, dp in zip(Ts, dst):
            p = dp + np.arange(T)
            check_rotated_keys(gather_positions(got, req_tab, p)[:, 0], kref[:, dp:dp + T], kmag[:, dp:dp + T],
                               gather_positions(ref, req_tab, p)[:, 0])
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [RAW, INT8, INT4])
def test_compose_with_zero_delta_equals_retrieve(codec):
    shape = synth.TOY.with_(n_blocks=40, block_size=16)
    dev = Device(shape, seed=3)
    try:
        host = dev.pool_np()
        perm = np.random.default_rng(4).permutation(40).astype(np.int32)
        T = 50
        buf = dev.chunk_buf(T, codec)
        dev.store([dev.op(dev.table(perm[:4]), 2, buf, T, codec)])
        dtab = dev.table(perm[10:15])
        dev.retrieve([dev.op(dtab, 7, buf, T, codec)])
        assert dev.sync() == 0
        a = dev.pool_np()
        dtab2 = dev.table(perm[20:25])
        dev.compose([dev.K.ComposeReq(dtab2.data_ptr(), 5, [dev.chunk(buf, T, codec, 7)], [7], 10000.0)])
        assert dev.sync() == 0
        b = dev.pool_np()
        p = 7 + np.arange(T)
        assert np.array_equal(gather_positions(b, perm[20:25], p), gather_positions(a, perm[10:15], p))
        ref = host.copy()
        oc = oracle.store(host, perm[:4], 2, T, codec)
        oracle.retrieve(ref, perm[10:15], 7, T, codec, oc)
        oracle.compose(ref, perm[20:25], [(oc, T, codec, 7, 7)], 10000.0)
        assert np.array_equal(b, ref)
    finally:
        dev.close()


def test_block_id_outside_the_pool_is_reported_not_faulted():
    shape = synth.TOY.with_(n_blocks=16, block_size=16)
    dev = Device(shape, seed=2)
    try:
        host = dev.pool_np()
        tab = np.array([3, 16, 5, -1], dtype=np.int32)          # 16 and -1 are outside [0, 16)
        buf = dev.chunk_buf(64, RAW, fill=0xA5)
        dev.store([dev.op(dev.table(tab), 0, buf, 64, RAW)])
        assert dev.sync() == dev.K.KDN_E_RANGE
        assert dev.sync() == 0                                   # the status is cleared by reading it
        got = to_np(buf).view(np.uint16).reshape(2, 2, 64, 2, 64)
        assert np.array_equal(got[:, :, 0:16], host[:, :, 3])    # tiles with a valid id are still done
        assert np.array_equal(got[:, :, 32:48], host[:, :, 5])
        assert np.all(got[:, :, 16:32] == 0xA5A5) and np.all(got[:, :, 48:64] == 0xA5A5)
        dev.retrieve([dev.op(dev.table(tab), 0, buf, 64, RAW)])
        assert dev.sync() == dev.K.KDN_E_RANGE
        ref = host.copy()
        ref[:, :, 3] = host[:, :, 3]; ref[:, :, 5] = host[:, :, 5]
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


def test_argument_errors_launch_nothing():
    shape = synth.TOY
    dev = Device(shape)
    try:
        K = dev.K
        n0 = K.kdn_launch_count(dev.ctx)
        tab = dev.table(np.arange(2, dtype=np.int32))
        buf = dev.chunk_buf(40, RAW)
        with pytest.raises(K.KdnError) as e:
            dev.store([dev.op(tab, 0, buf, 40, RAW)])           # 40 tokens > 2 blocks
        assert e.value.status == K.KDN_E_RANGE
        with pytest.raises(K.KdnError) as e:
            K.kdn_store(dev.ctx, 7, [], dev.stream.cuda_stream)
        assert e.value.status == K.KDN_E_INVAL
        bad = dev.op(tab, 0, buf[:32 * 1024], 32, RAW)
        bad.chunk.data += 8
        with pytest.raises(K.KdnError) as e:
            dev.retrieve([bad])
        assert e.value.status == K.KDN_E_ALIGN
        assert K.kdn_launch_count(dev.ctx) == n0
        assert dev.sync() == 0
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [RAW, INT8, INT4])
def test_pinned_host_chunks_through_small_staging_slabs(codec):
    """Chunks in page-locked host memory: store copies out, retrieve and compose copy in, layer range by layer
    range through staging slabs far smaller than the chunk."""
    shape = synth.TOY.with_(n_layers=6, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=64)
    dev = Device(shape, seed=12)
    try:
        K = dev.K
        K.kdn_set_staging_bytes(dev.ctx, 96 * 1024)             # one layer of 100 tokens is 50 KiB raw
        host = dev.pool_np()
        perm = np.random.default_rng(6).permutation(64).astype(np.int32)
        T = 100
        hbuf1, hbuf2 = dev.chunk_buf(T, codec, pinned=True), dev.chunk_buf(37, codec, pinned=True)
        dbuf = dev.chunk_buf(T, codec)
        dev.store([dev.op(dev.table(perm[:7]), 5, hbuf1, T, codec), dev.op(dev.table(perm[7:10]), 0, hbuf2, 37, codec),
                   dev.op(dev.table(perm[:7]), 5, dbuf, T, codec)])
        assert dev.sync() == 0
        o1, o2 = oracle.store(host, perm[:7], 5, T, codec), oracle.store(host, perm[7:10], 0, 37, codec)
        assert np.array_equal(to_np(hbuf1), o1)
        assert np.array_equal(to_np(hbuf2), o2)
        assert np.array_equal(to_np(dbuf), o1)
        ref = host.copy()
        dev.retrieve([dev.op(dev.table(perm[20:27]), 3, hbuf1, T, codec), dev.op(dev.table(perm[30:33]), 9, hbuf2, 37, codec)])
        assert dev.sync() == 0
        oracle.retrieve(ref, perm[20:27], 3, T, codec, o1)
        oracle.retrieve(ref, perm[30:33], 9, 37, codec, o2)
        assert np.array_equal(dev.pool_np(), ref)
        # compose from host chunks, one rotated
        rt = perm[40:50]
        dt = dev.table(rt)
        dev.compose([K.ComposeReq(dt.data_ptr(), 10, [dev.chunk(hbuf2, 37, codec, 0), dev.chunk(hbuf1, T, codec, 0)], [0, 40], 10000.0)])
        assert dev.sync() == 0
        kref, kmag = oracle.compose(ref, rt, [(o2, 37, codec, 0, 0), (o1, T, codec, 0, 40)], 10000.0, want_ref=True)
        got = dev.pool_np()
        p = 40 + np.arange(T)
        rot = np.zeros(got.shape, dtype=bool)
        rot[:, 0, rt[p // 16], p % 16] = True
        assert np.array_equal(got[~rot], ref[~rot])
        check_rotated_keys(gather_positions(got, rt, p)[:, 0], kref[:, 40:40 + T], kmag[:, 40:40 + T],
                           gather_positions(ref, rt, p)[:, 0])
    finally:
        dev.close()


def test_tuning_shapes_give_identical_results():
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=8, head_dim=128, block_size=16, n_blocks=64)
    dev = Device(shape, seed=41)
    try:
        K = dev.K
        host = dev.pool_np()
        tab = np.random.default_rng(2).permutation(64)[:20].astype(np.int32)
        T, off = 300, 7
        want = {c: oracle.store(host, tab, off, T, c) for c in (RAW, INT8, INT4)}
        for tile, stages, ctas, groups, lag in [(0, 0, 0, 0, 0), (2048, 4, 1, 1, 1), (4096, 12, 3, 3, 2), (32768, 4, 1, 4, 2),
                                                (16384, 5, 2, 2, 3), (1024, 16, 4, 6, 4), (8192, 3, 2, 3, 1), (8192, 7, 1, 6, 1)]:
            K.kdn_set_tuning(dev.ctx, tile, stages, ctas, groups, lag)
            for c in (RAW, INT8, INT4):
                buf = dev.chunk_buf(T, c)
                dev.store([dev.op(dev.table(tab), off, buf, T, c)])
                assert dev.sync() == 0
                assert np.array_equal(to_np(buf), want[c]), (tile, stages, ctas, groups, lag, c)
        with pytest.raises(K.KdnError):
            K.kdn_set_tuning(dev.ctx, 100, 0, 0)                 # not a multiple of 128
    finally:
        dev.close()


def test_more_ops_than_one_launch_carries():
    """7000 tiny ops in one call: the library splits them over several launches; every chunk must still be right."""
    shape = synth.TOY.with_(n_layers=1, n_kv_heads=1, head_dim=64, block_size=4, n_blocks=512)
    dev = Device(shape, seed=8)
    try:
        K = dev.K
        rng = np.random.default_rng(3)
        host = dev.pool_np()
        n = 7000
        Ts = rng.integers(0, 4, n)                              # 0..3 tokens, some empty
        offs = rng.integers(0, 4, n)
        codecs = rng.integers(0, 3, n)
        tabs = rng.integers(0, 512, (n, 2)).astype(np.int32)     # two blocks each, repeats allowed as a source
        d_tabs = dev.table(tabs.reshape(-1))
        sizes = [K.kdn_chunk_bytes(dev.desc, int(t), int(c)) for t, c in zip(Ts, codecs)]
        starts = np.concatenate([[0], np.cumsum([(sz + 255) // 256 * 256 for sz in sizes])])
        arena = torch.full((int(starts[-1]) + 256,), 0xA5, dtype=torch.uint8, device=dev.dev)
        ops = [K.XferOp(d_tabs.data_ptr() + i * 8, 2, int(offs[i]),
                        K.Chunk(arena.data_ptr() + int(starts[i]), sizes[i], int(Ts[i]), int(codecs[i]))) for i in range(n)]
        n0 = K.kdn_launch_count(dev.ctx)
        dev.store(ops)
        assert dev.sync() == 0
        assert K.kdn_launch_count(dev.ctx) - n0 >= 2
        got = to_np(arena)
        for i in range(n):
            want = oracle.store(host, tabs[i], int(offs[i]), int(Ts[i]), int(codecs[i]))
            assert np.array_equal(got[starts[i]:starts[i] + sizes[i]], want), i
            assert np.all(got[starts[i] + sizes[i]:starts[i + 1]] == 0xA5)       # gaps between chunks untouched
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [RAW, INT8, INT4])
def test_layerwise_retrieve_equals_retrieve_and_events_order_layers(codec):
    """Layer-wise delivery: same bits as a plain retrieve; after waiting for layer l's event, layers 0..l are complete
    (checked while later layers may still be in flight); device and pinned-host chunks mixed in one call."""
    shape = synth.TOY.with_(n_layers=7, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=64)
    dev = Device(shape, seed=19)
    try:
        K = dev.K
        K.kdn_set_staging_bytes(dev.ctx, 64 * 1024)
        host = dev.pool_np()
        perm = np.random.default_rng(9).permutation(64).astype(np.int32)
        T1, T2 = 70, 33
        b1, b2 = dev.chunk_buf(T1, codec), dev.chunk_buf(T2, codec, pinned=True)
        dev.store([dev.op(dev.table(perm[:5]), 3, b1, T1, codec), dev.op(dev.table(perm[5:8]), 0, b2, T2, codec)])
        assert dev.sync() == 0
        ops = [dev.op(dev.table(perm[20:25]), 9, b1, T1, codec), dev.op(dev.table(perm[30:33]), 2, b2, T2, codec)]
        ref = host.copy()
        oracle.retrieve(ref, perm[20:25], 9, T1, codec, oracle.store(host, perm[:5], 3, T1, codec))
        oracle.retrieve(ref, perm[30:33], 2, T2, codec, oracle.store(host, perm[5:8], 0, T2, codec))
        events = [torch.cuda.Event() for _ in range(shape.n_layers)]
        for e in events:
            e.record(dev.stream)                                  # creates the underlying CUDA event
        torch.cuda.synchronize()
        K.kdn_retrieve_layerwise(dev.ctx, dev.pool_id, ops, 3, dev.stream.cuda_stream, 0, [e.cuda_event for e in events])
        for l in range(shape.n_layers):
            events[l].synchronize()
            got_k = dev.k[l].view(torch.int16).cpu().numpy().view(np.uint16)
            got_v = dev.v[l].view(torch.int16).cpu().numpy().view(np.uint16)
            assert np.array_equal(got_k, ref[l, 0]) and np.array_equal(got_v, ref[l, 1]), l
        assert dev.sync() == 0
        assert np.array_equal(dev.pool_np(), ref)
        with pytest.raises(K.KdnError):
            K.kdn_retrieve_layerwise(dev.ctx, dev.pool_id, ops, 0, dev.stream.cuda_stream)
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [RAW, INT8])
def test_staged_calls_are_ordered_on_the_callers_stream(codec):
    """Host-resident chunks move on a side stream, but the call is ordered on cuda_stream alone: (a) an event recorded
    on cuda_stream after a store covers the bytes in page-locked memory, even when the caller's side stream is busy;
    (b) a page-locked chunk filled by a copy on cuda_stream is retrieved without a host synchronisation in between."""
    shape = synth.TOY.with_(n_layers=6, n_kv_heads=4, head_dim=64, block_size=16, n_blocks=128)
    dev = Device(shape, seed=77)
    try:
        K = dev.K
        K.kdn_set_staging_bytes(dev.ctx, 1024 * 1024)          # one layer of 400 tokens is 400 KiB raw
        host = dev.pool_np()
        perm = np.random.default_rng(8).permutation(128).astype(np.int32)
        T = 400
        want = oracle.store(host, perm[:26], 9, T, codec)
        ballast = torch.empty(1 << 28, dtype=torch.uint8, device=dev.dev)
        # (a) the caller's own side stream is kept busy, so the copies out of the slabs start late
        side = torch.cuda.Stream(device=dev.dev)
        hbuf = dev.chunk_buf(T, codec, pinned=True, fill=0)
        with torch.cuda.stream(side):
            for _ in range(8):
                ballast.fill_(1)
        K.kdn_store(dev.ctx, dev.pool_id, [dev.op(dev.table(perm[:26]), 9, hbuf, T, codec)], dev.stream.cuda_stream, side.cuda_stream)
        ev = torch.cuda.Event()
        ev.record(dev.stream)
        ev.synchronize()                                        # nothing else is waited for
        assert np.array_equal(hbuf.numpy(), want)
        torch.cuda.synchronize()
        # (b) the chunk reaches page-locked memory by a copy queued on cuda_stream behind other work
        hbuf2 = dev.chunk_buf(T, codec, pinned=True, fill=0)
        staged = torch.from_numpy(want).to(dev.dev)
        torch.cuda.synchronize()
        with torch.cuda.stream(dev.stream):
            for _ in range(8):
                ballast.fill_(2)
            hbuf2.copy_(staged, non_blocking=True)
        dev.retrieve([dev.op(dev.table(perm[40:66]), 2, hbuf2, T, codec)])
        assert dev.sync() == 0
        ref = host.copy()
        oracle.retrieve(ref, perm[40:66], 2, T, codec, want)
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


@pytest.mark.parametrize("codec,bs", [(RAW, 16), (INT8, 16), (INT8, 1)], ids=["raw", "int8", "int8-as-token-rows"])
def test_a_wait_that_runs_out_is_reported_and_the_context_recovers(codec, bs):
    """Every wait inside the tile pipeline is bounded.  With the bound set below the latency of a memory access the
    launch gives up at once: the call returns, kdn_status_sync reports KDN_E_TIMEOUT, no CTA leaves with a copy in
    flight, and once the default bound is back the same context gives bit-exact results.  (block_size 1: the kernels
    whose tiles take up to 16 token rows.)"""
    nblk = 64 * 16 // bs
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=4, head_dim=64, block_size=bs, n_blocks=nblk)
    dev = Device(shape, seed=5)
    try:
        K = dev.K
        host = dev.pool_np()
        tab = np.random.default_rng(4).permutation(nblk)[:20 * 16 // bs].astype(np.int32)
        T, off = 300, 5
        buf = dev.chunk_buf(T, codec)
        K.kdn_set_wait_limit_ns(dev.ctx, 40)
        dev.store([dev.op(dev.table(tab), off, buf, T, codec)])
        assert dev.sync() == K.KDN_E_TIMEOUT
        assert dev.sync() == 0                                  # the status word was cleared by the read
        assert np.array_equal(dev.pool_np(), host)              # a store never writes the pool
        K.kdn_set_wait_limit_ns(dev.ctx, 0)                     # back to the default
        dev.store([dev.op(dev.table(tab), off, buf, T, codec)])
        assert dev.sync() == 0
        assert np.array_equal(to_np(buf), oracle.store(host, tab, off, T, codec))
        dst = np.random.default_rng(5).permutation(nblk)[:20 * 16 // bs].astype(np.int32)
        K.kdn_set_wait_limit_ns(dev.ctx, 40)                    # the same for a retrieve: it may have written some rows, no more
        dev.retrieve([dev.op(dev.table(dst), off, buf, T, codec)])
        assert dev.sync() == K.KDN_E_TIMEOUT
        K.kdn_set_wait_limit_ns(dev.ctx, 0)
        dev.retrieve([dev.op(dev.table(dst), off, buf, T, codec)])
        assert dev.sync() == 0
        ref = host.copy()
        oracle.retrieve(ref, dst, off, T, codec, oracle.store(host, tab, off, T, codec))
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()


@pytest.mark.parametrize("codec", [INT8, INT4])
@pytest.mark.parametrize("bs,heads,head_dim", [(1, 8, 128), (2, 2, 128), (1, 2, 64), (4, 1, 64)])
def test_coded_ops_on_pool_blocks_of_2_kib_or_less_run_as_token_rows(codec, bs, heads, head_dim):
    """Pool blocks of at most 2 KiB: a coding tile that ends with its block would be tiny, so the launch takes whole
    token rows, several per tile, wherever their blocks are.  Same bytes, same pool as any other dense op."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=heads, head_dim=head_dim, block_size=bs, n_blocks=2048)
    dev = Device(shape, seed=83)
    try:
        K = dev.K
        rng = np.random.default_rng(bs * 10 + codec)
        host = dev.pool_np()
        perm = rng.permutation(2048).astype(np.int32)
        ops, metas, used = [], [], 0
        for T, off in ((150, 0), (64, 3), (1, 0), (37, 5 * bs + 1), (257, 2)):
            nb = -(-(off + T) // bs)
            tab = perm[used:used + nb]
            used += nb
            buf = dev.chunk_buf(T, codec)
            ops.append(dev.op(dev.table(tab), off, buf, T, codec))
            metas.append((tab, off, T, buf))
        dev.store(ops)
        assert dev.sync() == 0
        assert "rows" in K.kdn_last_launch(dev.ctx)["kernel"]
        wants = [oracle.store(host, tab, off, T, codec) for tab, off, T, _ in metas]
        for (tab, off, T, buf), want in zip(metas, wants):
            assert np.array_equal(to_np(buf), want), (T, off)
        assert np.array_equal(dev.pool_np(), host)
        ref = host.copy()
        rops = []
        for (tab, off, T, buf), want in zip(metas, wants):
            off2 = off + 1
            nb = -(-(off2 + T) // bs)
            dtab = perm[used:used + nb]
            used += nb
            rops.append(dev.op(dev.table(dtab), off2, buf, T, codec))
            oracle.retrieve(ref, dtab, off2, T, codec, want)
        dev.retrieve(rops)
        assert dev.sync() == 0
        assert "rows" in K.kdn_last_launch(dev.ctx)["kernel"]
        assert np.array_equal(dev.pool_np(), ref)
    finally:
        dev.close()
