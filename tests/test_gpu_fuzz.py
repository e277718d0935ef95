"""Seeded random parity cases: shapes, block sizes, offsets, lengths, codecs and batch mixes drawn at random, every call
checked against the CPU oracle (store: chunk bytes; retrieve: the whole pool; compose: exact off the re-rotated keys,
rotation tolerance on them).  The other GPU tests pick their cases by hand; this one looks where nobody thought to."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np, check_rotated_keys

pytestmark = pytest.mark.gpu
RAW, INT8, INT4, KC8, KC4, TD8, TD4 = range(7)
GROUPED = (KC8, KC4, TD8, TD4)          # codecs whose first token must sit at a block start, block_size | 64


def chunk_equal(got, want, shape, T, codec):
    if codec in (TD8, TD4):
        used = oracle.td_used_bytes(want, shape.n_layers, shape.n_kv_heads, shape.head_dim, T, codec)
        return np.array_equal(got[:used], want[:used])
    return np.array_equal(got, want)


@pytest.mark.parametrize("seed", range(48))
def test_random_batches_against_the_oracle(seed):
    rng = np.random.default_rng(1000 + seed)
    D = int(rng.choice([64, 128, 192, 256]))
    H = int(rng.choice([1, 2, 3, 8] if D <= 128 else [1, 2]))
    bs = int(rng.choice([1, 2, 4, 8, 16, 32, 64]))
    L = int(rng.integers(1, 4))
    n_blocks = max(64, 4096 // bs)
    shape = synth.TOY.with_(n_layers=L, n_kv_heads=H, head_dim=D, block_size=bs, n_blocks=n_blocks,
                            rope_theta=float(rng.choice([1e4, 5e5])))
    dev = Device(shape, seed=200 + seed)
    try:
        K = dev.K
        pool = dev.pool_np()
        n_ops = int(rng.integers(1, 40))
        free = list(rng.permutation(n_blocks))
        ops, metas = [], []
        for _ in range(n_ops):
            codec = int(rng.integers(0, 7))
            T = int(rng.choice([0, 1, 2, 15, 16, 17, 63, 64, 65, 100, 130, 200])) if rng.random() < 0.7 else int(rng.integers(0, 700))
            off = int(rng.integers(0, 3 * bs)) if codec not in GROUPED else int(rng.integers(0, 3)) * bs
            if codec in GROUPED and 64 % bs:
                codec = int(rng.integers(0, 3))
                off = int(rng.integers(0, 3 * bs))
            nb = max(1, -(-(off + T) // bs))
            if len(free) < 3 * nb + 2:
                break
            tab = np.array([free.pop() for _ in range(nb)], dtype=np.int32)
            buf = dev.chunk_buf(T, codec, pinned=codec not in (TD8, TD4) and rng.random() < 0.2)
            ops.append(dev.op(dev.table(tab), off, buf, T, codec))
            metas.append((tab, off, T, codec, buf))
        dev.store(ops)
        assert dev.sync() == 0
        wants = []
        for tab, off, T, codec, buf in metas:
            want = oracle.store(pool, tab, off, T, codec)
            wants.append(want)
            assert T == 0 or chunk_equal(to_np(buf), want, shape, T, codec), (seed, codec, T, off)
        assert np.array_equal(dev.pool_np(), pool)
        # retrieve everything into fresh blocks at another offset, in one call
        ref = pool.copy()
        rops, placed = [], []
        for (tab, off, T, codec, buf), want in zip(metas, wants):
            off2 = int(rng.integers(0, 3 * bs)) if codec not in GROUPED else int(rng.integers(0, 3)) * bs
            nb = max(1, -(-(off2 + T) // bs))
            if len(free) < nb:
                continue
            dtab = np.array([free.pop() for _ in range(nb)], dtype=np.int32)
            rops.append(dev.op(dev.table(dtab), off2, buf, T, codec))
            oracle.retrieve(ref, dtab, off2, T, codec, want)
            placed.append((dtab, off2, T, codec, buf, want))
        dev.retrieve(rops)
        assert dev.sync() == 0
        assert np.array_equal(dev.pool_np(), ref)
        # compose a few of the chunks into one request, each with its own base position
        picks = [p for p in placed if p[2] > 0][:4]
        wide = D * H > 512 and 256 % D != 0                       # rows too wide for the rotating token-delta decoder
        pos, parts, oparts = int(rng.integers(0, bs)), [], []
        for dtab, off2, T, codec, buf, want in picks:
            if codec in GROUPED:
                pos = -(-pos // bs) * bs
            base = int(rng.choice([0, pos, 7, 100000])) if codec not in GROUPED else int(rng.choice([0, pos, 3 * bs, 4096 * bs]))
            if codec in GROUPED and wide:
                base = pos
            parts.append(dev.chunk(buf, T, codec, base))
            oparts.append((want, T, codec, base, pos))
            pos += T + int(rng.integers(0, 4))
        nbr = -(-pos // bs) + 1
        if parts and len(free) >= nbr:
            rtab = np.array([free.pop() for _ in range(nbr)], dtype=np.int32)
            before = dev.pool_np()
            dev.compose([K.ComposeReq(dev.table(rtab).data_ptr(), nbr, parts, [o[4] for o in oparts], shape.rope_theta)])
            assert dev.sync() == 0
            ref2 = before.copy()
            kref, kmag = oracle.compose(ref2, rtab, oparts, shape.rope_theta, want_ref=True)
            got = dev.pool_np()
            rot = np.zeros(got.shape, dtype=bool)
            g, r64, m64, o = [], [], [], []
            for want, T, codec, base, dpos in oparts:
                if base != dpos:
                    p = dpos + np.arange(T)
                    rot[:, 0, rtab[p // bs], p % bs] = True
                    g.append(got[:, 0, rtab[p // bs], p % bs])
                    o.append(ref2[:, 0, rtab[p // bs], p % bs])
                    r64.append(kref[:, dpos:dpos + T])
                    m64.append(kmag[:, dpos:dpos + T])
            assert np.array_equal(got[~rot], ref2[~rot]), seed
            if g:
                g, o, r64, m64 = (np.concatenate(x, axis=1) for x in (g, o, r64, m64))
                check_rotated_keys(g, r64, m64, o, min_equal=0.995 if g.size >= 8192 else 0.95)
    finally:
        dev.close()


@pytest.mark.parametrize("seed", range(32))
def test_random_keep_and_select_lists_against_the_oracle(seed):
    """Token lists under random shapes: a batch of keep-list stores in every codec (bytes against the oracle), their
    keep-list retrieves into other blocks (the whole pool), then one compose with a select-list per part (listed
    positions against the oracle, re-rotated keys within the rotation tolerance, everything else untouched)."""
    rng = np.random.default_rng(5000 + seed)
    D = int(rng.choice([64, 128, 192, 256]))
    H = int(rng.choice([1, 2, 3, 8] if D <= 128 else [1, 2]))
    bs = int(rng.choice([1, 2, 4, 8, 16, 32, 64]))
    L = int(rng.integers(1, 4))
    n_blocks = max(96, 6144 // bs)
    shape = synth.TOY.with_(n_layers=L, n_kv_heads=H, head_dim=D, block_size=bs, n_blocks=n_blocks,
                            rope_theta=float(rng.choice([1e4, 5e5])))
    dev = Device(shape, seed=300 + seed)
    try:
        K = dev.K
        pool = dev.pool_np()
        free = list(rng.permutation(n_blocks))
        span = int(rng.choice([70, 130, 260]))
        nb = -(-(3 * bs + span) // bs)
        ops, keeps, metas = [], [], []
        reserve = 4 * (span + 4) // bs + 8                                   # blocks of the composed request
        for _ in range(max(1, min(int(rng.integers(1, 8)), (n_blocks - reserve) // (2 * nb)))):
            codec = int(rng.integers(0, 7))
            off = int(rng.integers(0, 3 * bs))
            n = int(rng.choice([1, 2, 17, 63, 64, 65, span // 2, span]))
            keep = np.sort(rng.choice(span, n, replace=False)).astype(np.int32)
            tab = np.array([free.pop() for _ in range(nb)], dtype=np.int32)
            buf = dev.chunk_buf(n, codec)
            ops.append(dev.op(dev.table(tab), off, buf, n, codec))
            keeps.append(dev.table(keep).data_ptr())
            metas.append((tab, off, n, codec, buf, keep))
        K.kdn_store_sparse(dev.ctx, dev.pool_id, ops, keeps, dev.stream.cuda_stream)
        assert dev.sync() == 0
        wants = []
        for tab, off, n, codec, buf, keep in metas:
            want = oracle.store(pool, tab, off, n, codec, keep=keep)
            wants.append(want)
            assert chunk_equal(to_np(buf), want, shape, n, codec), (seed, codec, n, off)
        assert np.array_equal(dev.pool_np(), pool)
        ref = pool.copy()
        rops = []
        for (tab, off, n, codec, buf, keep), want in zip(metas, wants):
            dtab = np.array([free.pop() for _ in range(nb)], dtype=np.int32)
            rops.append(dev.op(dev.table(dtab), off, buf, n, codec))
            oracle.retrieve(ref, dtab, off, n, codec, want, keep=keep)
        K.kdn_retrieve_sparse(dev.ctx, dev.pool_id, rops, keeps, dev.stream.cuda_stream)
        assert dev.sync() == 0
        assert np.array_equal(dev.pool_np(), ref)
        # compose with select-lists: each stored chunk is an ordinary chunk of n tokens
        wide = D * H > 512 and 256 % D != 0
        pos, parts, oparts, sels, osels = 0, [], [], [], []
        for (tab, off, n, codec, buf, keep), want in list(zip(metas, wants))[:4]:
            if D % 16:
                break
            if codec in GROUPED:
                pos = -(-pos // bs) * bs
                if 64 % bs:
                    continue
            base = int(rng.choice([0, pos, 11, 70000]))
            if codec in (TD8, TD4) and wide:
                base = pos
            sel = np.sort(rng.choice(n, int(rng.integers(1, n + 1)), replace=False)).astype(np.int32) if rng.random() < 0.8 else None
            parts.append(dev.chunk(buf, n, codec, base))
            oparts.append((want, n, codec, base, pos))
            sels.append((dev.table(sel).data_ptr(), len(sel)) if sel is not None else None)
            osels.append(sel)
            pos += n + int(rng.integers(0, 4))
        nbr = -(-pos // bs) + 1
        if parts and len(free) >= nbr:
            rtab = np.array([free.pop() for _ in range(nbr)], dtype=np.int32)
            before = dev.pool_np()
            K.kdn_compose_select(dev.ctx, dev.pool_id, [K.ComposeReq(dev.table(rtab).data_ptr(), nbr, parts, [o[4] for o in oparts], shape.rope_theta)],
                                 [sels], dev.stream.cuda_stream)
            assert dev.sync() == 0
            ref2 = before.copy()
            kref, kmag = oracle.compose(ref2, rtab, oparts, shape.rope_theta, want_ref=True, select=osels)
            got = dev.pool_np()
            rot = np.zeros(got.shape, dtype=bool)
            g, o, r64, m64 = [], [], [], []
            for (want, n, codec, base, dpos), sel in zip(oparts, osels):
                if base != dpos:
                    p = dpos + (sel if sel is not None else np.arange(n))
                    rot[:, 0, rtab[p // bs], p % bs] = True
                    g.append(got[:, 0, rtab[p // bs], p % bs])
                    o.append(ref2[:, 0, rtab[p // bs], p % bs])
                    r64.append(kref[:, p])
                    m64.append(kmag[:, p])
            assert np.array_equal(got[~rot], ref2[~rot]), seed
            if g:
                g, o, r64, m64 = (np.concatenate(x, axis=1) for x in (g, o, r64, m64))
                check_rotated_keys(g, r64, m64, o, min_equal=0.995 if g.size >= 8192 else 0.9)
    finally:
        dev.close()
