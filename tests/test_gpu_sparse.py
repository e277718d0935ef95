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
        assert np.array_equal(got[:, :, 0], host[:, :, 3, 0]) and np.array_equal(got[:, :, 1], host[:, :, 3, 5])
        assert np.array_equal(got[:, :, 3], host[:, :, 9, 15]) and np.all(got[:, :, 2] == 0xA5A5)
        with pytest.raises(K.KdnError):                                   # more listed tokens than positions
            K.kdn_store_sparse(dev.ctx, dev.pool_id, [dev.op(dev.table(tab), 30, buf, 4, RAW)], [dev_list(dev, keep).data_ptr()],
                               dev.stream.cuda_stream)
        assert dev.sync() == 0
    finally:
        dev.close()
