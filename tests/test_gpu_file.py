"""GPU parity for file-backed chunks: kdn_store_file / kdn_retrieve_file against the CPU oracle, through the C ABI."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np

pytestmark = pytest.mark.gpu
RAW, INT8, INT4 = oracle.RAW_BF16, oracle.INT8_G64, oracle.INT4_G64


@pytest.mark.parametrize("codec", [RAW, INT8, INT4])
def test_store_to_file_and_retrieve_from_file(tmp_path, codec):
    """Two chunks go to one file (at offsets that are not multiples of anything) through small staging slabs, so every
    chunk crosses in several layer ranges; the file must hold the oracle's chunks byte for byte, and retrieving them
    from the file into other blocks must equal the oracle's retrieve."""
    shape = synth.TOY.with_(n_layers=5, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=96)
    dev = Device(shape, seed=21)
    try:
        K = dev.K
        K.kdn_set_staging_bytes(dev.ctx, 96 * 1024)                       # a 100-token raw layer is 50 KiB: one or two per slab
        host = dev.pool_np()
        perm = np.random.default_rng(3).permutation(shape.n_blocks).astype(np.int32)
        cases = [(perm[0:8], 5, 100), (perm[8:14], 0, 77)]               # (source table, offset, tokens)
        dsts = [perm[20:28], perm[30:36]]
        path = tmp_path / "chunks.bin"
        fd = os.open(path, os.O_RDWR | os.O_CREAT, 0o600)
        try:
            offs, ops, want = [], [], []
            pos = 7
            for tab, off, T in cases:
                nbytes = K.kdn_chunk_bytes(dev.desc, T, codec)
                ops.append(K.XferOp(dev.table(tab).data_ptr(), len(tab), off, K.Chunk(0, nbytes, T, codec)))
                offs.append(pos)
                want.append(oracle.store(host, tab, off, T, codec))
                pos += nbytes + 13
            K.kdn_store_file(dev.ctx, dev.pool_id, ops, [fd] * len(ops), offs, dev.stream.cuda_stream)
            assert dev.sync() == 0
            assert os.fstat(fd).st_size == pos - 13
            data = np.fromfile(path, dtype=np.uint8)
            for o, w in zip(offs, want):
                assert np.array_equal(data[o:o + len(w)], w)
            assert not data[:7].any()                                     # the gaps were never written
            rops = [K.XferOp(dev.table(d).data_ptr(), len(d), off, K.Chunk(0, len(w), T, codec))
                    for d, (tab, off, T), w in zip(dsts, cases, want)]
            K.kdn_retrieve_file(dev.ctx, dev.pool_id, rops, [fd] * len(rops), offs, dev.stream.cuda_stream)
            assert dev.sync() == 0
            ref = host.copy()
            for d, (tab, off, T), w in zip(dsts, cases, want):
                oracle.retrieve(ref, d, off, T, codec, w)
            assert np.array_equal(dev.pool_np(), ref)
        finally:
            os.close(fd)
    finally:
        dev.close()


def test_file_errors_are_reported():
    shape = synth.TOY.with_(n_blocks=32)
    dev = Device(shape, seed=22)
    try:
        K = dev.K
        tab = dev.table(np.arange(4, dtype=np.int32))
        nbytes = K.kdn_chunk_bytes(dev.desc, 40, RAW)
        op = K.XferOp(tab.data_ptr(), 4, 0, K.Chunk(0, nbytes, 40, RAW))
        with pytest.raises(K.KdnError) as e:
            K.kdn_retrieve_file(dev.ctx, dev.pool_id, [op], [-1], [0], dev.stream.cuda_stream)
        assert e.value.status == K.KDN_E_INVAL
        r, w = os.pipe()                                                  # pread on a pipe fails
        try:
            with pytest.raises(K.KdnError) as e:
                K.kdn_retrieve_file(dev.ctx, dev.pool_id, [op], [r], [0], dev.stream.cuda_stream)
            assert e.value.status == K.KDN_E_IO
        finally:
            os.close(r)
            os.close(w)
        fd = os.open("/dev/null", os.O_RDONLY)                            # a file that ends before the chunk does
        try:
            with pytest.raises(K.KdnError) as e:
                K.kdn_retrieve_file(dev.ctx, dev.pool_id, [op], [fd], [0], dev.stream.cuda_stream)
            assert e.value.status == K.KDN_E_IO
        finally:
            os.close(fd)
        assert dev.sync() == 0
    finally:
        dev.close()
