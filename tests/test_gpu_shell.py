"""GPU side of the storage-module shell: the payload checksum kernel against the oracle, and one trip of a chunk through
store -> checksum -> header -> index -> lookup by text -> verify -> retrieve."""
import ctypes as C

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np

pytestmark = pytest.mark.gpu


def gpu_checksum(K, t: torch.Tensor, stream) -> int:
    out = torch.zeros(1, dtype=torch.int64, device=t.device)
    K.kdn_checksum(0, t.data_ptr(), t.numel(), out.data_ptr(), stream.cuda_stream)
    torch.cuda.synchronize()
    return int(out.item()) & ((1 << 64) - 1)


def test_checksum_matches_the_oracle_at_many_sizes_and_alignments():
    from paper_2409_13761_b200 import kdn as K
    dev = torch.device("cuda:0")
    stream = torch.cuda.Stream()
    g = torch.Generator(device="cpu").manual_seed(5)
    big = torch.randint(0, 256, ((64 << 20) + 64,), dtype=torch.uint8, generator=g)
    dbig = big.to(dev)
    host = big.numpy()
    for off, n in [(0, 0), (0, 4), (0, 12), (0, 16), (0, 4096), (0, 4100), (16, 1 << 20), (4, 1 << 20), (8, (1 << 20) + 12),
                   (0, 64 << 20), (32, (64 << 20) - 4)]:
        assert gpu_checksum(K, dbig[off:off + n], stream) == oracle.checksum(host[off:off + n]), (off, n)
    zeros = torch.zeros(1 << 16, dtype=torch.uint8, device=dev)
    assert gpu_checksum(K, zeros, stream) == oracle.checksum(np.zeros(1 << 16, dtype=np.uint8))
    assert K.lib.kdn_checksum(0, C.c_void_p(dbig.data_ptr() + 1), 8, C.c_void_p(zeros.data_ptr()), None) == K.KDN_E_ALIGN
    assert K.lib.kdn_checksum(0, C.c_void_p(dbig.data_ptr()), 6, C.c_void_p(zeros.data_ptr()), None) == K.KDN_E_ALIGN


def test_a_chunk_through_the_shell():
    shape = synth.TOY.with_(n_layers=4, n_kv_heads=4, head_dim=128, block_size=16, n_blocks=64)
    dev = Device(shape, seed=61)
    try:
        K = dev.K
        host = dev.pool_np()
        text = list(range(1000, 1000 + 90))                            # the text's token ids
        key = K.kdn_key_hash(text)
        assert key == oracle.key_hash(text)
        tab = np.random.default_rng(1).permutation(64)[:6].astype(np.int32)
        codec = oracle.INT8_G64
        buf = dev.chunk_buf(90, codec)
        dev.store([dev.op(dev.table(tab), 2, buf, 90, codec)])
        assert dev.sync() == 0
        want = oracle.store(host, tab, 2, 90, codec)
        csum = gpu_checksum(K, buf, dev.stream)
        assert csum == oracle.checksum(want)
        ch = dev.chunk(buf, 90, codec, base_pos=2)
        header = K.kdn_header_fill(dev.desc, ch, key, csum)
        idx = K.kdn_index_create(10 * buf.numel())
        try:
            assert K.kdn_index_put(idx, key, ch)[0] == K.KDN_OK
            assert K.kdn_index_get(idx, K.kdn_key_hash(text[:-1]))[0] == K.KDN_E_NOTFOUND      # another text
            st, found = K.kdn_index_get(idx, K.kdn_key_hash(list(text)))
            assert st == K.KDN_OK and found.data == buf.data_ptr() and found.bytes == buf.numel()
            # verify before use, then deliver into other blocks
            st, desc_chunk = K.kdn_header_check(dev.desc, header, gpu_checksum(K, buf, dev.stream))
            assert st == K.KDN_OK and desc_chunk.n_tokens == 90 and desc_chunk.base_pos == 2
            dst = np.setdiff1d(np.arange(64), tab)[:6].astype(np.int32)
            dev.retrieve([dev.K.XferOp(dev.table(dst).data_ptr(), 6, 2, found)])
            assert dev.sync() == 0
            ref = host.copy()
            oracle.retrieve(ref, dst, 2, 90, codec, want)
            assert np.array_equal(dev.pool_np(), ref)
            # a flipped payload byte is caught
            buf[12345] ^= 0x40
            assert K.kdn_header_check(dev.desc, header, gpu_checksum(K, buf, dev.stream))[0] == K.KDN_E_CHECKSUM
        finally:
            K.kdn_index_destroy(idx)
    finally:
        dev.close()
