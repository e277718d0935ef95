"""kdn_compose_static: the compose entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not available to them: an engine whose own allocator
already owns the whole GPU, a thread that works while another captures a CUDA graph in global mode, a
loop that cannot afford the device-wide synchronisation an allocation may bring.  They cannot create a
context (that allocates), so they call kdn_compose_static, which keeps its scratch in a fixed array inside
the library.  This test drives that call through the C ABI twice in a row, with different requests, and
requires the pool it leaves behind to be bit-identical to what kdn_compose (the context-based call) leaves
from the same inputs; a third call checks that a bad block id is reported, and that size limits are refused.
It is collected last so that a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device

pytestmark = pytest.mark.gpu

RAW, INT8 = oracle.RAW_BF16, oracle.INT8_G64


def restore(dev, host):
    for l in range(dev.shape.n_layers):
        dev.k[l].copy_(torch.from_numpy(host[l, 0].view(np.int16)).view(torch.bfloat16))
        dev.v[l].copy_(torch.from_numpy(host[l, 1].view(np.int16)).view(torch.bfloat16))
    torch.cuda.synchronize()


def test_static_compose_matches_context_compose_on_two_calls_in_a_row():
    shape = synth.TOY.with_(n_layers=3, n_kv_heads=4, head_dim=128, block_size=16, n_blocks=96, rope_theta=500000.0)
    dev = Device(shape, seed=51)
    try:
        K = dev.K
        rng = np.random.default_rng(15)
        perm = rng.permutation(shape.n_blocks).astype(np.int32)
        # three stored chunks (made with the ordinary store call): raw, int8, raw
        specs = [(perm[0:5], 3, 70, RAW), (perm[5:9], 0, 64, INT8), (perm[9:12], 5, 40, RAW)]
        bufs = []
        for tab, off, T, codec in specs:
            b = dev.chunk_buf(T, codec)
            dev.store([dev.op(dev.table(tab), off, b, T, codec)])
            bufs.append(b)
        assert dev.sync() == 0
        host = dev.pool_np()
        t1, t2 = dev.table(perm[20:32]), dev.table(perm[40:50])
        # call 1: three parts, two re-rotated (one by a large negative shift); call 2: other parts, other
        # shifts, other blocks -- stale records or a stale rotation table from call 1 would show here
        calls = [
            [K.ComposeReq(t1.data_ptr(), 12, [dev.chunk(bufs[0], 70, RAW, 0), dev.chunk(bufs[1], 64, INT8, 100000),
                                              dev.chunk(bufs[2], 40, RAW, 150)], [0, 75, 150], shape.rope_theta)],
            [K.ComposeReq(t2.data_ptr(), 10, [dev.chunk(bufs[1], 64, INT8, 0), dev.chunk(bufs[2], 40, RAW, 7)],
                          [9, 100], shape.rope_theta),
             K.ComposeReq(t1.data_ptr(), 12, [dev.chunk(bufs[0], 70, RAW, 17)], [101], 10000.0)],
        ]
        want = []
        for reqs in calls:                                   # the existing entry point, one call after the other
            dev.compose(reqs)
            assert dev.sync() == 0
            want.append(dev.pool_np())
        restore(dev, host)
        for reqs, w in zip(calls, want):                     # the new entry point, same sequence, same inputs
            st = K.kdn_compose_static(0, dev.desc, reqs, dev.stream.cuda_stream, wait=True)
            assert st == K.KDN_OK, K.kdn_strerror(st)
            assert np.array_equal(dev.pool_np(), w)          # same kernels, same arithmetic: bit-identical
        # fire-and-forget form followed by a waiting call on the same stream
        restore(dev, host)
        assert K.kdn_compose_static(0, dev.desc, calls[0], dev.stream.cuda_stream, wait=False) == K.KDN_OK
        assert K.kdn_compose_static(0, dev.desc, calls[1], dev.stream.cuda_stream, wait=True) == K.KDN_OK
        assert np.array_equal(dev.pool_np(), want[1])
        # a block id outside the pool: reported by the waiting call, nothing faults, and the next call is clean
        bad = dev.table(np.array([perm[60], shape.n_blocks + 5, perm[61]], dtype=np.int32))
        st = K.kdn_compose_static(0, dev.desc, [K.ComposeReq(bad.data_ptr(), 3, [dev.chunk(bufs[2], 40, RAW, 0)], [0], 1e4)],
                                  dev.stream.cuda_stream, wait=True)
        assert st == K.KDN_E_RANGE
        assert K.kdn_compose_static(0, dev.desc, calls[1], dev.stream.cuda_stream, wait=True) == K.KDN_OK
        # limits and unsupported forms are refused before anything is enqueued
        many = [dev.chunk(bufs[2][: K.kdn_chunk_bytes(dev.desc, 1, RAW)], 1, RAW, 0)] * 129
        big = dev.table(np.arange(9, dtype=np.int32))
        st = K.kdn_compose_static(0, dev.desc, [K.ComposeReq(big.data_ptr(), 9, many, list(range(129)), 1e4)],
                                  dev.stream.cuda_stream, wait=True)
        assert st == K.KDN_E_UNSUPPORTED
        hb = dev.chunk_buf(40, RAW, pinned=True)
        st = K.kdn_compose_static(0, dev.desc, [K.ComposeReq(t1.data_ptr(), 12, [dev.chunk(hb, 40, RAW, 0)], [0], 1e4)],
                                  dev.stream.cuda_stream, wait=True)
        assert st == K.KDN_E_UNSUPPORTED
        assert K.kdn_compose_static(99, dev.desc, calls[0], dev.stream.cuda_stream, wait=True) == K.KDN_E_CUDA
    finally:
        dev.close()
