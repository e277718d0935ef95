"""kdn_compose_static: the compose entry point for callers that cannot allocate device memory.

Some users of this library run where cudaMalloc is not available to them: an engine whose own allocator
already owns the whole GPU, a thread that works while another captures a CUDA graph in global mode, a
loop that cannot afford the device-wide synchronisation an allocation may bring.  They cannot create a
context (that allocates), so they call kdn_compose_static, which keeps its scratch in a fixed array inside
the library.  These tests drive that call through the C ABI: twice in a row with different requests, where
the pool it leaves behind must be bit-identical to what kdn_compose (the context-based call) leaves from the
same inputs and must agree with the CPU oracle; with the free device memory read before and after, which
must not move; with more parts than travel as kernel parameters; with a bad block id and with sizes beyond
the limits; and as the very first CUDA work of a fresh process, before any context exists.
The file is collected last so that a failure here cannot hide the result of any other test.
"""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, check_rotated_keys

pytestmark = pytest.mark.gpu

RAW, INT8 = oracle.RAW_BF16, oracle.INT8_G64
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def restore(dev, host):
    for l in range(dev.shape.n_layers):
        dev.k[l].copy_(torch.from_numpy(host[l, 0].view(np.int16)).view(torch.bfloat16))
        dev.v[l].copy_(torch.from_numpy(host[l, 1].view(np.int16)).view(torch.bfloat16))
    torch.cuda.synchronize()


def gather(pool, table, positions, bs):
    """[L][2][len(positions)][H][D] bit patterns of the request positions."""
    p = np.asarray(positions)
    return pool[:, :, np.asarray(table)[p // bs], p % bs]


def test_static_compose_matches_context_compose_and_the_oracle_on_two_calls_in_a_row():
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
        och = [oracle.store(host, tab, off, T, codec) for tab, off, T, codec in specs]
        tab1, tab2 = perm[20:32], perm[40:50]
        t1, t2 = dev.table(tab1), dev.table(tab2)
        # call 1: three parts, two re-rotated (one by a large negative shift); call 2: other parts, other
        # shifts, other blocks -- stale records or a stale rotation table from call 1 would show here
        calls = [
            [K.ComposeReq(t1.data_ptr(), 12, [dev.chunk(bufs[0], 70, RAW, 0), dev.chunk(bufs[1], 64, INT8, 100000),
                                              dev.chunk(bufs[2], 40, RAW, 150)], [0, 75, 150], shape.rope_theta)],
            [K.ComposeReq(t2.data_ptr(), 10, [dev.chunk(bufs[1], 64, INT8, 0), dev.chunk(bufs[2], 40, RAW, 7)],
                          [9, 100], shape.rope_theta),
             K.ComposeReq(t1.data_ptr(), 12, [dev.chunk(bufs[0], 70, RAW, 17)], [101], 10000.0)],
        ]
        # the same requests as the oracle takes them: (table, [(chunk, T, codec, base_pos, dst_pos)], theta)
        oracle_calls = [
            [(tab1, [(och[0], 70, RAW, 0, 0), (och[1], 64, INT8, 100000, 75), (och[2], 40, RAW, 150, 150)], shape.rope_theta)],
            [(tab2, [(och[1], 64, INT8, 0, 9), (och[2], 40, RAW, 7, 100)], shape.rope_theta),
             (tab1, [(och[0], 70, RAW, 17, 101)], 10000.0)],
        ]
        want = []
        for reqs in calls:                                   # the existing entry point, one call after the other
            dev.compose(reqs)
            assert dev.sync() == 0
            want.append(dev.pool_np())
        restore(dev, host)
        before = host
        for reqs, oreqs, w in zip(calls, oracle_calls, want):    # the new entry point, same sequence, same inputs
            st = K.kdn_compose_static(0, dev.desc, reqs, dev.stream.cuda_stream, wait=True)
            assert st == K.KDN_OK, K.kdn_strerror(st)
            got = dev.pool_np()
            assert np.array_equal(got, w)                    # same kernels, same arithmetic: bit-identical
            ref = before.copy()                              # and right by the oracle, request by request
            rot = np.zeros(got.shape, dtype=bool)
            for table, parts, theta in oreqs:
                kref, kmag = oracle.compose(ref, np.asarray(table, dtype=np.int32), parts, theta, want_ref=True)
                for _, T, _, base, dst in parts:
                    if base != dst:
                        p = dst + np.arange(T)
                        rot[:, 0, table[p // 16], p % 16] = True
                        check_rotated_keys(gather(got, table, p, 16)[:, 0], kref[:, dst:dst + T], kmag[:, dst:dst + T],
                                           gather(ref, table, p, 16)[:, 0])
            assert np.array_equal(got[~rot], ref[~rot])      # everything that is not a re-rotated key: exact
            ref[rot] = got[rot]                              # rotated keys are within tolerance: carry the device's bits on
            before = ref
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
        # a pool with more layers, or a wider head, than the fixed array has room for
        ptrs = [dev.k[0].data_ptr()] * 129
        deep = K.pool_desc(129, shape.n_kv_heads, shape.head_dim, shape.block_size, shape.n_blocks, ptrs, ptrs)
        one = [K.ComposeReq(t1.data_ptr(), 12, [K.Chunk(bufs[0].data_ptr(), K.kdn_chunk_bytes(deep, 1, RAW), 1, RAW)], [0], 1e4)]
        assert K.kdn_compose_static(0, deep, one, dev.stream.cuda_stream, wait=True) == K.KDN_E_UNSUPPORTED
        wide = K.pool_desc(1, 1, 576, 16, 8, ptrs[:1], ptrs[:1])
        one = [K.ComposeReq(t1.data_ptr(), 12, [K.Chunk(bufs[0].data_ptr(), K.kdn_chunk_bytes(wide, 1, RAW), 1, RAW)], [0], 1e4)]
        assert K.kdn_compose_static(0, wide, one, dev.stream.cuda_stream, wait=True) == K.KDN_E_UNSUPPORTED
    finally:
        dev.close()


def test_static_compose_leaves_free_device_memory_unchanged_and_takes_up_to_128_parts():
    """The property the call exists for: it allocates nothing.  After one warm call, the device's free memory
    (cudaMemGetInfo) is read around calls that cover raw, int8 and re-rotated parts, and around a call of 100 parts
    (more than travel as kernel parameters); it must not move.  The 100-part call must also leave the pool
    bit-identical to kdn_compose."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=256, rope_theta=10000.0)
    dev = Device(shape, seed=52)
    try:
        K = dev.K
        perm = np.random.default_rng(16).permutation(shape.n_blocks).astype(np.int32)
        raw, i8 = dev.chunk_buf(48, RAW), dev.chunk_buf(48, INT8)
        dev.store([dev.op(dev.table(perm[:3]), 0, raw, 48, RAW), dev.op(dev.table(perm[3:6]), 0, i8, 48, INT8)])
        assert dev.sync() == 0
        host = dev.pool_np()
        n_many = 100
        tab = dev.table(perm[10:10 + 150])
        small = [K.ComposeReq(tab.data_ptr(), 150, [dev.chunk(raw, 48, RAW, 0), dev.chunk(i8, 48, INT8, 0), dev.chunk(raw, 48, RAW, 5)],
                              [0, 48, 96], shape.rope_theta)]
        cb1 = K.kdn_chunk_bytes(dev.desc, 16, RAW)
        # 100 parts of 16 tokens cut out of... one stored 16-token chunk per codec, placed at 100 different positions
        r16, q16 = dev.chunk_buf(16, RAW), dev.chunk_buf(16, INT8)
        dev.store([dev.op(dev.table(perm[:1]), 0, r16, 16, RAW), dev.op(dev.table(perm[1:2]), 0, q16, 16, INT8)])
        assert dev.sync() == 0
        parts = [dev.chunk(r16 if j % 2 == 0 else q16, 16, RAW if j % 2 == 0 else INT8, 0 if j % 3 else 16 * j) for j in range(n_many)]
        many = [K.ComposeReq(tab.data_ptr(), 150, parts, [16 * j for j in range(n_many)], shape.rope_theta)]
        assert cb1 == r16.numel()
        dev.compose(many)
        assert dev.sync() == 0
        want_many = dev.pool_np()
        restore(dev, host)
        s = dev.stream.cuda_stream
        assert K.kdn_compose_static(0, dev.desc, small, s, wait=True) == K.KDN_OK      # warm: one-time set-up happens here
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        assert K.kdn_compose_static(0, dev.desc, small, s, wait=True) == K.KDN_OK
        free1, _ = torch.cuda.mem_get_info()
        assert K.kdn_compose_static(0, dev.desc, many, s, wait=False) == K.KDN_OK
        assert K.kdn_compose_static(0, dev.desc, many, s, wait=True) == K.KDN_OK
        free2, _ = torch.cuda.mem_get_info()
        assert free0 == free1 == free2, (free0, free1, free2)
        assert np.array_equal(dev.pool_np(), want_many)
    finally:
        dev.close()


CHILD = r"""
import sys
sys.path.insert(0, %r)
import numpy as np, torch
from paper_2409_13761_b200 import kdn as K
# no context is ever created in this process: the static call is the first thing the library does here
L, H, D, bs, nb, T = 2, 2, 64, 16, 32, 40
dev = torch.device("cuda:0")
g = torch.Generator(device="cpu").manual_seed(3)
k = [torch.randn(nb, bs, H, D, generator=g).to(torch.bfloat16).to(dev) for _ in range(L)]
v = [torch.randn(nb, bs, H, D, generator=g).to(torch.bfloat16).to(dev) for _ in range(L)]
desc = K.pool_desc(L, H, D, bs, nb, [t.data_ptr() for t in k], [t.data_ptr() for t in v])
chunk = torch.randn(L, 2, T, H, D, generator=g).to(torch.bfloat16).to(dev)
table = torch.tensor([7, 3, 30], dtype=torch.int32, device=dev)
torch.cuda.synchronize()
free0, _ = torch.cuda.mem_get_info()
st = K.kdn_compose_static(0, desc, [K.ComposeReq(table.data_ptr(), 3, [K.Chunk(chunk.data_ptr(), chunk.numel() * 2, T, 0)], [5], 1e4)], 0, True)
assert st == K.KDN_OK, st
free1, _ = torch.cuda.mem_get_info()
st = K.kdn_compose_static(0, desc, [K.ComposeReq(table.data_ptr(), 3, [K.Chunk(chunk.data_ptr(), chunk.numel() * 2, T, 0, 0, 9)], [5], 1e4)], 0, True)
assert st == K.KDN_OK, st
free2, _ = torch.cuda.mem_get_info()
# a part placed where its keys were computed (base_pos = dst_pos = 5): a plain scatter, checked here by hand
# (position p -> block table[p // bs], slot p %% bs)
st = K.kdn_compose_static(0, desc, [K.ComposeReq(table.data_ptr(), 3, [K.Chunk(chunk.data_ptr(), chunk.numel() * 2, T, 0, 0, 5)], [5], 1e4)], 0, True)
assert st == K.KDN_OK, st
tab = [7, 3, 30]
for l in range(L):
    for kv, pool in ((0, k), (1, v)):
        for t in range(T):
            p = 5 + t
            assert torch.equal(pool[l][tab[p // bs], p %% bs], chunk[l, kv, t]), (l, kv, t)
# the first call may load code (its one-time set-up); the calls after it must not move the free memory at all
assert free1 == free2, (free0, free1, free2)
print("child ok", free0 - free1)
"""


def test_static_compose_as_the_first_cuda_work_of_a_fresh_process():
    """An engine that cannot allocate never creates a context, so the call has to work with nothing set up before
    it: a child process makes it the library's first call, checks the scatter by hand, and checks that from the
    second call on the device's free memory does not move."""
    out = subprocess.run([sys.executable, "-c", CHILD % ROOT], capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stdout + out.stderr
    assert "child ok" in out.stdout
