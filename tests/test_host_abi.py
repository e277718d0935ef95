"""CPU-only checks of the C-ABI library: it loads, exports what include/kdn.h declares, and its host-side
argument validation and size arithmetic agree with the oracle's. No compute call is made."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2409_13761_b200 import kdn as K

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "kdn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kdn_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = declared_functions()
    assert "kdn_store" in names and "kdn_retrieve" in names and "kdn_compose" in names
    for n in names:
        assert hasattr(K.lib, n), n
    assert sorted(names) == sorted(K.EXPORTS)


def test_chunk_bytes_matches_oracle():
    for (L, H, D) in [(2, 2, 64), (32, 8, 128), (80, 8, 128), (1, 3, 8), (4, 1, 192), (2, 2, 96)]:
        d = K.pool_desc(L, H, D, 16, 64)
        for T in (0, 1, 17, 512, 2048):
            for codec in (0, 1, 2, 3, 4, 5, 6):
                assert K.kdn_chunk_bytes(d, T, codec) == oracle.chunk_bytes(L, H, D, T, codec), (L, H, D, T, codec)
    d = K.pool_desc(2, 2, 64, 16, 64)
    assert K.kdn_chunk_bytes(d, -1, 0) == 0
    assert K.kdn_chunk_bytes(d, 4, 7) == 0


def test_strerror_is_total():
    seen = {K.kdn_strerror(s) for s in range(12)}
    assert len(seen) == 12 and "unknown status" not in seen
    assert K.kdn_strerror(99) == "unknown status"


def good_op(desc, T=20, off=3, n_table=2, codec=0, data=0x10000, table=0x20000):
    return K.XferOp(table, n_table, off, K.Chunk(data, K.kdn_chunk_bytes(desc, T, codec), T, codec))


def test_validate_xfer_status_codes():
    d = K.pool_desc(2, 2, 64, 16, 64)
    assert K.kdn_validate_xfer(d, [good_op(d)]) == K.KDN_OK
    assert K.kdn_validate_xfer(d, []) == K.KDN_OK
    assert K.kdn_validate_xfer(d, [good_op(d, T=30, off=3)]) == K.KDN_E_RANGE        # 33 > 32 slots
    assert K.kdn_validate_xfer(d, [good_op(d, T=29, off=3)]) == K.KDN_OK
    assert K.kdn_validate_xfer(d, [good_op(d, off=-1)]) == K.KDN_E_INVAL
    assert K.kdn_validate_xfer(d, [good_op(d, data=0x10008)]) == K.KDN_E_ALIGN
    assert K.kdn_validate_xfer(d, [good_op(d, data=0)]) == K.KDN_E_INVAL
    assert K.kdn_validate_xfer(d, [good_op(d, table=0)]) == K.KDN_E_INVAL
    assert K.kdn_validate_xfer(d, [good_op(d, codec=7)]) == K.KDN_E_INVAL
    op = good_op(d)
    op.chunk.bytes += 2
    assert K.kdn_validate_xfer(d, [op]) == K.KDN_E_SHAPE
    op = good_op(d)
    op.chunk.mem = 3
    assert K.kdn_validate_xfer(d, [op]) == K.KDN_E_INVAL
    op = good_op(d, T=0)
    op.chunk.data = 0                                                                # empty chunk needs no buffer
    assert K.kdn_validate_xfer(d, [op]) == K.KDN_OK
    assert K.kdn_validate_xfer(d, [good_op(d), good_op(d, data=0x10004)]) == K.KDN_E_ALIGN   # any op of a batch
    d96 = K.pool_desc(2, 2, 96, 16, 64)
    op = K.XferOp(0x20000, 2, 0, K.Chunk(0x10000, 0, 4, 1))
    assert K.kdn_validate_xfer(d96, [op]) == K.KDN_E_UNSUPPORTED                      # int8 needs head_dim % 64 == 0
    assert K.kdn_validate_xfer(K.pool_desc(2, 1, 4, 16, 64), [good_op(d)]) == K.KDN_E_ALIGN   # row of 8 bytes
    assert K.kdn_validate_xfer(K.pool_desc(0, 2, 64, 16, 64), []) == K.KDN_E_INVAL


def test_validate_per_channel_key_codecs():
    d = K.pool_desc(2, 2, 64, 16, 64)
    for codec in (K.KDN_CODEC_INT8_KC64, K.KDN_CODEC_INT4_KC64, K.KDN_CODEC_INT8_TD64, K.KDN_CODEC_INT4_TD64):
        assert K.kdn_validate_xfer(d, [good_op(d, T=20, off=0, codec=codec)]) == K.KDN_OK
        assert K.kdn_validate_xfer(d, [good_op(d, T=10, off=16, codec=codec)]) == K.KDN_OK
        assert K.kdn_validate_xfer(d, [good_op(d, T=20, off=3, codec=codec)]) == K.KDN_E_UNSUPPORTED     # not at a block start
        assert K.kdn_validate_xfer(d, [good_op(d, T=0, off=3, n_table=1, codec=codec)]) == K.KDN_OK      # nothing to move
    d3 = K.pool_desc(2, 2, 64, 3, 64)                                                                     # 3 does not divide 64
    assert K.kdn_validate_xfer(d3, [good_op(d3, T=5, off=0, n_table=2, codec=K.KDN_CODEC_INT8_KC64)]) == K.KDN_E_UNSUPPORTED
    d96 = K.pool_desc(2, 2, 96, 16, 64)                                                                   # head_dim % 64 != 0
    assert K.kdn_chunk_bytes(d96, 4, K.KDN_CODEC_INT4_KC64) == 0


def test_validate_compose_status_codes():
    d = K.pool_desc(2, 2, 64, 16, 64)

    def part(T=16, codec=0, base=0, data=0x10000):
        return K.Chunk(data, K.kdn_chunk_bytes(d, T, codec), T, codec, 0, base)

    ok = K.ComposeReq(0x20000, 4, [part(), part(T=20)], [0, 16], 10000.0)
    assert K.kdn_validate_compose(d, [ok]) == K.KDN_OK
    assert K.kdn_validate_compose(d, [K.ComposeReq(0x20000, 4, [part(), part()], [0, 15], 1e4)]) == K.KDN_E_RANGE  # overlap
    assert K.kdn_validate_compose(d, [K.ComposeReq(0x20000, 4, [part(T=20)], [48], 1e4)]) == K.KDN_E_RANGE        # past table
    assert K.kdn_validate_compose(d, [K.ComposeReq(0x20000, 4, [part()], [16], 0.0)]) == K.KDN_E_INVAL            # theta
    assert K.kdn_validate_compose(d, [K.ComposeReq(0x20000, 4, [part(base=16)], [16], 0.0)]) == K.KDN_OK          # no rotation, theta unused
    assert K.kdn_validate_compose(d, [K.ComposeReq(0x20000, 4, [part()], [0], 1e4, rope_style=1)]) == K.KDN_E_UNSUPPORTED
    d8 = K.pool_desc(1, 3, 8, 4, 8)
    p8 = K.Chunk(0x10000, K.kdn_chunk_bytes(d8, 4, 0), 4, 0, 0, 0)
    assert K.kdn_validate_compose(d8, [K.ComposeReq(0x20000, 4, [p8], [4], 1e4)]) == K.KDN_E_UNSUPPORTED          # head_dim % 16
    assert K.kdn_validate_compose(d8, [K.ComposeReq(0x20000, 4, [p8], [0], 1e4)]) == K.KDN_OK
    assert K.kdn_validate_compose(d, []) == K.KDN_OK


def test_calls_on_a_null_context_are_refused():
    assert K.lib.kdn_store(None, 0, None, 0, None, None) == K.KDN_E_INVAL
    assert K.lib.kdn_retrieve(None, 0, None, 0, None, None) == K.KDN_E_INVAL
    assert K.lib.kdn_compose(None, 0, None, 0, None, None) == K.KDN_E_INVAL
    assert K.lib.kdn_status_sync(None, None) == K.KDN_E_INVAL
    assert K.lib.kdn_set_tuning(None, None) == K.KDN_E_INVAL
    assert K.lib.kdn_launch_count(None) == 0
    K.lib.kdn_destroy(None)
    assert K.lib.kdn_create(None, 0) == K.KDN_E_INVAL


def test_create_without_a_gpu_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(K.KdnError) as e:
        K.kdn_create(0)
    assert e.value.status == K.KDN_E_CUDA
