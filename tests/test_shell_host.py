"""The storage-module shell's host side, on CPU: key hash against the oracle, header round trip and rejection, index
semantics (least-recently-used eviction under a byte budget)."""
import ctypes as C

import numpy as np

import oracle
from paper_2409_13761_b200 import kdn as K


def test_key_hash_matches_the_oracle():
    rng = np.random.default_rng(3)
    for n in (0, 1, 7, 4096):
        toks = rng.integers(-2 ** 31, 2 ** 31 - 1, n).astype(np.int32)
        assert K.kdn_key_hash(toks.tolist()) == oracle.key_hash(toks)
    assert K.kdn_key_hash([]) == 0xcbf29ce484222325


def test_header_round_trip_and_rejections():
    d = K.pool_desc(32, 8, 128, 16, 16384)
    ch = K.Chunk(0x1000, K.kdn_chunk_bytes(d, 512, K.KDN_CODEC_INT8_G64), 512, K.KDN_CODEC_INT8_G64, 0, 77)
    h = K.kdn_header_fill(d, ch, key=0xABCDEF, checksum=0x1234)
    assert C.sizeof(h) == 128 and h.magic == b"KDNCHNK1" and h.header_bytes == 128
    assert (h.n_layers, h.n_kv_heads, h.head_dim, h.n_tokens, h.base_pos, h.payload_bytes, h.key) == (32, 8, 128, 512, 77, ch.bytes, 0xABCDEF)
    st, back = K.kdn_header_check(d, h, 0x1234)
    assert st == K.KDN_OK and (back.bytes, back.n_tokens, back.codec, back.base_pos) == (ch.bytes, 512, 1, 77)
    assert K.kdn_header_check(d, h, 0x1235)[0] == K.KDN_E_CHECKSUM                  # damaged payload
    assert K.kdn_header_check(K.pool_desc(80, 8, 128, 16, 16384), h, 0x1234)[0] == K.KDN_E_SHAPE   # another model
    bad = K.kdn_chunk_header.from_buffer_copy(bytes(h)); bad.magic = b"NOTKDN!!"
    assert K.kdn_header_check(d, bad, 0x1234)[0] == K.KDN_E_INVAL
    bad = K.kdn_chunk_header.from_buffer_copy(bytes(h)); bad.payload_bytes += 4
    assert K.kdn_header_check(d, bad, 0x1234)[0] == K.KDN_E_SHAPE
    bad = K.kdn_chunk_header.from_buffer_copy(bytes(h)); bad.codec = 9
    assert K.kdn_header_check(d, bad, 0x1234)[0] == K.KDN_E_SHAPE
    wrong = K.Chunk(0x1000, ch.bytes - 8, 512, K.KDN_CODEC_INT8_G64)
    try:
        K.kdn_header_fill(d, wrong, 1, 2)
        assert False
    except K.KdnError as e:
        assert e.status == K.KDN_E_SHAPE


def chunk(i, nbytes):
    return K.Chunk(0x100000 * (i + 1), nbytes, 16, 0, 0, i)


def test_index_lru_eviction_under_a_byte_budget():
    idx = K.kdn_index_create(1000)
    try:
        assert K.kdn_index_get(idx, 1)[0] == K.KDN_E_NOTFOUND
        for i in range(4):                                       # 4 x 250 bytes fill the budget exactly
            st, ev = K.kdn_index_put(idx, 10 + i, chunk(i, 250))
            assert st == K.KDN_OK and ev == []
        st, c = K.kdn_index_get(idx, 10)                          # touch the oldest: 11 is now least recently used
        assert st == K.KDN_OK and c.data == 0x100000 and c.base_pos == 0
        st, ev = K.kdn_index_put(idx, 20, chunk(7, 300))          # needs 300 bytes: evicts 11 and 12
        assert st == K.KDN_OK and [e.base_pos for e in ev] == [1, 2]
        assert K.kdn_index_get(idx, 11)[0] == K.KDN_E_NOTFOUND and K.kdn_index_get(idx, 10)[0] == K.KDN_OK
        info = K.kdn_index_stats(idx)
        assert (info.capacity_bytes, info.bytes, info.entries, info.evictions) == (1000, 800, 3, 2)
        assert info.hits == 2 and info.misses == 2
        # replacing a key hands the old descriptor back first and counts its bytes as freed
        st, ev = K.kdn_index_put(idx, 20, chunk(8, 450))
        assert st == K.KDN_OK and [e.base_pos for e in ev] == [7] and K.kdn_index_stats(idx).bytes == 950
        # too large for the budget, or more victims than the caller accepts: nothing changes
        assert K.kdn_index_put(idx, 30, chunk(9, 1001))[0] == K.KDN_E_NOMEM
        assert K.kdn_index_put(idx, 30, chunk(9, 900), max_evicted=1)[0] == K.KDN_E_NOMEM
        assert K.kdn_index_stats(idx).entries == 3 and K.kdn_index_stats(idx).bytes == 950
        st, c = K.kdn_index_remove(idx, 13)
        assert st == K.KDN_OK and c.base_pos == 3 and K.kdn_index_remove(idx, 13)[0] == K.KDN_E_NOTFOUND
        st, ev = K.kdn_index_put(idx, 30, chunk(9, 900))          # evicts everything else, least recent first
        assert st == K.KDN_OK and [e.base_pos for e in ev] == [0, 8]
        assert K.kdn_index_stats(idx).entries == 1
    finally:
        K.kdn_index_destroy(idx)
    assert K.lib.kdn_index_get(None, 1, None) == K.KDN_E_INVAL
