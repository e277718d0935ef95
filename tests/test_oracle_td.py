"""Pins for the oracle's token-delta Rice codecs (codecs 5 and 6): the bitstream, the parameter choice, the chunk
layout, and what a retrieve or compose makes of a stored chunk.  CPU only.

The pins: sub-streams worked by hand (tests/golden/td_rice_handworked.txt); a second formulation of the encoder and
of the bit reader that works on strings of '0' and '1' characters; exhaustive code words (every symbol at every
parameter is decodable and costs what rice_bits says, and no code word is a prefix of another); the length bound the
chunk capacity relies on; decode(encode(q)) = q; the quantisation half against the per-channel key codec, which is
pinned on its own; the layout against a by-hand walk through a stored chunk; and what compression it buys on
token-correlated and on uncorrelated inputs."""
import os

import numpy as np
import pytest

import oracle
from paper_2409_13761_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "td_rice_handworked.txt")
TD8, TD4 = oracle.INT8_TD64, oracle.INT4_TD64
QMAX = {TD8: 127, TD4: 7}
RAW_BITS = {127: 9, 7: 5}


def load_golden():
    cases = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, qmax, codes, mode, k, hexbytes = [s.strip() for s in line.split("|")]
            q = []
            for tok in codes.split():
                if "x" in tok:
                    v, n = tok.split("x")
                    q += [int(v)] * int(n)
                else:
                    q.append(int(tok))
            cases.append((name, int(qmax), q, int(mode), int(k), bytes.fromhex(hexbytes.replace(" ", ""))))
    return cases


@pytest.mark.parametrize("case", load_golden(), ids=lambda c: c[0])
def test_handworked_substreams(case):
    _, qmax, q, mode, k, want = case
    data, param = oracle.td_encode_channel(q, qmax)
    assert (param >> 3, param & 7) == (mode, k)
    assert bytes(data) == want
    assert list(oracle.td_decode_channel(data, param, len(q), qmax)) == q


# ------------------------------------------------------------------ a second formulation, on character strings --

def zz(e):
    return 2 * e if e >= 0 else -2 * e - 1


def word(u, k, raw_bits):
    """The code word of symbol u as a string of '0' / '1'."""
    quo = u >> k
    if quo < 15:
        return "1" * quo + "0" + (format(u & ((1 << k) - 1), "0%db" % k) if k else "")
    return "1" * 15 + format(u, "0%db" % raw_bits)


def symbols(q, mode):
    return [zz(int(v) - (int(q[t - 1]) if mode == 1 and t > 0 else 0)) for t, v in enumerate(q)]


def encode_str(q, qmax):
    """(bit string, mode, k): every (mode, k) is written out in full and the shortest string wins, the first such."""
    best = None
    for mode in (0, 1):
        for k in range(8):
            s = "".join(word(u, k, RAW_BITS[qmax]) for u in symbols(q, mode))
            if best is None or len(s) < len(best[0]):
                best = (s, mode, k)
    return best


def to_bytes(bits):
    bits = bits + "0" * (-len(bits) % 8)
    return bytes(int(bits[i:i + 8], 2) for i in range(0, len(bits), 8))


def decode_str(data, mode, k, n, qmax):
    """Read n symbols from a string of bits with string operations only."""
    bits = "".join(format(b, "08b") for b in data) + "0" * 32
    out, prev = [], 0
    for _ in range(n):
        ones = len(bits) - len(bits.lstrip("1"))
        if ones < 15:
            u = (ones << k) | (int(bits[ones + 1:ones + 1 + k], 2) if k else 0)
            bits = bits[ones + 1 + k:]
        else:
            u = int(bits[15:15 + RAW_BITS[qmax]], 2)
            bits = bits[15 + RAW_BITS[qmax]:]
        e = -((u + 1) // 2) if u & 1 else u // 2
        v = prev + e if mode == 1 else e
        out.append(v)
        prev = v
    return out


def test_zigzag_is_the_interleaving_of_signs():
    assert [oracle.zigzag(e) for e in (0, -1, 1, -2, 2, -254, 254)] == [0, 1, 2, 3, 4, 507, 508]
    for e in range(-254, 255):
        assert oracle.unzigzag(oracle.zigzag(e)) == e
    assert sorted(oracle.zigzag(e) for e in range(-254, 255)) == list(range(509))


@pytest.mark.parametrize("qmax", [127, 7])
def test_code_words_are_prefix_free_and_cost_what_rice_bits_says(qmax):
    umax, raw = 4 * qmax, RAW_BITS[qmax]
    assert umax < (1 << raw)
    for k in range(8):
        words = [word(u, k, raw) for u in range(umax + 1)]
        assert len(set(words)) == len(words)
        for u, w in enumerate(words):
            assert oracle.rice_bits(u, k, raw) == len(w)
        srt = sorted(words)
        for a, b in zip(srt, srt[1:]):
            assert not b.startswith(a), (k, a, b)          # a sorted neighbour would be the extension of a prefix


def random_groups(rng, qmax, count):
    """Code sequences of every kind: uniform, narrow, smooth (a random walk), constant, saw-tooth, extremes."""
    out = []
    for i in range(count):
        n = int(rng.integers(1, 65)) if i % 3 else 64
        kind = i % 6
        if kind == 0:
            q = rng.integers(-qmax, qmax + 1, n)
        elif kind == 1:
            q = np.clip(np.rint(rng.standard_normal(n) * qmax / 12), -qmax, qmax)
        elif kind == 2:
            q = np.clip(np.cumsum(rng.integers(-2, 3, n)) + rng.integers(-qmax // 2, qmax // 2 + 1), -qmax, qmax)
        elif kind == 3:
            q = np.full(n, rng.integers(-qmax, qmax + 1))
        elif kind == 4:
            q = np.where(np.arange(n) % 2 == 0, qmax, -qmax)
        else:
            q = rng.choice([-qmax, 0, qmax], n)
        out.append(q.astype(np.int8))
    return out


@pytest.mark.parametrize("qmax", [127, 7])
def test_encoder_equals_the_string_formulation_and_round_trips(qmax):
    rng = np.random.default_rng(100 + qmax)
    longest = 0
    for q in random_groups(rng, qmax, 600):
        data, param = oracle.td_encode_channel(q, qmax)
        bits, mode, k = encode_str(q, qmax)
        assert (param >> 3, param & 7) == (mode, k)
        assert bytes(data) == to_bytes(bits)
        assert len(data) == (len(bits) + 7) // 8
        assert list(oracle.td_decode_channel(data, param, len(q), qmax)) == list(q)
        assert decode_str(bytes(data), mode, k, len(q), qmax) == list(q)
        longest = max(longest, len(data))
    assert longest <= oracle.td_max_len(qmax)


@pytest.mark.parametrize("qmax", [127, 7])
def test_no_substream_is_longer_than_the_capacity_assumes(qmax):
    """Mode 0 with k = 7 (codes to 127) or k = 3 (codes to 7) costs at most 9 or 5 bits a symbol, and the encoder takes
    the shortest candidate: 64 symbols never need more than 72 or 40 bytes.  Checked on the inputs that are worst for
    the small parameters."""
    assert oracle.td_max_len(qmax) == (72 if qmax == 127 else 40)
    k_cap, cap_bits = (7, 9) if qmax == 127 else (3, 5)
    for u in range(2 * qmax + 1):
        assert oracle.rice_bits(u, k_cap, RAW_BITS[qmax]) <= cap_bits
    rng = np.random.default_rng(5)
    worst = [np.where(np.arange(64) % 2 == 0, qmax, -qmax), np.full(64, qmax), np.full(64, -qmax),
             rng.choice([-qmax, qmax], 64), rng.integers(-qmax, qmax + 1, 64)]
    for q in worst:
        data, _ = oracle.td_encode_channel(q.astype(np.int8), qmax)
        assert len(data) <= oracle.td_max_len(qmax)


# ------------------------------------------------------------------------------------------- chunks --

SHAPES = [synth.TOY, synth.TOY.with_(n_layers=1, n_kv_heads=3, head_dim=128, block_size=4, n_blocks=48)]


def walk_chunk(chunk, L, H, D, T, codec):
    """The chunk read by hand from the layout's definition: {(l, kv, g, ch): (scale, codes)} and the used bytes."""
    G, R, S = -(-T // 64), H * D, 2 * L * -(-T // 64)
    a_bytes = (8 * (S + 1) + 15) // 16 * 16
    seg_off = chunk[:8 * (S + 1)].view(np.uint64)
    scales = chunk[a_bytes:a_bytes + 4 * S * R].view(np.float32).reshape(S, R)
    lens = chunk[a_bytes + 4 * S * R:a_bytes + 5 * S * R].reshape(S, R)
    params = chunk[a_bytes + 5 * S * R:a_bytes + 6 * S * R].reshape(S, R)
    assert int(seg_off[0]) == a_bytes + 6 * S * R
    out = {}
    for l in range(L):
        for kv in range(2):
            for g in range(G):
                s = (2 * l + kv) * G + g
                n = min(64, T - 64 * g)
                cur = int(seg_off[s])
                assert cur % 16 == 0
                for ch in range(R):
                    ln = int(lens[s, ch])
                    data = bytes(chunk[cur:cur + ln])
                    out[(l, kv, g, ch)] = (scales[s, ch], decode_str(data, int(params[s, ch]) >> 3, int(params[s, ch]) & 7, n, QMAX[codec]))
                    cur += ln
                end = (cur + 15) // 16 * 16
                assert not chunk[cur:end].any()                  # padding is zero
                assert int(seg_off[s + 1]) == end
    return out, int(seg_off[S])


@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: "H%dD%dbs%d" % (s.n_kv_heads, s.head_dim, s.block_size))
@pytest.mark.parametrize("codec", [TD8, TD4])
@pytest.mark.parametrize("T,off", [(64, 0), (150, 4), (37, 8)])
def test_stored_chunk_layout_and_codes(shape, codec, T, off):
    """Walk a stored chunk by hand: every group's scale and codes equal the per-channel quantiser's (pinned with the
    per-channel key codecs), for keys and for values; segments are 16-byte aligned, zero padded and in order."""
    k, v = synth.make_pool(shape, "cpu", seed=21)
    pool = synth.pool_to_numpy(k, v)
    L, H, D, bs = shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size
    nblk = -(-(off + T) // bs)
    table = np.random.default_rng(3).permutation(shape.n_blocks)[:nblk].astype(np.int32)
    chunk = oracle.store(pool, table, off, T, codec)
    lay = oracle.td_layout(L, H, D, T, codec)
    assert chunk.size == lay["capacity"] == oracle.chunk_bytes(L, H, D, T, codec)
    groups, used = walk_chunk(chunk, L, H, D, T, codec)
    assert used == oracle.td_used_bytes(chunk, L, H, D, T, codec) <= lay["capacity"]
    assert not chunk[used:].any()
    pos = off + np.arange(T)
    x = pool[:, :, table[pos // bs], pos % bs].reshape(L, 2, T, H * D)       # [L][2][T][R] bit patterns
    for (l, kv, g, ch), (scale, codes) in groups.items():
        q, s = oracle.quant_channel(x[l, kv, 64 * g:64 * g + 64, ch], QMAX[codec])
        assert np.float32(s).view(np.uint32) == np.float32(scale).view(np.uint32)
        assert list(q) == codes


@pytest.mark.parametrize("codec,kc", [(TD8, oracle.INT8_KC64), (TD4, oracle.INT4_KC64)])
def test_retrieve_and_compose_equal_the_per_channel_key_codec_on_keys(codec, kc):
    """The entropy coding loses nothing: keys come back exactly as from the per-channel key codec (same groups, same
    arithmetic), and values exactly as keys would if the value planes were key planes."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=16, n_blocks=32)
    k, v = synth.make_pool(shape, "cpu", seed=33)
    pool = synth.pool_to_numpy(k, v)
    swapped = np.ascontiguousarray(pool[:, ::-1])                      # values in the key planes
    table = np.random.default_rng(8).permutation(32)[:10].astype(np.int32)
    T, off = 150, 0
    dst = np.arange(10, dtype=np.int32) + 12
    a, b, c = np.zeros_like(pool), np.zeros_like(pool), np.zeros_like(pool)
    oracle.retrieve(a, dst, 0, T, codec, oracle.store(pool, table, off, T, codec))
    oracle.retrieve(b, dst, 0, T, kc, oracle.store(pool, table, off, T, kc))
    oracle.retrieve(c, dst, 0, T, kc, oracle.store(swapped, table, off, T, kc))
    assert np.array_equal(a[:, 0], b[:, 0])
    assert np.array_equal(a[:, 1], c[:, 0])
    # compose: re-rotated keys come from the unrounded q * scale, as for every codec
    a2, b2 = np.zeros_like(pool), np.zeros_like(pool)
    ka, _ = oracle.compose(a2, dst, [(oracle.store(pool, table, off, T, codec), T, codec, 0, 5)], 10000.0, want_ref=True)
    kb, _ = oracle.compose(b2, dst, [(oracle.store(pool, table, off, T, kc), T, kc, 0, 5)], 10000.0, want_ref=True)
    assert np.array_equal(a2[:, 0], b2[:, 0])
    assert np.array_equal(ka[:, 5:5 + T], kb[:, 5:5 + T])


@pytest.mark.parametrize("codec", [TD8, TD4])
def test_keep_list_chunk_is_the_chunk_of_the_listed_tokens(codec):
    """A keep-list chunk (R9 with R7) is, byte for byte, the dense chunk of a pool in which the listed tokens sit side by
    side: groups are 64 consecutive CHUNK tokens and a difference is taken from the listed token before.  Walked by hand
    as well: every group's codes are the per-channel quantiser's of the listed rows.  Retrieve writes the listed
    positions, each with what the dense retrieve of the compacted pool gives, and nothing else."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=4, n_blocks=64)
    k, v = synth.make_pool(shape, "cpu", seed=27)
    pool = synth.pool_to_numpy(k, v)
    L, H, D, bs = shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size
    rng = np.random.default_rng(4)
    table = rng.permutation(64)[:40].astype(np.int32)                     # 160 positions
    off = 3
    keep = np.sort(rng.choice(150, 100, replace=False)).astype(np.int32)  # two groups: 64 + 36 chunk tokens
    T = len(keep)
    chunk = oracle.store(pool, table, off, T, codec, keep=keep)
    # the same tokens side by side in another pool, stored densely
    pos = off + keep
    packed = np.zeros_like(pool)
    ptab = np.arange(-(-T // bs), dtype=np.int32)
    t = np.arange(T)
    packed[:, :, ptab[t // bs], t % bs] = pool[:, :, table[pos // bs], pos % bs]
    assert np.array_equal(chunk, oracle.store(packed, ptab, 0, T, codec))
    groups, used = walk_chunk(chunk, L, H, D, T, codec)
    x = pool[:, :, table[pos // bs], pos % bs].reshape(L, 2, T, H * D)
    for (l, kv, g, ch), (scale, codes) in groups.items():
        q, sc = oracle.quant_channel(x[l, kv, 64 * g:64 * g + 64, ch], QMAX[codec])
        assert np.float32(sc).view(np.uint32) == np.float32(scale).view(np.uint32) and list(q) == codes
    # with every position listed the list changes nothing
    assert np.array_equal(oracle.store(pool, table, off, 150, codec, keep=np.arange(150)), oracle.store(pool, table, off, 150, codec))
    # retrieve
    dtab = rng.permutation(64)[:40].astype(np.int32)
    got = np.full_like(pool, 0x1234)
    oracle.retrieve(got, dtab, off, T, codec, chunk, keep=keep)
    dense = np.zeros_like(pool)
    oracle.retrieve(dense, ptab, 0, T, codec, chunk)
    want = np.full_like(pool, 0x1234)
    want[:, :, dtab[pos // bs], pos % bs] = dense[:, :, ptab[t // bs], t % bs]
    assert np.array_equal(got, want)


@pytest.mark.parametrize("codec", [TD8, TD4])
def test_select_list_delivers_the_listed_tokens_of_the_full_compose(codec):
    """A select-list changes which positions are written, never what is written there (re-rotated keys and their fp64
    references included); a keep-list that is not strictly increasing is refused as for every codec."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=4, n_blocks=64)
    k, v = synth.make_pool(shape, "cpu", seed=32)
    pool = synth.pool_to_numpy(k, v)
    bs, T, dp, theta = shape.block_size, 100, 8, 10000.0
    rng = np.random.default_rng(10)
    table = rng.permutation(64)[:30].astype(np.int32)
    chunk = oracle.store(pool, table, 0, T, codec)
    rtab = rng.permutation(64)[:30].astype(np.int32)
    sel = np.sort(rng.choice(T, 37, replace=False)).astype(np.int32)
    full = np.full_like(pool, 0x4321)
    kf, _ = oracle.compose(full, rtab, [(chunk, T, codec, 3, dp)], theta, want_ref=True)
    part = np.full_like(pool, 0x4321)
    ks, _ = oracle.compose(part, rtab, [(chunk, T, codec, 3, dp)], theta, want_ref=True, select=[sel])
    pos = dp + sel
    want = np.full_like(pool, 0x4321)
    want[:, :, rtab[pos // bs], pos % bs] = full[:, :, rtab[pos // bs], pos % bs]
    assert np.array_equal(part, want)
    assert np.array_equal(ks[:, pos], kf[:, pos])
    with pytest.raises(ValueError):
        oracle.store(pool, table, 0, 3, codec, keep=[0, 5, 2])


def ar1(rng, n_tokens, n_channels, rho):
    x = np.empty((n_tokens, n_channels))
    x[0] = rng.standard_normal(n_channels)
    for t in range(1, n_tokens):
        x[t] = rho * x[t - 1] + np.sqrt(1 - rho * rho) * rng.standard_normal(n_channels)
    return x


@pytest.mark.parametrize("qmax", [127, 7])
def test_what_the_coding_buys(qmax):
    """Bits per code on channels that vary smoothly along tokens (AR(1), rho = 0.95) and on uncorrelated ones: the
    smooth ones take the delta mode and come out smaller; uncorrelated ones take the direct mode and still beat the
    fixed-rate code (8 or 4 bits) they replace, or at least do not lose to it by more than a fraction of a bit."""
    rng = np.random.default_rng(9)
    res = {}
    for name, rho in (("smooth", 0.95), ("iid", 0.0)):
        x = ar1(rng, 64, 200, rho)
        bits, modes = 0, []
        for c in range(200):
            a = np.abs(x[:, c]).max()
            q = np.rint(x[:, c] / a * qmax).astype(np.int8)
            data, param = oracle.td_encode_channel(q, qmax)
            bits += 8 * len(data)
            modes.append(param >> 3)
        res[name] = (bits / (64 * 200), np.mean(modes))
    fixed = 8 if qmax == 127 else 4
    assert res["smooth"][1] > 0.9 and res["iid"][1] < 0.1
    assert res["smooth"][0] < res["iid"][0] - 0.5
    assert res["iid"][0] < fixed + 0.25
    assert res["smooth"][0] < fixed - 0.6
