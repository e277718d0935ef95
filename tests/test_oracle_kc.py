"""Pins for the oracle's per-channel key codecs (keys grouped along tokens, values along head_dim; CPU only)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from test_oracle_codec import bf16_bits, bits_to_f32, FLT_MIN
from test_oracle_int4 import unpack_nibbles
from test_oracle_rope import rope_complex, bits_to_f64

KC = [(oracle.INT8_KC64, oracle.INT8_G64, 127), (oracle.INT4_KC64, oracle.INT4_G64, 7)]


def split_chunk(chunk, L, T, H, D, codec):
    """codes int [L][2][T][H*D], k_scales fp32 [L][G][H*D], v_scales fp32 [L][T][H*D/64] -- from the layout as documented,
    not through the oracle."""
    n, hd, G = L * 2 * T * H * D, H * D, -(-T // 64)
    if codec == oracle.INT4_KC64:
        codes = unpack_nibbles(chunk[:n // 2]).reshape(L, 2, T, hd)
        sc = chunk[n // 2:].view(np.float32)
    else:
        codes = chunk[:n].view(np.int8).astype(np.int32).reshape(L, 2, T, hd)
        sc = chunk[n:].view(np.float32)
    per_layer = G * hd + T * hd // 64
    assert sc.size == L * per_layer
    sc = sc.reshape(L, per_layer)
    return codes, sc[:, :G * hd].reshape(L, G, hd), sc[:, G * hd:].reshape(L, T, hd // 64)


def gathered(pool, table, off, T):
    bs = pool.shape[3]
    p = off + np.arange(T)
    L, _, _, _, H, D = pool.shape
    return pool[:, :, table[p // bs], p % bs].reshape(L, 2, T, H * D)


def second_formulation(xbits, qmax):
    """One group along axis 0 (any length): fp32 arithmetic in numpy, rounding by floor and compare."""
    x = bits_to_f32(xbits)
    a = np.max(np.abs(x), axis=0).astype(np.float32)
    scale = (a / np.float32(qmax)).astype(np.float32)
    ok = scale >= FLT_MIN
    with np.errstate(divide="ignore"):
        inv = np.where(ok, (np.float32(qmax) / a).astype(np.float32), np.float32(0))
    p = (x * inv[None]).astype(np.float32).astype(np.float64)
    fl = np.floor(p)
    frac = p - fl
    r = np.where(frac > 0.5, fl + 1, np.where(frac < 0.5, fl, np.where(np.mod(fl, 2) == 0, fl, fl + 1)))
    return np.clip(r, -qmax, qmax).astype(np.int32), np.where(ok, scale, np.float32(0))


@pytest.mark.parametrize("codec,base,qmax", KC)
def test_hand_worked_channel_groups(codec, base, qmax):
    # absmax = qmax -> scale exactly 1, codes are the values rounded half to even; a short group of 5 tokens
    x = np.array([qmax, 0.5, 1.5, 2.5, -3.5], dtype=np.float32)
    q, s = oracle.quant_channel(bf16_bits(x), qmax)
    assert s == np.float32(1.0) and list(q) == [qmax, 0, 2, 2, -4]
    # absmax 1: scale is fl(1/qmax), 0.5 -> qmax/2 rounded half to even
    q, s = oracle.quant_channel(bf16_bits(np.array([0.5, -1.0, 0.25], dtype=np.float32)), qmax)
    assert s == np.float32(1.0) / np.float32(qmax)
    assert list(q) == ([64, -127, 32] if qmax == 127 else [4, -7, 2])        # 63.5 -> 64, 31.75 -> 32; 3.5 -> 4, 1.75 -> 2
    # an all-zero channel, and one whose scale would be subnormal
    q, s = oracle.quant_channel(np.zeros(64, dtype=np.uint16), qmax)
    assert s == 0 and not q.any()
    q, s = oracle.quant_channel(bf16_bits(np.full(3, 2.0 ** -126, dtype=np.float32)), qmax)
    assert s == 0 and not q.any()


@pytest.mark.parametrize("codec,base,qmax", KC)
@pytest.mark.parametrize("off,T", [(0, 64), (5, 100), (3, 7), (16, 192)])
def test_store_matches_second_formulation_layout_and_bound(codec, base, qmax, off, T):
    shape = synth.TOY.with_(n_blocks=40, block_size=16, head_dim=128)
    k, v = synth.make_pool(shape, "cpu", seed=11)
    pool = synth.pool_to_numpy(k, v)
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    table = np.random.default_rng(4).permutation(shape.n_blocks)[:14].astype(np.int32)
    chunk = oracle.store(pool, table, off, T, codec)
    assert chunk.size == oracle.chunk_bytes(L, H, D, T, codec) == (L * 2 * T * H * D // (2 if qmax == 7 else 1)
                                                                    + 4 * L * (-(-T // 64) * H * D + T * H * D // 64))
    codes, ks, vs = split_chunk(chunk, L, T, H, D, codec)
    x = gathered(pool, table, off, T)
    # values: exactly the group-64 codec's value planes
    bcodes = oracle.store(pool, table, off, T, base)
    n = L * 2 * T * H * D
    if qmax == 7:
        want_codes = unpack_nibbles(bcodes[:n // 2]).reshape(L, 2, T, H * D)
        want_sc = bcodes[n // 2:].view(np.float32).reshape(L, 2, T, H * D // 64)
    else:
        want_codes = bcodes[:n].view(np.int8).astype(np.int32).reshape(L, 2, T, H * D)
        want_sc = bcodes[n:].view(np.float32).reshape(L, 2, T, H * D // 64)
    assert np.array_equal(codes[:, 1], want_codes[:, 1]) and np.array_equal(vs, want_sc[:, 1])
    # keys: every (64-token span, channel) group against the second formulation, and the error bound
    for l in range(L):
        for g in range(-(-T // 64)):
            t0, t1 = 64 * g, min(T, 64 * g + 64)
            q2, s2 = second_formulation(x[l, 0, t0:t1], qmax)
            assert np.array_equal(codes[l, 0, t0:t1], q2)
            assert np.array_equal(ks[l, g].view(np.uint32), s2.astype(np.float32).view(np.uint32))
            xv = bits_to_f32(x[l, 0, t0:t1]).astype(np.float64)
            s64 = ks[l, g].astype(np.float64)
            assert np.all(np.abs(xv - codes[l, 0, t0:t1] * s64[None]) <= s64[None] / 2 * (1 + 2.0 ** -12))
            top = np.abs(codes[l, 0, t0:t1]).max(axis=0)
            assert np.all((top == qmax) | (s64 == 0))                  # the largest element of a channel codes to +-qmax


@pytest.mark.parametrize("codec,base,qmax", KC)
def test_an_outlier_channel_does_not_cost_its_neighbours(codec, base, qmax):
    """The point of grouping keys along tokens: with a few channels 20x larger, ordinary key channels keep their own
    step.  Their error must be far below that of the group-64 codec, which shares the outliers' scale."""
    shape = synth.TOY.with_(n_blocks=16, head_dim=128)
    k, v = synth.make_pool(shape, "cpu", seed=5)
    pool = synth.pool_to_numpy(k, v)
    gain = synth.outlier_gain(shape).numpy()[:, 0].reshape(shape.n_layers, -1)           # [L][H*D] for keys
    table = np.arange(8, dtype=np.int32)
    T = 128
    x = bits_to_f32(gathered(pool, table, 0, T)[:, 0]).astype(np.float64)
    err = {}
    for cd in (codec, base):
        ref = np.zeros_like(pool)
        oracle.retrieve(ref, table, 0, T, cd, oracle.store(pool, table, 0, T, cd))
        y = bits_to_f32(gathered(ref, table, 0, T)[:, 0]).astype(np.float64)
        e = (x - y) ** 2
        err[cd] = np.array([e[l][:, gain[l] == 1].mean() for l in range(shape.n_layers)]).mean()
    assert err[codec] * 20 < err[base]


@pytest.mark.parametrize("codec,base,qmax", KC)
def test_retrieve_decodes_with_the_elements_own_scale(codec, base, qmax):
    shape = synth.TOY.with_(n_blocks=40, block_size=8)
    k, v = synth.make_pool(shape, "cpu", seed=12)
    pool = synth.pool_to_numpy(k, v)
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    table = np.random.default_rng(9).permutation(shape.n_blocks)[:20].astype(np.int32)
    off, T = 3, 150
    chunk = oracle.store(pool, table, 0, T, codec)
    codes, ks, vs = split_chunk(chunk, L, T, H, D, codec)
    kscale = np.repeat(ks, 64, axis=1)[:, :T]                                  # [L][T][H*D]
    vscale = np.repeat(vs, 64, axis=-1)
    want_k = (torch.from_numpy(codes[:, 0].astype(np.float32)) * torch.from_numpy(kscale)).to(torch.bfloat16)
    want_v = (torch.from_numpy(codes[:, 1].astype(np.float32)) * torch.from_numpy(vscale)).to(torch.bfloat16)
    dst = pool.copy()
    oracle.retrieve(dst, table, off, T, codec, chunk)
    got = gathered(dst, table, off, T)
    assert np.array_equal(got[:, 0], want_k.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(got[:, 1], want_v.view(torch.int16).numpy().view(np.uint16))
    # only the addressed slots changed
    bs = shape.block_size
    mask = np.ones(pool.shape[2:4], dtype=bool)
    p = off + np.arange(T)
    mask[table[p // bs], p % bs] = False
    assert np.array_equal(dst[:, :, mask], pool[:, :, mask])


@pytest.mark.parametrize("codec,base,qmax", KC)
def test_compose_rotates_the_unrounded_stored_key(codec, base, qmax):
    theta = 10000.0
    shape = synth.TOY.with_(n_blocks=40, block_size=4)
    k, v = synth.make_pool(shape, "cpu", seed=13)
    pool = synth.pool_to_numpy(k, v)
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    src = np.arange(20, dtype=np.int32)
    T, bp, dp = 70, 5, 9
    chunk = oracle.store(pool, src, 2, T, codec)
    codes, ks, _ = split_chunk(chunk, L, T, H, D, codec)
    stored = (codes[:, 0].astype(np.float64) * np.repeat(ks, 64, axis=1)[:, :T].astype(np.float64)).reshape(L, T, H, D)
    table = np.arange(20, 40, dtype=np.int32)
    before = pool.copy()
    kref, kmag = oracle.compose(pool, table, [(chunk, T, codec, bp, dp)], theta, want_ref=True)
    want = rope_complex(stored, np.full((1, T, 1), dp - bp), theta)
    assert np.allclose(kref[:, dp:dp + T], want, rtol=0, atol=1e-12 * np.abs(stored).max())
    half = D // 2
    mag = np.abs(stored[..., :half]) + np.abs(stored[..., half:])
    assert np.allclose(kmag[:, dp:dp + T, :, :half], mag)
    p = dp + np.arange(T)
    ref = before.copy()
    oracle.retrieve(ref, table, dp, T, codec, chunk)                           # values are a plain retrieve
    assert np.array_equal(pool[:, 1, table[p // 4], p % 4], ref[:, 1, table[p // 4], p % 4])
    same = before.copy()                                                       # delta 0: keys too
    oracle.compose(same, table, [(chunk, T, codec, dp, dp)], theta)
    assert np.array_equal(same, ref)


@pytest.mark.parametrize("codec,base,qmax", KC)
def test_keep_list_chunk_is_the_chunk_of_the_listed_tokens(codec, base, qmax):
    """A keep-list chunk is, byte for byte, the dense chunk of a pool in which the listed tokens sit side by side (key
    groups are 64 consecutive CHUNK tokens), its codes and scales are the second formulation's on the listed rows, and
    retrieve writes the listed positions with what the dense retrieve of that pool gives, nothing else.  Select-lists
    stay refused."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=4, n_blocks=64)
    k, v = synth.make_pool(shape, "cpu", seed=29)
    pool = synth.pool_to_numpy(k, v)
    L, H, D, bs = shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size
    rng = np.random.default_rng(6)
    table = rng.permutation(64)[:40].astype(np.int32)
    off = 2
    keep = np.sort(rng.choice(150, 100, replace=False)).astype(np.int32)
    T = len(keep)
    chunk = oracle.store(pool, table, off, T, codec, keep=keep)
    pos = off + keep
    t = np.arange(T)
    ptab = np.arange(-(-T // bs), dtype=np.int32)
    packed = np.zeros_like(pool)
    packed[:, :, ptab[t // bs], t % bs] = pool[:, :, table[pos // bs], pos % bs]
    assert np.array_equal(chunk, oracle.store(packed, ptab, 0, T, codec))
    codes, k_sc, _ = split_chunk(chunk, L, T, H, D, codec)
    x = pool[:, :, table[pos // bs], pos % bs].reshape(L, 2, T, H * D)
    for l in range(L):
        for g in range(-(-T // 64)):
            q, sc = second_formulation(x[l, 0, 64 * g:64 * g + 64], qmax)
            assert np.array_equal(codes[l, 0, 64 * g:64 * g + 64], q)
            assert np.array_equal(k_sc[l, g].view(np.uint32), sc.astype(np.float32).view(np.uint32))
    dtab = rng.permutation(64)[:40].astype(np.int32)
    got = np.full_like(pool, 0x1234)
    oracle.retrieve(got, dtab, off, T, codec, chunk, keep=keep)
    dense = np.zeros_like(pool)
    oracle.retrieve(dense, ptab, 0, T, codec, chunk)
    want = np.full_like(pool, 0x1234)
    want[:, :, dtab[pos // bs], pos % bs] = dense[:, :, ptab[t // bs], t % bs]
    assert np.array_equal(got, want)


@pytest.mark.parametrize("codec,base,qmax", KC)
def test_select_list_delivers_the_listed_tokens_of_the_full_compose(codec, base, qmax):
    """A select-list changes which positions are written, never what is written there: the listed positions hold what
    the compose of the whole part puts there (rotated keys included, their fp64 references too), every other position
    keeps its bits."""
    shape = synth.TOY.with_(n_layers=2, n_kv_heads=2, head_dim=64, block_size=4, n_blocks=64)
    k, v = synth.make_pool(shape, "cpu", seed=30)
    pool = synth.pool_to_numpy(k, v)
    bs, T, dp, theta = shape.block_size, 100, 8, 10000.0
    rng = np.random.default_rng(9)
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
