"""Pins for the oracle's int4 group-64 codec (CPU only)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from test_oracle_codec import bf16_bits, bits_to_f32, groups_from_pool, FLT_MIN

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "int4_g64_handworked.txt")


def unpack_nibbles(packed):
    """uint8 [..., n] -> int [..., 2n]: low nibble first, sign-extended (written without reference to the oracle)."""
    p = np.asarray(packed, dtype=np.uint8).astype(np.int32)
    lo, hi = p & 15, p >> 4
    both = np.stack([lo, hi], axis=-1).reshape(p.shape[:-1] + (-1,))
    return np.where(both >= 8, both - 16, both)


def load_golden():
    cases = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, amax, bits, pairs = [s.strip() for s in line.split("|")]
            cases.append((name, float(amax), int(bits, 16), [(float(p.split(":")[0]), int(p.split(":")[1])) for p in pairs.split()]))
    return cases


@pytest.mark.parametrize("case", load_golden(), ids=lambda c: c[0])
def test_handworked_groups(case):
    _, amax, scale_bits, pairs = case
    x = np.zeros(64, dtype=np.float32)
    x[0] = amax
    for i, (val, _) in enumerate(pairs):
        x[1 + i] = val
    packed, scale = oracle.quant4_group(bf16_bits(x))
    q = unpack_nibbles(packed)
    assert np.float32(scale).view(np.uint32) == scale_bits
    assert q[0] == 7
    for i, (val, code) in enumerate(pairs):
        assert q[1 + i] == code, (val, code, q[1 + i])
    assert np.all(q[1 + len(pairs):] == 0)


def test_nibble_order_by_hand():
    x = np.zeros(64, dtype=np.float32)
    x[0], x[1], x[2], x[3], x[63] = 7.0, -1.0, 2.0, -7.0, 5.0          # scale 1: codes are the values
    packed, _ = oracle.quant4_group(bf16_bits(x))
    assert packed[0] == 0xF7          # element 0 (7) low, element 1 (-1 = 0xF) high
    assert packed[1] == 0x92          # element 2 (2) low, element 3 (-7 = 0x9) high
    assert packed[31] == 0x50         # element 62 (0) low, element 63 (5) high
    assert np.all(packed[2:31] == 0)


def second_formulation(xbits):
    x = bits_to_f32(xbits)
    a = np.max(np.abs(x)).astype(np.float32)
    scale = np.float32(a / np.float32(7.0))
    if not scale >= FLT_MIN:
        return np.zeros(64, dtype=np.int32), np.float32(0.0)
    inv = np.float32(np.float32(7.0) / a)
    p = (x * inv).astype(np.float32).astype(np.float64)
    fl = np.floor(p)
    frac = p - fl
    r = np.where(frac > 0.5, fl + 1, np.where(frac < 0.5, fl, np.where(np.mod(fl, 2) == 0, fl, fl + 1)))
    return np.clip(r, -7, 7).astype(np.int32), scale


def test_matches_second_formulation_and_bounds():
    groups = groups_from_pool(4000, seed=77)
    rng = np.random.default_rng(5)
    worst = 0.0
    for gi, g in enumerate(groups):
        if gi % 3 == 1:
            g = bf16_bits(bits_to_f32(g) * np.float32(2.0) ** int(rng.integers(-100, 100)))
        packed, s = oracle.quant4_group(g)
        q = unpack_nibbles(packed)
        q2, s2 = second_formulation(g)
        assert np.array_equal(q, q2), gi
        assert np.float32(s).view(np.uint32) == np.float32(s2).view(np.uint32)
        if s == 0:
            continue
        x = bits_to_f32(g).astype(np.float64)
        err = np.abs(x - q * np.float64(s))
        worst = max(worst, float(err.max() / (np.float64(s) / 2)))
        assert np.all(err <= (np.float64(s) / 2) * (1 + 2.0 ** -12))
        assert abs(int(q[int(np.argmax(np.abs(x)))])) == 7 and q.min() >= -7 and q.max() <= 7
        assert np.all(np.diff(q[np.argsort(x, kind="stable")]) >= 0)
    assert worst > 0.9
    z = np.zeros(64, dtype=np.uint16)
    packed, s = oracle.quant4_group(z)
    assert s == 0 and not packed.any()
    g = np.zeros(64, dtype=np.float32); g[0] = 2.0 ** -124; g[1] = -2.0 ** -125      # 2^-124 / 7 < 2^-126: flushed
    packed, s = oracle.quant4_group(bf16_bits(g))
    assert s == 0 and not packed.any()


def test_chunk_layout_and_decode_against_torch():
    shape = synth.TOY.with_(n_blocks=8, block_size=4)
    k, v = synth.make_pool(shape, seed=6)
    pool = synth.pool_to_numpy(k, v)
    table = np.array([5, 0, 2], dtype=np.int32)
    off, T = 1, 10
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    chunk = oracle.store(pool, table, off, T, oracle.INT4_G64)
    n = L * 2 * T * H * D
    assert chunk.size == n // 2 + 4 * n // 64 == oracle.chunk_bytes(L, H, D, T, oracle.INT4_G64)
    codes = unpack_nibbles(chunk[:n // 2]).reshape(L, 2, T, H, D)
    scales = chunk[n // 2:].view(np.float32).reshape(L, 2, T, H * D // 64)
    p = off + np.arange(T)
    src = pool[:, :, table[p // 4], p % 4]
    for l in range(L):
        for kv in range(2):
            for t in range(T):
                for h in range(H):
                    q, s = second_formulation(src[l, kv, t, h])
                    assert np.array_equal(codes[l, kv, t, h], q)
                    assert scales[l, kv, t, h].view(np.uint32) == np.float32(s).view(np.uint32)
    # decode = torch's (q.float() * scale).bfloat16(), written only into the addressed slots
    out = np.full_like(pool, 0x7fa5)
    dst = np.array([7, 3, 1], dtype=np.int32)
    oracle.retrieve(out, dst, 2, T, oracle.INT4_G64, chunk)
    want = (torch.from_numpy(codes.astype(np.float32)) * torch.from_numpy(np.repeat(scales, 64, axis=-1).reshape(L, 2, T, H, D))
            ).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    p2 = 2 + np.arange(T)
    assert np.array_equal(out[:, :, dst[p2 // 4], p2 % 4], want)
    mask = np.ones(out.shape[2:4], dtype=bool)
    mask[dst[p2 // 4], p2 % 4] = False
    assert np.all(out[:, :, mask] == 0x7fa5)


def test_compose_int4_rotates_the_unrounded_stored_value():
    from test_oracle_rope import rope_complex, bits_to_f64
    theta = 10000.0
    shape = synth.TOY.with_(block_size=4, n_blocks=16)
    k, v = synth.make_pool(shape, seed=3)
    pool = synth.pool_to_numpy(k, v)
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    T = 9
    src = np.array([1, 5, 9], dtype=np.int32)
    chunk = oracle.store(pool, src, 0, T, oracle.INT4_G64)
    n = L * 2 * T * H * D
    codes = unpack_nibbles(chunk[:n // 2]).reshape(L, 2, T, H, D)[:, 0].astype(np.float64)
    scales = np.repeat(chunk[n // 2:].view(np.float32).reshape(L, 2, T, H * D // 64)[:, 0].astype(np.float64), 64, axis=-1).reshape(L, T, H, D)
    stored = codes * scales
    table = np.array([12, 3, 7, 14], dtype=np.int32)
    before = pool.copy()
    kref, _ = oracle.compose(pool, table, [(chunk, T, oracle.INT4_G64, 40, 5)], theta, want_ref=True)
    want = rope_complex(stored, np.full((1, T, 1), 5 - 40), theta)
    assert np.allclose(kref[:, 5:5 + T], want, rtol=0, atol=1e-12 * np.abs(stored).max())
    ref = before.copy()
    oracle.retrieve(ref, table, 5, T, oracle.INT4_G64, chunk)
    assert np.array_equal(pool[:, 1], ref[:, 1])                                  # values: a plain retrieve


def test_double_rounding_witnesses_int4():
    """x = a/2 with fl(7/a) < 7/a: the exact product is just below 3.5, the fp32 product IS 3.5 -> tie -> 4."""
    from fractions import Fraction
    for a in [16.125, 17.25, 19.0, 20.0, 25.75]:
        inv = np.float32(7.0) / np.float32(a)
        x = np.float32(a / 2)
        assert Fraction(float(x)) * Fraction(float(inv)) < Fraction(7, 2) and np.float32(x * inv) == np.float32(3.5)
        g = np.zeros(64, dtype=np.float32); g[0] = a; g[1] = x; g[2] = -x
        q = unpack_nibbles(oracle.quant4_group(bf16_bits(g))[0])
        assert (q[0], q[1], q[2]) == (7, 4, -4)
