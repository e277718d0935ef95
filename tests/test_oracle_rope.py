"""Pins for the oracle's key re-rotation and composition (CPU only)."""
import math

import numpy as np
import pytest

import oracle
from paper_2409_13761_b200 import synth


def bits_to_f64(b):
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def f32_to_bf16_bits(x):
    import torch
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def rope_complex(x, pos, theta):
    """Rotary embedding by complex multiplication: (x[i] + 1j*x[i+D/2]) * exp(1j*pos*theta^(-2i/D))."""
    D = x.shape[-1]
    half = D // 2
    i = np.arange(half, dtype=np.float64)
    ang = np.asarray(pos, dtype=np.float64)[..., None] * theta ** (-2.0 * i / D)
    z = (x[..., :half] + 1j * x[..., half:]) * np.exp(1j * ang)
    return np.concatenate([z.real, z.imag], axis=-1)


def test_angle_and_pair_closed_forms():
    # i = 0: frequency 1, angle = delta exactly; theta irrelevant
    for delta in (0, 1, -7, 131072, -(1 << 40)):
        assert oracle.rope_angle(delta, 500000.0, 0, 128) == float(delta)
    # theta = 10000, D = 64, i = 16: theta^(-1/2) = 0.01
    assert oracle.rope_angle(256, 10000.0, 16, 64) == pytest.approx(2.56, rel=1e-15)
    # theta = 16, D = 8: inverse frequencies 1, 1/2, 1/4, 1/8
    for i in range(4):
        assert oracle.rope_angle(24, 16.0, i, 8) == pytest.approx(24.0 / 2 ** i, rel=1e-15)
    # quarter and half turns: (u, w) -> (-w, u) and (-u, -w)
    u2, w2 = oracle.rotate_pair(3.0, 5.0, math.pi / 2)
    assert u2 == pytest.approx(-5.0, abs=1e-15) and w2 == pytest.approx(3.0, abs=1e-15)
    u2, w2 = oracle.rotate_pair(3.0, 5.0, math.pi)
    assert u2 == pytest.approx(-3.0, abs=1e-15) and w2 == pytest.approx(-5.0, abs=1e-15)
    assert oracle.rotate_pair(3.0, 5.0, 0.0) == (3.0, 5.0)
    # a small positive angle moves (1, 0) counter-clockwise: second component becomes positive
    u2, w2 = oracle.rotate_pair(1.0, 0.0, 0.1)
    assert u2 == pytest.approx(math.cos(0.1)) and w2 == pytest.approx(math.sin(0.1))


def test_rotations_compose_and_preserve_norm():
    rng = np.random.default_rng(3)
    for _ in range(2000):
        u, w = rng.standard_normal(2) * 10
        a, b = rng.uniform(-1e5, 1e5, 2)
        u1, w1 = oracle.rotate_pair(u, w, a)
        u2, w2 = oracle.rotate_pair(u1, w1, b)
        u3, w3 = oracle.rotate_pair(u, w, a + b)
        n = math.hypot(u, w)
        assert abs(u2 - u3) <= 1e-10 * n and abs(w2 - w3) <= 1e-10 * n     # 1e5 rad * 2^-53 ~ 1e-11
        assert math.hypot(u1, w1) == pytest.approx(n, rel=1e-14)


def make_request(seed, shape, T_parts, base_pos, dst_pos, codecs, theta):
    """Pool holding, for each part, keys = rotary(x, base_pos + t) rounded to bf16; returns everything."""
    rng = np.random.default_rng(seed)
    L, H, D, bs, nb = shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size, shape.n_blocks
    pool = rng.integers(0, 1 << 16, size=(L, 2, nb, bs, H, D), dtype=np.uint16)
    free = list(rng.permutation(nb))
    parts, xs = [], []
    for T, bp, dp, cd in zip(T_parts, base_pos, dst_pos, codecs):
        n_tb = -(-T // bs)
        tab = np.array([free.pop() for _ in range(n_tb)], dtype=np.int32)
        x = rng.standard_normal((L, T, H, D))
        kk = rope_complex(x, (bp + np.arange(T))[None, :, None], theta)
        vv = rng.standard_normal((L, T, H, D))
        p = np.arange(T)
        pool[:, 0, tab[p // bs], p % bs] = f32_to_bf16_bits(kk)
        pool[:, 1, tab[p // bs], p % bs] = f32_to_bf16_bits(vv)
        chunk = oracle.store(pool, tab, 0, T, cd)
        parts.append((chunk, T, cd, bp, dp))
        xs.append(x)
    return pool, free, parts, xs


def stored_keys_f64(chunk, L, T, H, D, codec):
    """The value the codec says a stored key element has, before any bf16 rounding."""
    n = L * 2 * T * H * D
    if codec == oracle.RAW_BF16:
        return bits_to_f64(chunk.view(np.uint16).reshape(L, 2, T, H, D)[:, 0])
    codes = chunk[:n].view(np.int8).reshape(L, 2, T, H, D)[:, 0].astype(np.float64)
    scales = chunk[n:].view(np.float32).reshape(L, 2, T, H * D // 64)[:, 0].astype(np.float64)
    return codes * np.repeat(scales, 64, axis=-1).reshape(L, T, H, D)


@pytest.mark.parametrize("codec", [oracle.RAW_BF16, oracle.INT8_G64])
@pytest.mark.parametrize("D", [64, 128])
def test_compose_rerotation_against_complex_formulation(codec, D):
    theta = 10000.0
    shape = synth.TOY.with_(head_dim=D, block_size=4, n_blocks=40)
    L, H, bs = shape.n_layers, shape.n_kv_heads, shape.block_size
    T_parts, base, dst = [9, 6, 5], [0, 100, 7], [3, 12, 18]           # deltas 3, -88, 11; unaligned starts
    pool, free, parts, xs = make_request(1, shape, T_parts, base, dst, [codec] * 3, theta)
    n_tb = 7
    table = np.array(free[:n_tb], dtype=np.int32)
    before = pool.copy()
    kref, kmag = oracle.compose(pool, table, parts, theta, want_ref=True)
    covered = np.zeros(n_tb * bs, dtype=bool)
    for (chunk, T, cd, bp, dp), x in zip(parts, xs):
        k_stored = stored_keys_f64(chunk, L, T, H, D, cd)                 # [L][T][H][D]
        want = rope_complex(k_stored, np.full((1, T, 1), dp - bp), theta)
        got = kref[:, dp:dp + T]
        assert np.allclose(got, want, rtol=0, atol=1e-12 * np.abs(k_stored).max())
        # pool holds the fp64 result rounded once to bf16
        p = dp + np.arange(T)
        inpool = bits_to_f64(pool[:, 0, table[p // bs], p % bs])
        half_ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(got), 2.0 ** -126))) - 8)
        assert np.all(np.abs(inpool - got) <= half_ulp)        # the nearest bf16 to the fp64 result
        # use-case invariant: keys made at base_pos + t, re-rotated, equal keys made at dst_pos + t,
        # up to the rounding the stored keys already carried (bf16, plus half a quantisation step for int8)
        scratch = rope_complex(x, (dp + np.arange(T))[None, :, None], theta)
        tol = 2.0 ** -8 * np.abs(x).max() * 2 + (0.0 if cd == oracle.RAW_BF16 else np.abs(x).max() / 127 * 1.01)
        assert np.max(np.abs(got - scratch)) <= tol
        assert np.max(np.abs(got - scratch)) > 0          # not trivially the same array
        # values are a plain retrieve
        ref = before.copy()
        oracle.retrieve(ref, table, dp, T, cd, chunk)
        assert np.array_equal(pool[:, 1, table[p // bs], p % bs], ref[:, 1, table[p // bs], p % bs])
        # pair magnitudes reported for the tolerance
        half = D // 2
        mag = np.abs(k_stored[..., :half]) + np.abs(k_stored[..., half:])
        assert np.allclose(kmag[:, dp:dp + T, :, :half], mag) and np.allclose(kmag[:, dp:dp + T, :, half:], mag)
        covered[dp:dp + T] = True
    # positions no part covers, and every block outside the table, keep their bits
    untouched = ~covered
    pu = np.flatnonzero(untouched)
    assert np.array_equal(pool[:, :, table[pu // bs], pu % bs], before[:, :, table[pu // bs], pu % bs])
    others = np.setdiff1d(np.arange(shape.n_blocks), table)
    assert np.array_equal(pool[:, :, others], before[:, :, others])
    assert np.all(np.isnan(kref[:, untouched]))


@pytest.mark.parametrize("codec", [oracle.RAW_BF16, oracle.INT8_G64])
def test_compose_with_zero_delta_is_a_sequence_of_retrieves(codec):
    theta = 500000.0
    shape = synth.TOY.with_(block_size=16, n_blocks=24)
    T_parts, pos = [20, 13], [5, 40]
    pool, free, parts, _ = make_request(2, shape, T_parts, pos, pos, [codec, codec], theta)
    table = np.array(free[:4], dtype=np.int32)
    ref = pool.copy()
    for chunk, T, cd, bp, dp in parts:
        oracle.retrieve(ref, table, dp, T, cd, chunk)
    oracle.compose(pool, table, parts, theta)
    assert np.array_equal(pool, ref)


def test_compose_brute_force_tiny():
    """Every element by hand-written Python loops, mixed codecs, block_size 3, negative and positive deltas."""
    theta = 100.0
    shape = synth.TOY.with_(n_layers=1, n_kv_heads=1, head_dim=64, block_size=3, n_blocks=12)
    L, H, D, bs = 1, 1, 64, 3
    pool, free, parts, _ = make_request(5, shape, [4, 2], [10, 0], [1, 6], [oracle.RAW_BF16, oracle.INT8_G64], theta)
    table = np.array(free[:3], dtype=np.int32)
    want = pool.copy()
    for chunk, T, cd, bp, dp in parts:
        ks = stored_keys_f64(chunk, L, T, H, D, cd)[0, :, 0]            # [T][D]
        delta = dp - bp
        for t in range(T):
            p = dp + t
            blk, slot = int(table[p // bs]), p % bs
            for i in range(D // 2):
                phi = delta * theta ** (-2.0 * i / D)
                u, w = ks[t, i], ks[t, i + D // 2]
                want[0, 0, blk, slot, 0, i] = oracle.f64_to_bf16(u * math.cos(phi) - w * math.sin(phi))
                want[0, 0, blk, slot, 0, i + D // 2] = oracle.f64_to_bf16(w * math.cos(phi) + u * math.sin(phi))
        ref = pool.copy()
        oracle.retrieve(ref, table, dp, T, cd, chunk)
        for t in range(T):
            p = dp + t
            want[0, 1, table[p // bs], p % bs] = ref[0, 1, table[p // bs], p % bs]
    oracle.compose(pool, table, parts, theta)
    assert np.array_equal(pool, want)
