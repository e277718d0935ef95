"""Pins for the oracle's int8 group-64 codec and its bf16 rounding (CPU only)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "int8_g64_handworked.txt")
FLT_MIN = np.float32(1.17549435e-38)


def bf16_bits(x):
    """bf16 bit patterns of float values that are exactly representable (asserted)."""
    f = np.asarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    assert np.all((u & 0xffff) == 0), "not a bf16 value"
    return (u >> 16).astype(np.uint16)


def bits_to_f32(b):
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def load_golden():
    cases = []
    with open(GOLDEN) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            name, amax, bits, pairs = [s.strip() for s in line.split("|")]
            pairs = [(float(p.split(":")[0]), int(p.split(":")[1])) for p in pairs.split()]
            cases.append((name, float(amax), int(bits, 16), pairs))
    return cases


@pytest.mark.parametrize("case", load_golden(), ids=lambda c: c[0])
def test_handworked_groups(case):
    _, amax, scale_bits, pairs = case
    x = np.zeros(64, dtype=np.float32)
    x[0] = amax
    for i, (val, _) in enumerate(pairs):
        x[1 + i] = val
    q, scale = oracle.quant_group(bf16_bits(x))
    assert np.float32(scale).view(np.uint32) == scale_bits
    assert q[0] == 127
    for i, (val, code) in enumerate(pairs):
        assert q[1 + i] == code, (val, code, q[1 + i])
    assert np.all(q[1 + len(pairs):] == 0)


def second_formulation(xbits):
    """The codec written again with numpy fp32 scalars and a floor/compare round-half-even."""
    x = bits_to_f32(xbits)
    a = np.max(np.abs(x)).astype(np.float32)
    scale = np.float32(a / np.float32(127.0))
    if not scale >= FLT_MIN:
        return np.zeros(64, dtype=np.int8), np.float32(0.0)
    inv = np.float32(np.float32(127.0) / a)
    prod = (x * inv).astype(np.float32)                 # one fp32 multiply per element
    p = prod.astype(np.float64)                         # exact
    fl = np.floor(p)
    frac = p - fl
    r = np.where(frac > 0.5, fl + 1, np.where(frac < 0.5, fl, np.where(np.mod(fl, 2) == 0, fl, fl + 1)))
    r = np.clip(r, -127, 127)
    return r.astype(np.int8), scale


def groups_from_pool(n_groups, seed):
    shape = synth.TOY.with_(n_blocks=max(1, n_groups // (2 * 2 * 16 * 2) + 1))
    k, v = synth.make_pool(shape, seed=seed)
    return synth.pool_to_numpy(k, v).reshape(-1, 64)[:n_groups]


def test_matches_second_formulation_and_bounds():
    groups = groups_from_pool(6000, seed=21)
    rng = np.random.default_rng(2)
    # widen the range of magnitudes: scale some groups by powers of two (exact in bf16)
    worst = 0.0
    for gi, g in enumerate(groups):
        if gi % 3 == 1:
            e = int(rng.integers(-100, 100))
            g = bf16_bits(bits_to_f32(g) * np.float32(2.0) ** e)
        q, s = oracle.quant_group(g)
        q2, s2 = second_formulation(g)
        assert np.array_equal(q, q2), gi
        assert np.float32(s).view(np.uint32) == np.float32(s2).view(np.uint32)
        x = bits_to_f32(g).astype(np.float64)
        if s == 0:
            continue
        # |x - q*scale| <= scale/2 in real arithmetic, up to the fp32 rounding of x*inv and of the scale
        err = np.abs(x - q.astype(np.float64) * np.float64(s))
        worst = max(worst, float(np.max(err) / (np.float64(s) / 2)))
        assert np.all(err <= (np.float64(s) / 2) * (1 + 2.0 ** -12)), gi
        # the largest-magnitude element codes to +-127; no code is -128
        i = int(np.argmax(np.abs(x)))
        assert abs(int(q[i])) == 127 and q.min() >= -127
        # codes are monotone in x, and carry x's sign or are zero
        order = np.argsort(x, kind="stable")
        assert np.all(np.diff(q[order].astype(np.int32)) >= 0)
        assert np.all((np.sign(q) == np.sign(x)) | (q == 0))
    assert worst > 0.9          # the bound is tight, so the test can notice a wrong rounding rule


def test_zero_and_subnormal_scale_groups():
    z = np.zeros(64, dtype=np.uint16)
    q, s = oracle.quant_group(z)
    assert s == 0 and np.all(q == 0)
    z[5] = 0x8000                                         # -0
    q, s = oracle.quant_group(z)
    assert s == 0 and np.all(q == 0)
    # absmax just under 127 * FLT_MIN -> a/127 is subnormal -> flushed; just above -> coded
    small = np.float32(2.0 ** -120)                       # 2^-120 / 127 < 2^-126
    g = np.zeros(64, dtype=np.float32); g[0] = small; g[1] = -small / 2
    q, s = oracle.quant_group(bf16_bits(g))
    assert s == 0 and np.all(q == 0)
    big = np.float32(2.0 ** -119)                         # 2^-119 / 127 > 2^-126
    g[0] = big; g[1] = -big / 2
    q, s = oracle.quant_group(bf16_bits(g))
    assert s > 0 and q[0] == 127 and q[1] == -64          # 63.5 -> tie -> 64


def test_multiply_and_divide_forms_differ_somewhere():
    """The codec multiplies by 127/a; x / scale is a different function. The oracle must be the former."""
    groups = groups_from_pool(20000, seed=33)
    differ = 0
    for g in groups[:20000:1]:
        x = bits_to_f32(g)
        a = np.max(np.abs(x))
        scale = np.float32(a / np.float32(127.0))
        if not scale >= FLT_MIN:
            continue
        div = np.rint((x / scale).astype(np.float32)).astype(np.int32)
        mul = np.rint((x * np.float32(np.float32(127.0) / a)).astype(np.float32)).astype(np.int32)
        if np.any(div != mul):
            differ += 1
            q, _ = oracle.quant_group(g)
            assert np.array_equal(q.astype(np.int32), np.clip(mul, -127, 127))
            if differ >= 3:
                break
    assert differ >= 1


def test_store_int8_layout_codes_then_scales():
    """Whole-chunk layout: codes [L][2][T][H][D] then scales [L][2][T][H*D/64], each from its own group."""
    shape = synth.TOY.with_(n_blocks=8, block_size=4)
    k, v = synth.make_pool(shape, seed=4)
    pool = synth.pool_to_numpy(k, v)
    table = np.array([6, 1, 3], dtype=np.int32)
    off, T = 1, 10
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    chunk = oracle.store(pool, table, off, T, oracle.INT8_G64)
    n = L * 2 * T * H * D
    assert chunk.size == n + 4 * n // 64
    codes = chunk[:n].view(np.int8).reshape(L, 2, T, H, D)
    scales = chunk[n:].view(np.float32).reshape(L, 2, T, H * D // 64)
    p = off + np.arange(T)
    src = pool[:, :, table[p // 4], p % 4]
    for l in range(L):
        for kv in range(2):
            for t in range(T):
                for h in range(H):
                    q, s = second_formulation(src[l, kv, t, h])
                    assert np.array_equal(codes[l, kv, t, h], q)
                    assert scales[l, kv, t, h].view(np.uint32) == np.float32(s).view(np.uint32)


def test_decode_is_one_fp32_product_rounded_to_bf16():
    """Retrieve of an int8 chunk equals torch's (q.float() * scale).bfloat16() for all codes x many scales."""
    rng = np.random.default_rng(17)
    L, H, D, bs, nb, T = 1, 1, 64, 4, 64, 256
    n = L * 2 * T * H * D
    codes = np.tile(np.arange(-128, 128, dtype=np.int8), n // 256)
    # scales: random normal-range values, powers of two, values whose products hit bf16 ties
    sc = np.abs(rng.standard_normal(n // 64)).astype(np.float32) * np.float32(2.0) ** rng.integers(-30, 30, n // 64)
    sc[:8] = [1.0, 0.5, 2.0 ** -100, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7 + 2.0 ** -8, 3.0 * 2.0 ** -9, 0.0, 2.0 ** -133]
    chunk = np.concatenate([codes.view(np.uint8), sc.astype(np.float32).view(np.uint8)])
    pool = np.zeros((L, 2, nb, bs, H, D), dtype=np.uint16)
    table = np.arange(nb, dtype=np.int32)
    oracle.retrieve(pool, table, 0, T, oracle.INT8_G64, chunk)
    got = pool.reshape(L, 2, T, H * D)
    q = torch.from_numpy(codes.reshape(L, 2, T, H * D).astype(np.float32))
    s = torch.from_numpy(np.repeat(sc.reshape(L, 2, T, H * D // 64), 64, axis=-1))
    want = (q * s).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(got, want)


def test_f32_to_bf16_against_torch_on_rounding_classes():
    hi = np.arange(0, 1 << 16, dtype=np.uint32)
    hi = hi[((hi & 0x7f80) != 0x7f80)]                        # finite upper halves
    lows = np.array([0x0000, 0x0001, 0x7fff, 0x8000, 0x8001, 0xffff], dtype=np.uint32)
    u = (hi[:, None] << 16 | lows[None, :]).reshape(-1)
    f = u.view(np.float32)
    want = torch.from_numpy(f.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    step = 37                                                  # scalar calls through ctypes: sample every 37th
    idx = np.concatenate([np.arange(0, u.size, step), np.arange(6 * 0x3f80, 6 * 0x3f80 + 600)])
    for i in idx:
        assert oracle.f32_to_bf16(f[i]) == want[i], hex(int(u[i]))


def test_f32_to_bf16_against_torch_on_every_bit_pattern():
    """All 2^32 fp32 bit patterns: the oracle's integer add-and-compare rounding against torch's conversion
    (NaNs: both must give a NaN; every other pattern must match bit for bit)."""
    from concurrent.futures import ThreadPoolExecutor
    span = 1 << 26

    def check(k):
        u = np.arange(k * span, (k + 1) * span, dtype=np.uint64).astype(np.uint32)
        f = u.view(np.float32)
        got = oracle.f32_to_bf16_many(f)
        want = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        nan = (u & 0x7fffffff) > 0x7f800000
        bad = (got != want) & ~nan
        got_nan = ((got & 0x7f80) == 0x7f80) & ((got & 0x007f) != 0)
        return int(bad.sum()), bool(np.array_equal(got_nan, nan))

    with ThreadPoolExecutor(max_workers=4) as ex:
        for bad, nans_ok in ex.map(check, range(64)):
            assert bad == 0 and nans_ok


def nearest_bf16_by_search(x):
    """Independent fp64 -> bf16 rounding: search the sorted table of all finite bf16 values."""
    codes = np.arange(0, 0x7f80, dtype=np.uint16)
    vals = bits_to_f32(codes).astype(np.float64)
    a = abs(x)
    i = int(np.searchsorted(vals, a, side="right")) - 1
    if i + 1 >= len(vals):
        j = i
    else:
        lo, hi = vals[i], vals[i + 1]
        if a - lo < hi - a:
            j = i
        elif a - lo > hi - a:
            j = i + 1
        else:
            j = i if (i % 2 == 0) else i + 1
    return int(codes[j]) | (0x8000 if np.signbit(x) else 0)


def test_f64_to_bf16_single_rounding():
    assert oracle.f64_to_bf16(1.0) == 0x3f80
    assert oracle.f64_to_bf16(1.0 + 2.0 ** -8) == 0x3f80            # tie -> even
    assert oracle.f64_to_bf16(1.0 + 3 * 2.0 ** -8) == 0x3f82        # tie -> even (up)
    # would be wrong through fp32: fp32 rounds this to the tie 1 + 2^-8, which then goes down
    assert oracle.f64_to_bf16(1.0 + 2.0 ** -8 + 2.0 ** -40) == 0x3f81
    assert oracle.f64_to_bf16(-0.0) == 0x8000
    assert oracle.f64_to_bf16(2.0 ** -133) == 0x0001                # smallest subnormal
    assert oracle.f64_to_bf16(2.0 ** -134) == 0x0000                # tie with zero -> even
    assert oracle.f64_to_bf16(1.5 * 2.0 ** -134) == 0x0001
    rng = np.random.default_rng(23)
    xs = rng.standard_normal(3000) * 10.0 ** rng.integers(-6, 6, 3000)
    for x in xs:
        assert oracle.f64_to_bf16(float(x)) == nearest_bf16_by_search(float(x))


def test_double_rounding_witnesses():
    """Groups where the codec's two roundings matter: x = a/2 and fl(127/a) < 127/a, so the exact product is just
    below 63.5 but the fp32 product IS 63.5, a tie that goes to 64.  One fused rounding would give 63."""
    from fractions import Fraction
    for a in [21.25, 38.5, 46.0, 84.0, 23.0, 25.75]:
        inv = np.float32(127.0) / np.float32(a)
        x = np.float32(a / 2)
        exact = Fraction(float(x)) * Fraction(float(inv))
        assert exact < Fraction(127, 2) and np.float32(x * inv) == np.float32(63.5)
        g = np.zeros(64, dtype=np.float32); g[0] = a; g[1] = x; g[2] = -x
        q, _ = oracle.quant_group(bf16_bits(g))
        assert (q[0], q[1], q[2]) == (127, 64, -64)
