"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's source (CPU only, never in the
CUDA path), builds it, and runs the oracle's pins against that build: at least one pin must fail.  A mistake the pins
let through would show up here as a surviving mutant."""
import importlib
import itertools
import os

import pytest

import oracle

SRC = os.path.join(os.path.dirname(oracle.__file__), "kdn_oracle.c")

# (name, text to find, replacement, pin modules to run in this order)
MUTANTS = [
    ("rotation_sign", "*u_out = u * c - w * s;", "*u_out = u * c + w * s;", ["test_oracle_rope"]),
    ("rotation_exponent", "pow(theta, -2.0 * (double)i / (double)D)", "pow(theta, -1.0 * (double)i / (double)D)", ["test_oracle_rope"]),
    ("delta_sign", "int64_t delta = dst_pos[j] - base_pos[j];", "int64_t delta = base_pos[j] - dst_pos[j];", ["test_oracle_rope"]),
    ("pair_partner", "size_t cw = chunk_index(&s, T, l, 0, t, h, i + half);", "size_t cw = chunk_index(&s, T, l, 0, t, h, (i + 1) % D);",
     ["test_oracle_rope"]),
    ("rotate_rounded_value", "u = (double)qu * (double)su;", "u = (double)kdn_oracle_bf16_to_f32(kdn_oracle_dequant((int8_t)qu, su));",
     ["test_oracle_rope", "test_oracle_kc"]),
    ("divide_instead_of_reciprocal", "volatile float prod = kdn_oracle_bf16_to_f32(x_bf16[i]) * inv;",
     "volatile float prod = kdn_oracle_bf16_to_f32(x_bf16[i]) / scale; (void)inv;", ["test_oracle_codec"]),
    ("round_half_away", "float r = rintf(prod);", "float r = roundf(prod);", ["test_oracle_codec"]),
    ("scale_divisor", "volatile float scale = a / qmax;", "volatile float scale = a / (qmax + 1.0f);", ["test_oracle_codec"]),
    ("no_flush_of_tiny_scales", "if (!(scale >= FLT_MIN)) {", "if (!(scale > 0.0f)) {", ["test_oracle_codec"]),
    ("bf16_ties_away", "if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u)))", "if (rest >= 0x8000u)", ["test_oracle_codec"]),
    ("f64_to_bf16_through_fp32", "    if (x != x) return 0x7fc0u;", "    return kdn_oracle_f32_to_bf16((float)x);\n    if (x != x) return 0x7fc0u;",
     ["test_oracle_codec"]),
    ("chunk_axes_swapped", "    i = i * (size_t)T + (size_t)t;\n    i = i * (size_t)s->H + (size_t)h;",
     "    i = i * (size_t)s->H + (size_t)h;\n    i = i * (size_t)T + (size_t)t;", ["test_oracle_mapping", "test_oracle_codec"]),
    ("slot_off_by_one", "int slot = (int)(p % bs);\n                for (int h = 0; h < H; ++h) {\n                    if (codec == KDN_ORACLE_INT4_G64) {",
     "int slot = (int)((p + 1) % bs);\n                for (int h = 0; h < H; ++h) {\n                    if (codec == KDN_ORACLE_INT4_G64) {",
     ["test_oracle_mapping"]),
    ("keep_list_ignored_on_retrieve", "int64_t p = off + (keep ? keep[t] : t);\n                int64_t block = table[p / bs];\n                int slot = (int)(p % bs);\n                for (int h = 0; h < H; ++h)\n                    for (int d = 0; d < D; ++d) {",
     "int64_t p = off + t;\n                int64_t block = table[p / bs];\n                int slot = (int)(p % bs);\n                for (int h = 0; h < H; ++h)\n                    for (int d = 0; d < D; ++d) {",
     ["test_oracle_sparse"]),
    ("nibble_order", "(uint8_t)(((uint8_t)q[2 * k] & 0x0fu) | (((uint8_t)q[2 * k + 1] & 0x0fu) << 4))",
     "(uint8_t)(((uint8_t)q[2 * k + 1] & 0x0fu) | (((uint8_t)q[2 * k] & 0x0fu) << 4))", ["test_oracle_int4"]),
    ("key_groups_all_share_group_0", "if (kv == 0) return (size_t)l * per_layer + (size_t)(t / KDN_ORACLE_GROUP) * hd + ch;",
     "if (kv == 0) return (size_t)l * per_layer + ch;", ["test_oracle_kc"]),
    ("key_groups_along_head_dim", "kdn_oracle_quant_channel(x, n, qmax, q, scales + kc_scale_index(s, T, l, 0, t0, ch));",
     "kdn_oracle_quant_channel(x, 1, qmax, q, scales + kc_scale_index(s, T, l, 0, t0, ch)); for (int i = 1; i < n; ++i) q[i] = q[0];",
     ["test_oracle_kc"]),
    ("checksum_weights", "2u * (uint32_t)i + 1u", "(uint32_t)i + 1u", ["test_oracle_shell"]),
    # the token-delta Rice codecs
    ("bits_from_the_low_end", "if (bit) buf[*pos / 8u] |= (uint8_t)(0x80u >> (*pos % 8u));", "if (bit) buf[*pos / 8u] |= (uint8_t)(1u << (*pos % 8u));",
     ["test_oracle_td"]),
    ("zigzag_signs_swapped", "return e >= 0 ? 2u * (unsigned)e : 2u * (unsigned)(-e) - 1u;", "return e > 0 ? 2u * (unsigned)e - 1u : 2u * (unsigned)(-e);",
     ["test_oracle_td"]),
    ("delta_from_two_tokens_back", "int prev = (mode == 1 && t > 0) ? q[t - 1] : 0;", "int prev = (mode == 1 && t > 1) ? q[t - 2] : 0;", ["test_oracle_td"]),
    ("escape_one_late", "if (quo < 15u) {\n        for (unsigned i = 0; i < quo; ++i) put_bit(buf, pos, 1u);",
     "if (quo < 16u) {\n        for (unsigned i = 0; i < quo; ++i) put_bit(buf, pos, 1u);", ["test_oracle_td"]),
    ("remainder_low_bit_first", "for (int b = k - 1; b >= 0; --b) put_bit(buf, pos, (u >> b) & 1u);", "for (int b = 0; b < k; ++b) put_bit(buf, pos, (u >> b) & 1u);",
     ["test_oracle_td"]),
    ("last_minimum_wins", "if (best_bits < 0 || bits < best_bits) {", "if (best_bits < 0 || bits <= best_bits) {", ["test_oracle_td"]),
    ("segments_not_aligned", "while (cursor % 16u) chunk[cursor++] = 0;", "while (cursor % 4u) chunk[cursor++] = 0;", ["test_oracle_td"]),
    ("values_keep_head_dim_groups", "x[i] = pool[pool_index(s, l, kv, table[p / s->bs], (int)(p % s->bs), h, d)];\n                        }\n                        size_t ch = (size_t)h * (size_t)s->D + (size_t)d;\n                        kdn_oracle_quant_channel(x, n, qmax, q, scales + seg * R + ch);",
     "x[i] = pool[pool_index(s, l, 0, table[p / s->bs], (int)(p % s->bs), h, d)];\n                        }\n                        size_t ch = (size_t)h * (size_t)s->D + (size_t)d;\n                        kdn_oracle_quant_channel(x, n, qmax, q, scales + seg * R + ch);",
     ["test_oracle_td"]),
    ("decoder_forgets_the_running_code", "int v = mode == 1 ? prev + e : e;", "int v = mode == 1 && t == 1 ? prev + e : e;", ["test_oracle_td"]),
    ("keep_list_ignored_by_the_key_groups", "int64_t p = off + (keep ? keep[t0 + i] : t0 + i);                 /* R7: the listed tokens */",
     "int64_t p = off + t0 + i; (void)keep;", ["test_oracle_kc"]),
    ("keep_list_ignored_by_the_token_delta_store", "int64_t p = off + (keep ? keep[t0 + i] : t0 + i);", "int64_t p = off + t0 + i; (void)keep;", ["test_oracle_td"]),
    ("keep_list_restarts_in_every_group", "int64_t p = off + (keep ? keep[t0 + i] : t0 + i);", "int64_t p = off + (keep ? keep[i] + t0 : t0 + i);", ["test_oracle_td"]),
]


def expand(fn):
    """All parameter sets of a test function decorated with pytest.mark.parametrize (none -> one empty set)."""
    axes = []
    for mark in getattr(fn, "pytestmark", []):
        if mark.name != "parametrize":
            continue
        names = [n.strip() for n in mark.args[0].split(",")] if isinstance(mark.args[0], str) else list(mark.args[0])
        vals = [v if isinstance(v, (tuple, list)) and len(names) > 1 else (v,) for v in mark.args[1]]
        axes.append([dict(zip(names, v)) for v in vals])
    for combo in itertools.product(*axes):
        kw = {}
        for d in combo:
            kw.update(d)
        yield kw


def first_failing_pin(modules):
    for modname in modules:
        mod = importlib.import_module(modname)
        for name in sorted(dir(mod)):
            fn = getattr(mod, name)
            if not name.startswith("test_") or not callable(fn) or getattr(fn, "__module__", None) != modname or "every_bit" in name:
                continue
            for kw in expand(fn):
                try:
                    fn(**kw)
                except Exception:                      # an assertion, or the oracle refusing what it should accept
                    return "%s.%s%s" % (modname, name, kw or "")
    return None


def test_the_source_still_has_every_line_the_mutants_replace():
    text = open(SRC).read()
    for name, old, _, _ in MUTANTS:
        assert text.count(old) >= 1, name


@pytest.mark.parametrize("mutant", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, mutant):
    name, old, new, modules = mutant
    text = open(SRC).read()
    assert old in text
    so = oracle.compile_source(text.replace(old, new), str(tmp_path / ("mutant_%s.so" % name)))
    with oracle.use_library(so):
        killer = first_failing_pin(modules)
    assert killer is not None, "no pin noticed the planted mistake '%s'" % name
