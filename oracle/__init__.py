"""CPU oracle for the KDN store / retrieve / compose path (test infrastructure).

The arithmetic lives in ``kdn_oracle.c`` (plain scalar C, one loop nest per
definition).  This module compiles it with gcc on first use and exposes it to
numpy.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
import this package; the CUDA library and its Python binding never do.

Array conventions (all host, C-contiguous numpy):
  pool    uint16 [L][2][n_blocks][block_size][H][D]   bf16 bit patterns, kv 0 = K, 1 = V
  table   int32  [n_table_blocks]
  chunk   uint8  [chunk_bytes]  raw: bf16 [L][2][T][H][D];
                                int8: int8 codes [L][2][T][H][D] then fp32 scales [L][2][T][H*D/64]
                                int4: nibbles [L][2][T][H][D/2] bytes (element 2k low, 2k+1 high) then the same scales
                                per-channel key codecs: the same codes, then per layer fp32 k_scales [ceil(T/64)][H*D]
                                followed by fp32 v_scales [T][H*D/64]
                                token-delta Rice codecs: uint64 seg_off[S+1], fp32 scales[S][H*D], uint8 lens[S][H*D],
                                uint8 params[S][H*D], then the segments' bit streams (see td_layout); the array has
                                the worst-case capacity, td_used_bytes() of it are defined
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

RAW_BF16 = 0
INT8_G64 = 1
INT4_G64 = 2
INT8_KC64 = 3      # keys grouped along tokens (64 tokens of one channel), values as INT8_G64
INT4_KC64 = 4      # the same with codes in [-7, 7]
INT8_TD64 = 5      # K and V grouped along tokens, each group's codes as a Rice-coded sub-stream (direct or token delta)
INT4_TD64 = 6      # the same with codes in [-7, 7]
GROUP = 64

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kdn_oracle.c")
_LIB = os.path.join(_HERE, "libkdn_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle (no fast-math, no fused multiply-add contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        cmd = ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    with _lock:
        if _lib is None:
            _lib = _declare(C.CDLL(build()))
    return _lib


class use_library:
    """Context manager for the pins' own self-check: run the wrappers of this module against another build of the
    oracle (a copy with a planted mistake), then put the real one back."""

    def __init__(self, path: str):
        self.path = path

    def __enter__(self):
        global _lib
        lib()
        self.saved = _lib
        _lib = _declare(C.CDLL(self.path))
        return self

    def __exit__(self, *exc):
        global _lib
        _lib = self.saved
        return False


def compile_source(source_text: str, out_path: str) -> str:
    """Compile oracle source given as text (same flags as build()) to out_path."""
    src = out_path + ".c"
    with open(src, "w") as fh:
        fh.write(source_text)
    subprocess.run(["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", "-w",
                    "-o", out_path, src, "-lm"], check=True)
    return out_path


def _declare(L):
    i32, i64, f64, sz = C.c_int, C.c_int64, C.c_double, C.c_size_t
    vp = C.c_void_p
    L.kdn_oracle_bf16_to_f32.restype = C.c_float
    L.kdn_oracle_bf16_to_f32.argtypes = [C.c_uint16]
    L.kdn_oracle_f32_to_bf16.restype = C.c_uint16
    L.kdn_oracle_f32_to_bf16.argtypes = [C.c_float]
    L.kdn_oracle_f32_to_bf16_many.restype = None
    L.kdn_oracle_f32_to_bf16_many.argtypes = [vp, vp, sz]
    L.kdn_oracle_f64_to_bf16.restype = C.c_uint16
    L.kdn_oracle_f64_to_bf16.argtypes = [f64]
    L.kdn_oracle_chunk_bytes.restype = sz
    L.kdn_oracle_chunk_bytes.argtypes = [i32, i32, i32, i32, i32]
    L.kdn_oracle_quant_group.restype = None
    L.kdn_oracle_quant_group.argtypes = [vp, vp, vp]
    L.kdn_oracle_quant4_group.restype = None
    L.kdn_oracle_quant4_group.argtypes = [vp, vp, vp]
    L.kdn_oracle_quant_channel.restype = None
    L.kdn_oracle_quant_channel.argtypes = [vp, i32, i32, vp, vp]
    L.kdn_oracle_td_layout.restype = i32
    L.kdn_oracle_td_layout.argtypes = [i32, i32, i32, i32, i32, vp]
    L.kdn_oracle_td_max_len.restype = i32
    L.kdn_oracle_td_max_len.argtypes = [i32]
    L.kdn_oracle_zigzag.restype = C.c_uint
    L.kdn_oracle_zigzag.argtypes = [i32]
    L.kdn_oracle_unzigzag.restype = i32
    L.kdn_oracle_unzigzag.argtypes = [C.c_uint]
    L.kdn_oracle_rice_bits.restype = i32
    L.kdn_oracle_rice_bits.argtypes = [C.c_uint, i32, i32]
    L.kdn_oracle_td_encode_channel.restype = None
    L.kdn_oracle_td_encode_channel.argtypes = [vp, i32, i32, vp, C.POINTER(i32), C.POINTER(i32)]
    L.kdn_oracle_td_decode_channel.restype = None
    L.kdn_oracle_td_decode_channel.argtypes = [vp, i32, i32, i32, vp]
    L.kdn_oracle_dequant.restype = C.c_uint16
    L.kdn_oracle_dequant.argtypes = [C.c_int8, C.c_float]
    L.kdn_oracle_rope_angle.restype = f64
    L.kdn_oracle_rope_angle.argtypes = [i64, f64, i32, i32]
    L.kdn_oracle_rotate_pair.restype = None
    L.kdn_oracle_rotate_pair.argtypes = [f64, f64, f64, C.POINTER(f64), C.POINTER(f64)]
    xfer = [vp, i32, i32, i32, i32, i64, vp, i32, i64, i32, i32, vp]
    L.kdn_oracle_store.restype = i32
    L.kdn_oracle_store.argtypes = xfer
    L.kdn_oracle_retrieve.restype = i32
    L.kdn_oracle_retrieve.argtypes = xfer
    xs = [vp, i32, i32, i32, i32, i64, vp, i32, i64, i32, i32, vp, vp]
    L.kdn_oracle_store_sparse.restype = i32
    L.kdn_oracle_store_sparse.argtypes = xs
    L.kdn_oracle_retrieve_sparse.restype = i32
    L.kdn_oracle_retrieve_sparse.argtypes = xs
    L.kdn_oracle_compose_select.restype = i32
    L.kdn_oracle_compose_select.argtypes = [vp, i32, i32, i32, i32, i64, vp, i32, i32,
                                            vp, vp, vp, vp, vp, f64, vp, vp, vp, vp]
    L.kdn_oracle_compose.restype = i32
    L.kdn_oracle_compose.argtypes = [vp, i32, i32, i32, i32, i64, vp, i32, i32,
                                     vp, vp, vp, vp, vp, f64, vp, vp]
    L.kdn_oracle_fnv1a.restype = C.c_uint64
    L.kdn_oracle_fnv1a.argtypes = [vp, sz]
    L.kdn_oracle_key_hash.restype = C.c_uint64
    L.kdn_oracle_key_hash.argtypes = [vp, sz]
    L.kdn_oracle_checksum.restype = C.c_uint64
    L.kdn_oracle_checksum.argtypes = [vp, sz]
    return L


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


def _check_pool(pool: np.ndarray):
    if pool.dtype != np.uint16 or pool.ndim != 6 or pool.shape[1] != 2 or not pool.flags.c_contiguous:
        raise ValueError("pool must be C-contiguous uint16 [L][2][n_blocks][block_size][H][D]")
    L, _, nb, bs, H, D = pool.shape
    return L, H, D, bs, nb


def _check_table(table: np.ndarray):
    if table.dtype != np.int32 or table.ndim != 1 or not table.flags.c_contiguous:
        raise ValueError("table must be C-contiguous int32 [n_table_blocks]")


def chunk_bytes(L: int, H: int, D: int, T: int, codec: int) -> int:
    return int(lib().kdn_oracle_chunk_bytes(L, H, D, T, codec))


def _list(x):
    a = np.ascontiguousarray(x, dtype=np.int32)
    if a.ndim != 1:
        raise ValueError("a token list is one-dimensional")
    return a


def store(pool: np.ndarray, table: np.ndarray, token_offset: int, n_tokens: int, codec: int, keep=None) -> np.ndarray:
    """Gather tokens into a new chunk: positions ``token_offset + t``, or ``token_offset + keep[t]`` for a keep-list
    (then ``n_tokens == len(keep)``)."""
    L, H, D, bs, nb = _check_pool(pool)
    _check_table(table)
    if keep is not None:
        keep = _list(keep)
        if len(keep) != n_tokens:
            raise ValueError("n_tokens must equal len(keep)")
    chunk = np.zeros(chunk_bytes(L, H, D, n_tokens, codec), dtype=np.uint8)
    rc = lib().kdn_oracle_store_sparse(_ptr(pool), L, H, D, bs, nb, _ptr(table), len(table),
                                       int(token_offset), int(n_tokens), int(codec),
                                       _ptr(keep) if keep is not None else None, _ptr(chunk))
    if rc:
        raise ValueError("oracle store: bad arguments (code %d)" % rc)
    return chunk


def retrieve(pool: np.ndarray, table: np.ndarray, token_offset: int, n_tokens: int, codec: int,
             chunk: np.ndarray, keep=None) -> None:
    """Scatter ``chunk`` into ``pool`` in place at request positions ``token_offset + t`` (or ``+ keep[t]``)."""
    if keep is not None:
        keep = _list(keep)
        if len(keep) != n_tokens:
            raise ValueError("n_tokens must equal len(keep)")
    L, H, D, bs, nb = _check_pool(pool)
    _check_table(table)
    if chunk.dtype != np.uint8 or chunk.size != chunk_bytes(L, H, D, n_tokens, codec):
        raise ValueError("chunk has the wrong size for this shape / codec")
    chunk = np.ascontiguousarray(chunk)
    rc = lib().kdn_oracle_retrieve_sparse(_ptr(pool), L, H, D, bs, nb, _ptr(table), len(table),
                                          int(token_offset), int(n_tokens), int(codec),
                                          _ptr(keep) if keep is not None else None, _ptr(chunk))
    if rc:
        raise ValueError("oracle retrieve: bad arguments (code %d)" % rc)


def compose(pool: np.ndarray, table: np.ndarray, parts, theta: float, want_ref: bool = False, select=None):
    """Compose ``parts`` into ``pool`` in place.

    ``parts`` is a list of ``(chunk, n_tokens, codec, base_pos, dst_pos)``.  ``select``: None, or one entry per part,
    each None (deliver every token) or a strictly increasing list of the chunk tokens to deliver.
    With ``want_ref`` returns ``(kref, kmag)``: fp64 ``[L][n_table*bs][H][D]`` arrays holding the
    unrounded key result (NaN where no part wrote) and ``|u| + |w|`` of each rotated pair.
    """
    L, H, D, bs, nb = _check_pool(pool)
    _check_table(table)
    n = len(parts)
    chunks = [np.ascontiguousarray(p[0]) for p in parts]
    for ch, p in zip(chunks, parts):
        if ch.dtype != np.uint8 or ch.size != chunk_bytes(L, H, D, p[1], p[2]):
            raise ValueError("part chunk has the wrong size for this shape / codec")
    ptrs = (C.c_void_p * max(n, 1))(*[c.ctypes.data for c in chunks])
    Ts = np.array([p[1] for p in parts], dtype=np.int32)
    codecs = np.array([p[2] for p in parts], dtype=np.int32)
    base = np.array([p[3] for p in parts], dtype=np.int64)
    dst = np.array([p[4] for p in parts], dtype=np.int64)
    kref = kmag = None
    if want_ref:
        kref = np.full((L, len(table) * bs, H, D), np.nan, dtype=np.float64)
        kmag = np.zeros((L, len(table) * bs, H, D), dtype=np.float64)
    sel_ptr = nsel_ptr = None
    if select is not None:
        if len(select) != n:
            raise ValueError("select needs one entry per part")
        sels = [_list(x if x is not None else np.arange(p[1])) for x, p in zip(select, parts)]
        sel_arr = (C.c_void_p * max(n, 1))(*[a.ctypes.data for a in sels])
        nsel = np.array([len(a) for a in sels], dtype=np.int32)
        sel_ptr, nsel_ptr = C.cast(sel_arr, C.c_void_p), _ptr(nsel)
    rc = lib().kdn_oracle_compose_select(_ptr(pool), L, H, D, bs, nb, _ptr(table), len(table), n,
                                         C.cast(ptrs, C.c_void_p), _ptr(Ts), _ptr(codecs), _ptr(base), _ptr(dst),
                                         float(theta), sel_ptr, nsel_ptr, _ptr(kref) if want_ref else None,
                                         _ptr(kmag) if want_ref else None)
    if rc:
        raise ValueError("oracle compose: bad arguments (code %d)" % rc)
    return (kref, kmag) if want_ref else None


def quant_group(x_bf16: np.ndarray):
    """Encode one group of 64 bf16 bit patterns -> (int8 codes [64], fp32 scale)."""
    x = np.ascontiguousarray(x_bf16, dtype=np.uint16)
    if x.shape != (GROUP,):
        raise ValueError("a group is 64 values")
    q = np.zeros(GROUP, dtype=np.int8)
    s = np.zeros(1, dtype=np.float32)
    lib().kdn_oracle_quant_group(_ptr(x), _ptr(q), _ptr(s))
    return q, s[0]


def quant4_group(x_bf16: np.ndarray):
    """Encode one group of 64 bf16 bit patterns -> (32 bytes of nibbles, fp32 scale)."""
    x = np.ascontiguousarray(x_bf16, dtype=np.uint16)
    if x.shape != (GROUP,):
        raise ValueError("a group is 64 values")
    q = np.zeros(GROUP // 2, dtype=np.uint8)
    s = np.zeros(1, dtype=np.float32)
    lib().kdn_oracle_quant4_group(_ptr(x), _ptr(q), _ptr(s))
    return q, s[0]


def quant_channel(x_bf16: np.ndarray, qmax: int):
    """Encode n <= 64 bf16 bit patterns of one key channel (consecutive tokens) -> (int8 codes [n], fp32 scale)."""
    x = np.ascontiguousarray(x_bf16, dtype=np.uint16)
    if x.ndim != 1 or not 1 <= x.size <= GROUP:
        raise ValueError("a channel group is 1..64 values")
    q = np.zeros(x.size, dtype=np.int8)
    s = np.zeros(1, dtype=np.float32)
    lib().kdn_oracle_quant_channel(_ptr(x), x.size, int(qmax), _ptr(q), _ptr(s))
    return q, s[0]


def td_layout(L: int, H: int, D: int, T: int, codec: int) -> dict:
    """Byte offsets of the regions of a token-delta chunk: segments, scales, lens, params, streams, capacity."""
    out = (C.c_size_t * 6)()
    if lib().kdn_oracle_td_layout(L, H, D, T, codec, out):
        raise ValueError("shape or codec not codable")
    return dict(zip(("segments", "scales", "lens", "params", "streams", "capacity"), [int(x) for x in out]))


def td_used_bytes(chunk: np.ndarray, L: int, H: int, D: int, T: int, codec: int) -> int:
    """The bytes of a stored token-delta chunk that are defined: seg_off[S]."""
    lay = td_layout(L, H, D, T, codec)
    return int(np.ascontiguousarray(chunk[:8 * (lay["segments"] + 1)]).view(np.uint64)[lay["segments"]])


def td_max_len(qmax: int) -> int:
    return int(lib().kdn_oracle_td_max_len(int(qmax)))


def zigzag(e: int) -> int:
    return int(lib().kdn_oracle_zigzag(int(e)))


def unzigzag(u: int) -> int:
    return int(lib().kdn_oracle_unzigzag(int(u)))


def rice_bits(u: int, k: int, raw_bits: int) -> int:
    return int(lib().kdn_oracle_rice_bits(int(u), int(k), int(raw_bits)))


def td_encode_channel(q, qmax: int):
    """Encode the n <= 64 codes of one group -> (bytes, param = mode * 8 + k)."""
    q = np.ascontiguousarray(q, dtype=np.int8)
    if q.ndim != 1 or not 1 <= q.size <= GROUP:
        raise ValueError("a group is 1..64 codes")
    out = np.zeros(td_max_len(qmax), dtype=np.uint8)
    n, p = C.c_int(0), C.c_int(0)
    lib().kdn_oracle_td_encode_channel(_ptr(q), q.size, int(qmax), _ptr(out), C.byref(n), C.byref(p))
    return out[:n.value].copy(), p.value


def td_decode_channel(data, param: int, n: int, qmax: int) -> np.ndarray:
    buf = np.zeros(td_max_len(qmax) + 8, dtype=np.uint8)
    data = np.ascontiguousarray(data, dtype=np.uint8)
    buf[:data.size] = data
    q = np.zeros(n, dtype=np.int8)
    lib().kdn_oracle_td_decode_channel(_ptr(buf), int(param), int(n), int(qmax), _ptr(q))
    return q


def dequant(q: int, scale) -> int:
    return int(lib().kdn_oracle_dequant(int(q), float(np.float32(scale))))


def f32_to_bf16(f) -> int:
    return int(lib().kdn_oracle_f32_to_bf16(float(np.float32(f))))


def f32_to_bf16_many(f: np.ndarray) -> np.ndarray:
    f = np.ascontiguousarray(f, dtype=np.float32)
    out = np.empty(f.shape, dtype=np.uint16)
    lib().kdn_oracle_f32_to_bf16_many(f.ctypes.data, out.ctypes.data, f.size)
    return out


def f64_to_bf16(x: float) -> int:
    return int(lib().kdn_oracle_f64_to_bf16(float(x)))


def bf16_to_f32(b: int) -> float:
    return float(lib().kdn_oracle_bf16_to_f32(int(b)))


def rope_angle(delta: int, theta: float, i: int, D: int) -> float:
    return float(lib().kdn_oracle_rope_angle(int(delta), float(theta), int(i), int(D)))


def rotate_pair(u: float, w: float, phi: float):
    a, b = C.c_double(), C.c_double()
    lib().kdn_oracle_rotate_pair(float(u), float(w), float(phi), C.byref(a), C.byref(b))
    return a.value, b.value


def fnv1a(data: bytes) -> int:
    a = np.frombuffer(data, dtype=np.uint8) if len(data) else np.zeros(0, dtype=np.uint8)
    a = np.ascontiguousarray(a)
    return int(lib().kdn_oracle_fnv1a(_ptr(a) if a.size else None, a.size))


def key_hash(tokens) -> int:
    a = np.ascontiguousarray(tokens, dtype=np.int32)
    return int(lib().kdn_oracle_key_hash(_ptr(a) if a.size else None, a.size))


def checksum(payload: np.ndarray) -> int:
    a = np.ascontiguousarray(payload, dtype=np.uint8)
    if a.size % 4:
        raise ValueError("payload must be a multiple of 4 bytes")
    return int(lib().kdn_oracle_checksum(_ptr(a) if a.size else None, a.size))
