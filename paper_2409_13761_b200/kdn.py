"""ctypes binding of libkdn.so: the functions of include/kdn.h under the same names.

Argument marshalling only.  Every step of store / retrieve / compose runs in the library's CUDA
kernels; there is no Python or CPU implementation behind these calls.  Importing this module fails
if libkdn.so is absent and cannot be built.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

from . import build as _build

KDN_OK, KDN_E_INVAL, KDN_E_SHAPE, KDN_E_ALIGN, KDN_E_RANGE, KDN_E_UNSUPPORTED, KDN_E_CUDA, KDN_E_NOMEM, \
    KDN_E_TIMEOUT, KDN_E_NOTFOUND, KDN_E_CHECKSUM, KDN_E_IO = range(12)
KDN_CODEC_RAW_BF16, KDN_CODEC_INT8_G64, KDN_CODEC_INT4_G64, KDN_CODEC_INT8_KC64, KDN_CODEC_INT4_KC64 = 0, 1, 2, 3, 4
KDN_CODEC_INT8_TD64, KDN_CODEC_INT4_TD64 = 5, 6
KDN_MEM_DEVICE, KDN_MEM_PINNED_HOST = 0, 1

EXPORTS = ["kdn_create", "kdn_destroy", "kdn_pool_register", "kdn_chunk_bytes", "kdn_validate_xfer",
           "kdn_validate_compose", "kdn_td_layout", "kdn_store", "kdn_retrieve", "kdn_compose", "kdn_status_sync",
           "kdn_set_tuning", "kdn_set_staging_bytes", "kdn_set_wait_limit_ns", "kdn_launch_count", "kdn_last_launch", "kdn_strerror",
           "kdn_compose_static", "kdn_retrieve_layerwise", "kdn_store_file", "kdn_retrieve_file",
           "kdn_store_sparse", "kdn_retrieve_sparse", "kdn_compose_select",
           "kdn_key_hash", "kdn_checksum", "kdn_header_fill", "kdn_header_check", "kdn_index_create", "kdn_index_destroy",
           "kdn_index_put", "kdn_index_get", "kdn_index_remove", "kdn_index_stats"]


class kdn_pool_desc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("block_size", C.c_int32), ("n_blocks", C.c_int64),
                ("k_layers", C.POINTER(C.c_void_p)), ("v_layers", C.POINTER(C.c_void_p))]


class kdn_chunk(C.Structure):
    _fields_ = [("data", C.c_void_p), ("bytes", C.c_size_t), ("n_tokens", C.c_int32), ("codec", C.c_int32),
                ("mem", C.c_int32), ("reserved", C.c_int32), ("base_pos", C.c_int64)]


class kdn_xfer_op(C.Structure):
    _fields_ = [("block_table", C.c_void_p), ("n_table_blocks", C.c_int32), ("reserved", C.c_int32),
                ("token_offset", C.c_int64), ("chunk", kdn_chunk)]


class kdn_compose_req(C.Structure):
    _fields_ = [("block_table", C.c_void_p), ("n_table_blocks", C.c_int32), ("n_parts", C.c_int32),
                ("parts", C.POINTER(kdn_chunk)), ("part_dst_pos", C.POINTER(C.c_int64)),
                ("rope_theta", C.c_double), ("rope_style", C.c_int32), ("reserved", C.c_int32)]


class kdn_sparse_op(C.Structure):
    _fields_ = [("op", kdn_xfer_op), ("keep", C.c_void_p)]


class kdn_file_op(C.Structure):
    _fields_ = [("op", kdn_xfer_op), ("fd", C.c_int32), ("reserved", C.c_int32), ("file_offset", C.c_int64)]


class kdn_select(C.Structure):
    _fields_ = [("part_select", C.POINTER(C.c_void_p)), ("part_n_select", C.POINTER(C.c_int32))]


class kdn_chunk_header(C.Structure):
    _fields_ = [("magic", C.c_char * 8), ("header_bytes", C.c_uint32), ("codec", C.c_uint32),
                ("n_layers", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("n_tokens", C.c_int32),
                ("base_pos", C.c_int64), ("payload_bytes", C.c_uint64), ("key", C.c_uint64), ("checksum", C.c_uint64),
                ("reserved", C.c_uint8 * 64)]


class kdn_index_info(C.Structure):
    _fields_ = [("capacity_bytes", C.c_size_t), ("bytes", C.c_size_t), ("entries", C.c_size_t),
                ("hits", C.c_uint64), ("misses", C.c_uint64), ("evictions", C.c_uint64)]


class kdn_td_layout_info(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("segments", "scales_offset", "lens_offset", "params_offset", "streams_offset", "capacity")]


class kdn_launch_info(C.Structure):
    _fields_ = [("op", C.c_int32), ("compute_groups", C.c_int32), ("group_warps", C.c_int32), ("tile_bytes", C.c_int32),
                ("stages", C.c_int32), ("ctas_per_sm", C.c_int32), ("store_lag", C.c_int32), ("grid", C.c_int32),
                ("smem_bytes", C.c_int32), ("n_tiles", C.c_uint32), ("rows_per_tile", C.c_int32), ("rows_kernel", C.c_int32)]


class kdn_tuning(C.Structure):
    _fields_ = [("tile_bytes", C.c_int32), ("stages", C.c_int32), ("ctas_per_sm", C.c_int32),
                ("compute_groups", C.c_int32), ("store_lag", C.c_int32), ("group_warps", C.c_int32)]


def _load() -> C.CDLL:
    path = _build.LIB
    if not _build.up_to_date():
        try:
            _build.build()
        except Exception as exc:                      # no nvcc, or the compile failed
            if not os.path.exists(path):
                raise ImportError("libkdn.so is missing and could not be built: %s" % exc) from exc
    lib = C.CDLL(path)
    vp, i32 = C.c_void_p, C.c_int
    lib.kdn_create.restype = i32
    lib.kdn_create.argtypes = [C.POINTER(vp), i32]
    lib.kdn_destroy.restype = None
    lib.kdn_destroy.argtypes = [vp]
    lib.kdn_pool_register.restype = i32
    lib.kdn_pool_register.argtypes = [vp, C.POINTER(kdn_pool_desc), C.POINTER(i32)]
    lib.kdn_chunk_bytes.restype = C.c_size_t
    lib.kdn_chunk_bytes.argtypes = [C.POINTER(kdn_pool_desc), C.c_int32, C.c_int32]
    lib.kdn_td_layout.restype = i32
    lib.kdn_td_layout.argtypes = [C.POINTER(kdn_pool_desc), C.c_int32, C.c_int32, C.POINTER(kdn_td_layout_info)]
    lib.kdn_validate_xfer.restype = i32
    lib.kdn_validate_xfer.argtypes = [C.POINTER(kdn_pool_desc), C.POINTER(kdn_xfer_op), i32]
    lib.kdn_validate_compose.restype = i32
    lib.kdn_validate_compose.argtypes = [C.POINTER(kdn_pool_desc), C.POINTER(kdn_compose_req), i32]
    for name in ("kdn_store", "kdn_retrieve"):
        fn = getattr(lib, name)
        fn.restype = i32
        fn.argtypes = [vp, i32, C.POINTER(kdn_xfer_op), i32, vp, vp]
    lib.kdn_retrieve_layerwise.restype = i32
    lib.kdn_retrieve_layerwise.argtypes = [vp, i32, C.POINTER(kdn_xfer_op), i32, i32, vp, vp, C.POINTER(vp)]
    for name in ("kdn_store_sparse", "kdn_retrieve_sparse"):
        fn = getattr(lib, name)
        fn.restype = i32
        fn.argtypes = [vp, i32, C.POINTER(kdn_sparse_op), i32, vp, vp]
    for name in ("kdn_store_file", "kdn_retrieve_file"):
        fn = getattr(lib, name)
        fn.restype = i32
        fn.argtypes = [vp, i32, C.POINTER(kdn_file_op), i32, vp, vp]
    lib.kdn_compose_select.restype = i32
    lib.kdn_compose_select.argtypes = [vp, i32, C.POINTER(kdn_compose_req), C.POINTER(kdn_select), i32, vp, vp]
    lib.kdn_compose.restype = i32
    lib.kdn_compose.argtypes = [vp, i32, C.POINTER(kdn_compose_req), i32, vp, vp]
    lib.kdn_compose_static.restype = i32
    lib.kdn_compose_static.argtypes = [i32, C.POINTER(kdn_pool_desc), C.POINTER(kdn_compose_req), i32, vp, i32]
    lib.kdn_status_sync.restype = i32
    lib.kdn_status_sync.argtypes = [vp, vp]
    lib.kdn_set_tuning.restype = i32
    lib.kdn_set_tuning.argtypes = [vp, C.POINTER(kdn_tuning)]
    lib.kdn_set_staging_bytes.restype = i32
    lib.kdn_set_staging_bytes.argtypes = [vp, C.c_size_t]
    lib.kdn_set_wait_limit_ns.restype = i32
    lib.kdn_set_wait_limit_ns.argtypes = [vp, C.c_uint64]
    lib.kdn_launch_count.restype = C.c_uint64
    lib.kdn_launch_count.argtypes = [vp]
    lib.kdn_last_launch.restype = i32
    lib.kdn_last_launch.argtypes = [vp, C.POINTER(kdn_launch_info)]
    lib.kdn_key_hash.restype = C.c_uint64
    lib.kdn_key_hash.argtypes = [vp, C.c_size_t]
    lib.kdn_checksum.restype = i32
    lib.kdn_checksum.argtypes = [i32, vp, C.c_size_t, vp, vp]
    lib.kdn_header_fill.restype = i32
    lib.kdn_header_fill.argtypes = [C.POINTER(kdn_pool_desc), C.POINTER(kdn_chunk), C.c_uint64, C.c_uint64, C.POINTER(kdn_chunk_header)]
    lib.kdn_header_check.restype = i32
    lib.kdn_header_check.argtypes = [C.POINTER(kdn_pool_desc), C.POINTER(kdn_chunk_header), C.c_uint64, C.POINTER(kdn_chunk)]
    lib.kdn_index_create.restype = i32
    lib.kdn_index_create.argtypes = [C.POINTER(vp), C.c_size_t]
    lib.kdn_index_destroy.restype = None
    lib.kdn_index_destroy.argtypes = [vp]
    lib.kdn_index_put.restype = i32
    lib.kdn_index_put.argtypes = [vp, C.c_uint64, C.POINTER(kdn_chunk), C.POINTER(kdn_chunk), i32, C.POINTER(i32)]
    lib.kdn_index_get.restype = i32
    lib.kdn_index_get.argtypes = [vp, C.c_uint64, C.POINTER(kdn_chunk)]
    lib.kdn_index_remove.restype = i32
    lib.kdn_index_remove.argtypes = [vp, C.c_uint64, C.POINTER(kdn_chunk)]
    lib.kdn_index_stats.restype = None
    lib.kdn_index_stats.argtypes = [vp, C.POINTER(kdn_index_info)]
    lib.kdn_strerror.restype = C.c_char_p
    lib.kdn_strerror.argtypes = [i32]
    return lib


lib = _load()


class KdnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__("%s: %s (status %d)" % (where, kdn_strerror(status), status))


def _check(status: int, where: str) -> None:
    if status != KDN_OK:
        raise KdnError(status, where)


# ------------------------------------------------------------ Python-side argument records --

@dataclass
class Chunk:
    data: int                  # address: device memory, or page-locked host memory with mem=KDN_MEM_PINNED_HOST
    bytes: int
    n_tokens: int
    codec: int = KDN_CODEC_RAW_BF16
    mem: int = KDN_MEM_DEVICE
    base_pos: int = 0

    def c(self) -> kdn_chunk:
        return kdn_chunk(self.data, self.bytes, self.n_tokens, self.codec, self.mem, 0, self.base_pos)


@dataclass
class XferOp:
    block_table: int           # device address of int32 [n_table_blocks]
    n_table_blocks: int
    token_offset: int
    chunk: Chunk


@dataclass
class ComposeReq:
    block_table: int
    n_table_blocks: int
    parts: Sequence[Chunk]
    part_dst_pos: Sequence[int]
    rope_theta: float
    rope_style: int = 0


def pool_desc(n_layers: int, n_kv_heads: int, head_dim: int, block_size: int, n_blocks: int,
              k_layers: Optional[Sequence[int]] = None, v_layers: Optional[Sequence[int]] = None) -> kdn_pool_desc:
    """Build a kdn_pool_desc; the pointer arrays are kept alive on the returned object."""
    d = kdn_pool_desc(n_layers, n_kv_heads, head_dim, block_size, n_blocks, None, None)
    if k_layers is not None:
        ka = (C.c_void_p * len(k_layers))(*k_layers)
        va = (C.c_void_p * len(v_layers))(*v_layers)
        d.k_layers = C.cast(ka, C.POINTER(C.c_void_p))
        d.v_layers = C.cast(va, C.POINTER(C.c_void_p))
        d._keep = (ka, va)
    return d


def xfer_array(ops: Sequence[XferOp]):
    arr = (kdn_xfer_op * max(1, len(ops)))()
    for i, o in enumerate(ops):
        arr[i] = kdn_xfer_op(o.block_table, o.n_table_blocks, 0, o.token_offset, o.chunk.c())
    return arr


def compose_array(reqs: Sequence[ComposeReq]):
    arr = (kdn_compose_req * max(1, len(reqs)))()
    keep = []
    for i, r in enumerate(reqs):
        n = len(r.parts)
        parts = (kdn_chunk * max(1, n))(*[p.c() for p in r.parts])
        pos = (C.c_int64 * max(1, n))(*[int(x) for x in r.part_dst_pos])
        keep.append((parts, pos))
        arr[i] = kdn_compose_req(r.block_table, r.n_table_blocks, n, C.cast(parts, C.POINTER(kdn_chunk)),
                                 C.cast(pos, C.POINTER(C.c_int64)), float(r.rope_theta), r.rope_style, 0)
    arr._keep = keep
    return arr


# ------------------------------------------------------------------------- the C ABI's calls --

def kdn_strerror(status: int) -> str:
    return lib.kdn_strerror(int(status)).decode()


def kdn_create(device: int = 0) -> C.c_void_p:
    ctx = C.c_void_p()
    _check(lib.kdn_create(C.byref(ctx), int(device)), "kdn_create")
    return ctx


def kdn_destroy(ctx) -> None:
    lib.kdn_destroy(ctx)


def kdn_pool_register(ctx, desc: kdn_pool_desc) -> int:
    pid = C.c_int(-1)
    _check(lib.kdn_pool_register(ctx, C.byref(desc), C.byref(pid)), "kdn_pool_register")
    return pid.value


def kdn_chunk_bytes(desc: kdn_pool_desc, n_tokens: int, codec: int) -> int:
    return int(lib.kdn_chunk_bytes(C.byref(desc), int(n_tokens), int(codec)))


def kdn_td_layout(desc: kdn_pool_desc, n_tokens: int, codec: int) -> dict:
    """Region offsets of a token-delta Rice chunk: segments, scales_offset, lens_offset, params_offset, streams_offset, capacity."""
    info = kdn_td_layout_info()
    _check(lib.kdn_td_layout(C.byref(desc), int(n_tokens), int(codec), C.byref(info)), "kdn_td_layout")
    return {name: int(getattr(info, name)) for name, _ in kdn_td_layout_info._fields_}


def kdn_validate_xfer(desc: kdn_pool_desc, ops: Sequence[XferOp]) -> int:
    return int(lib.kdn_validate_xfer(C.byref(desc), xfer_array(ops), len(ops)))


def kdn_validate_compose(desc: kdn_pool_desc, reqs: Sequence[ComposeReq]) -> int:
    return int(lib.kdn_validate_compose(C.byref(desc), compose_array(reqs), len(reqs)))


def kdn_store(ctx, pool_id: int, ops: Sequence[XferOp], stream: int = 0, side_stream: int = 0) -> None:
    _check(lib.kdn_store(ctx, pool_id, xfer_array(ops), len(ops), stream, side_stream), "kdn_store")


def kdn_retrieve(ctx, pool_id: int, ops: Sequence[XferOp], stream: int = 0, side_stream: int = 0) -> None:
    _check(lib.kdn_retrieve(ctx, pool_id, xfer_array(ops), len(ops), stream, side_stream), "kdn_retrieve")


def kdn_retrieve_layerwise(ctx, pool_id: int, ops: Sequence[XferOp], layers_per_step: int, stream: int = 0,
                           side_stream: int = 0, layer_ready: Optional[Sequence[int]] = None) -> None:
    """layer_ready: one cudaEvent_t handle (int, 0 = none) per layer, or None."""
    ev = None
    if layer_ready is not None:
        ev = (C.c_void_p * len(layer_ready))(*[int(e) if e else None for e in layer_ready])
    _check(lib.kdn_retrieve_layerwise(ctx, pool_id, xfer_array(ops), len(ops), int(layers_per_step), stream, side_stream,
                                      ev), "kdn_retrieve_layerwise")


def sparse_array(ops: Sequence[XferOp], keeps: Sequence[int]):
    arr = (kdn_sparse_op * max(1, len(ops)))()
    for i, (o, kp) in enumerate(zip(ops, keeps)):
        arr[i] = kdn_sparse_op(kdn_xfer_op(o.block_table, o.n_table_blocks, 0, o.token_offset, o.chunk.c()), kp)
    return arr


def kdn_store_sparse(ctx, pool_id: int, ops: Sequence[XferOp], keeps: Sequence[int], stream: int = 0, side_stream: int = 0) -> None:
    """keeps[i]: device address of the int32 keep-list of ops[i] (ops[i].chunk.n_tokens entries)."""
    _check(lib.kdn_store_sparse(ctx, pool_id, sparse_array(ops, keeps), len(ops), stream, side_stream), "kdn_store_sparse")


def kdn_retrieve_sparse(ctx, pool_id: int, ops: Sequence[XferOp], keeps: Sequence[int], stream: int = 0, side_stream: int = 0) -> None:
    _check(lib.kdn_retrieve_sparse(ctx, pool_id, sparse_array(ops, keeps), len(ops), stream, side_stream), "kdn_retrieve_sparse")


def file_array(ops: Sequence[XferOp], fds: Sequence[int], file_offsets: Sequence[int]):
    arr = (kdn_file_op * max(1, len(ops)))()
    for i, (o, fd, off) in enumerate(zip(ops, fds, file_offsets)):
        arr[i] = kdn_file_op(kdn_xfer_op(o.block_table, o.n_table_blocks, 0, o.token_offset, o.chunk.c()), int(fd), 0, int(off))
    return arr


def kdn_store_file(ctx, pool_id: int, ops: Sequence[XferOp], fds: Sequence[int], file_offsets: Sequence[int],
                   stream: int = 0, side_stream: int = 0) -> None:
    """ops[i].chunk describes the chunk (its data address is ignored); its bytes go to fds[i] at file_offsets[i]."""
    _check(lib.kdn_store_file(ctx, pool_id, file_array(ops, fds, file_offsets), len(ops), stream, side_stream), "kdn_store_file")


def kdn_retrieve_file(ctx, pool_id: int, ops: Sequence[XferOp], fds: Sequence[int], file_offsets: Sequence[int],
                      stream: int = 0, side_stream: int = 0) -> None:
    _check(lib.kdn_retrieve_file(ctx, pool_id, file_array(ops, fds, file_offsets), len(ops), stream, side_stream), "kdn_retrieve_file")


def kdn_compose_select(ctx, pool_id: int, reqs: Sequence[ComposeReq], selects, stream: int = 0, side_stream: int = 0) -> None:
    """selects[r]: list with one entry per part of reqs[r]: None (every token) or (device address, count)."""
    arr = (kdn_select * max(1, len(reqs)))()
    keep = []
    for r, sel in enumerate(selects):
        n = len(sel)
        ptrs = (C.c_void_p * max(1, n))(*[(x[0] if x else None) for x in sel])
        cnts = (C.c_int32 * max(1, n))(*[(x[1] if x else 0) for x in sel])
        keep.append((ptrs, cnts))
        arr[r] = kdn_select(C.cast(ptrs, C.POINTER(C.c_void_p)), C.cast(cnts, C.POINTER(C.c_int32)))
    _check(lib.kdn_compose_select(ctx, pool_id, compose_array(reqs), arr, len(reqs), stream, side_stream), "kdn_compose_select")


def kdn_compose(ctx, pool_id: int, reqs: Sequence[ComposeReq], stream: int = 0, side_stream: int = 0) -> None:
    _check(lib.kdn_compose(ctx, pool_id, compose_array(reqs), len(reqs), stream, side_stream), "kdn_compose")


def kdn_compose_static(device: int, desc: kdn_pool_desc, reqs: Sequence[ComposeReq], stream: int = 0,
                       wait: bool = True) -> int:
    """kdn_compose without a context and without any device allocation (fixed scratch inside the library).

    Returns the status code instead of raising: an argument error, or (with ``wait``) what the kernels recorded."""
    return int(lib.kdn_compose_static(int(device), C.byref(desc), compose_array(reqs), len(reqs), stream, 1 if wait else 0))


def kdn_status_sync(ctx, stream: int = 0) -> int:
    return int(lib.kdn_status_sync(ctx, stream))


def kdn_set_tuning(ctx, tile_bytes: int = 0, stages: int = 0, ctas_per_sm: int = 0, compute_groups: int = 0,
                   store_lag: int = 0, group_warps: int = 0) -> None:
    t = kdn_tuning(tile_bytes, stages, ctas_per_sm, compute_groups, store_lag, group_warps)
    _check(lib.kdn_set_tuning(ctx, C.byref(t)), "kdn_set_tuning")


def kdn_set_staging_bytes(ctx, bytes_per_slab: int) -> None:
    _check(lib.kdn_set_staging_bytes(ctx, int(bytes_per_slab)), "kdn_set_staging_bytes")


def kdn_set_wait_limit_ns(ctx, ns: int) -> None:
    _check(lib.kdn_set_wait_limit_ns(ctx, int(ns)), "kdn_set_wait_limit_ns")


def kdn_launch_count(ctx) -> int:
    return int(lib.kdn_launch_count(ctx))


def kdn_last_launch(ctx) -> dict:
    """Shape of the most recent tile-pipeline launch, with the kernel's name as the profiler prints it."""
    info = kdn_launch_info()
    _check(lib.kdn_last_launch(ctx, C.byref(info)), "kdn_last_launch")
    d = {name: int(getattr(info, name)) for name, _ in kdn_launch_info._fields_}
    d["kernel"] = "kdn_%s%s_kernel<%d, %d>" % (("store", "retrieve", "compose")[d["op"]], "_rows" if d["rows_kernel"] else "",
                                               d["compute_groups"], d["group_warps"])
    return d


# ------------------------------------------------------------------------ storage-module shell --

def _chunk_from_c(c: kdn_chunk) -> Chunk:
    return Chunk(c.data or 0, c.bytes, c.n_tokens, c.codec, c.mem, c.base_pos)


def kdn_key_hash(token_ids) -> int:
    arr = (C.c_int32 * max(1, len(token_ids)))(*[int(t) for t in token_ids])
    return int(lib.kdn_key_hash(arr, len(token_ids)))


def kdn_checksum(device: int, payload: int, nbytes: int, device_out: int, stream: int = 0) -> None:
    _check(lib.kdn_checksum(int(device), payload, int(nbytes), device_out, stream), "kdn_checksum")


def kdn_header_fill(desc: kdn_pool_desc, chunk: Chunk, key: int, checksum: int) -> kdn_chunk_header:
    h = kdn_chunk_header()
    c = chunk.c()
    _check(lib.kdn_header_fill(C.byref(desc), C.byref(c), key, checksum, C.byref(h)), "kdn_header_fill")
    return h


def kdn_header_check(desc: kdn_pool_desc, header: kdn_chunk_header, checksum_of_payload: int):
    """Returns (status, Chunk or None); the Chunk has bytes, n_tokens, codec, base_pos filled in."""
    c = kdn_chunk()
    st = int(lib.kdn_header_check(C.byref(desc), C.byref(header), checksum_of_payload, C.byref(c)))
    return st, (_chunk_from_c(c) if st == KDN_OK else None)


def kdn_index_create(capacity_bytes: int) -> C.c_void_p:
    idx = C.c_void_p()
    _check(lib.kdn_index_create(C.byref(idx), int(capacity_bytes)), "kdn_index_create")
    return idx


def kdn_index_destroy(idx) -> None:
    lib.kdn_index_destroy(idx)


def kdn_index_put(idx, key: int, chunk: Chunk, max_evicted: int = 64):
    """Returns (status, [evicted Chunks])."""
    ev = (kdn_chunk * max(1, max_evicted))()
    n = C.c_int(0)
    c = chunk.c()
    st = int(lib.kdn_index_put(idx, key, C.byref(c), ev, max_evicted, C.byref(n)))
    return st, [_chunk_from_c(ev[i]) for i in range(n.value)]


def kdn_index_get(idx, key: int):
    c = kdn_chunk()
    st = int(lib.kdn_index_get(idx, key, C.byref(c)))
    return st, (_chunk_from_c(c) if st == KDN_OK else None)


def kdn_index_remove(idx, key: int):
    c = kdn_chunk()
    st = int(lib.kdn_index_remove(idx, key, C.byref(c)))
    return st, (_chunk_from_c(c) if st == KDN_OK else None)


def kdn_index_stats(idx) -> kdn_index_info:
    info = kdn_index_info()
    lib.kdn_index_stats(idx, C.byref(info))
    return info
