"""Shared helpers for the GPU parity tests: run the C-ABI library and the CPU oracle on the same inputs."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2409_13761_b200 import synth


def kdn():
    from paper_2409_13761_b200 import kdn as _kdn
    return _kdn


class Device:
    """A pool on cuda:0 registered with a fresh library context."""

    def __init__(self, shape: synth.KVShape, seed=synth.SEED_VALUES, outliers=True, pool_np: np.ndarray = None):
        K = kdn()
        self.K = K
        self.shape = shape
        self.dev = torch.device("cuda:0")
        if pool_np is None:
            self.k, self.v = synth.make_pool(shape, self.dev, seed=seed, outliers=outliers)
        else:
            self.k, self.v = synth.numpy_to_layers(pool_np, self.dev)
        self.ctx = K.kdn_create(0)
        self.desc = K.pool_desc(shape.n_layers, shape.n_kv_heads, shape.head_dim, shape.block_size, shape.n_blocks,
                                [t.data_ptr() for t in self.k], [t.data_ptr() for t in self.v])
        self.pool_id = K.kdn_pool_register(self.ctx, self.desc)
        self.stream = torch.cuda.Stream(device=self.dev)
        self._keep = []

    def close(self):
        torch.cuda.synchronize()
        self.K.kdn_destroy(self.ctx)
        self.ctx = None

    def table(self, t: np.ndarray) -> torch.Tensor:
        x = torch.from_numpy(np.ascontiguousarray(t, dtype=np.int32)).to(self.dev)
        self._keep.append(x)
        return x

    def chunk_buf(self, n_tokens: int, codec: int, pinned=False, fill=0xA5) -> torch.Tensor:
        nbytes = self.K.kdn_chunk_bytes(self.desc, n_tokens, codec)
        if pinned:
            b = torch.full((max(nbytes, 1),), fill, dtype=torch.uint8).pin_memory()
        else:
            b = torch.full((max(nbytes, 1),), fill, dtype=torch.uint8, device=self.dev)
        self._keep.append(b)
        return b[:nbytes]

    def chunk(self, buf: torch.Tensor, n_tokens: int, codec: int, base_pos=0):
        K = self.K
        mem = K.KDN_MEM_DEVICE if buf.is_cuda else K.KDN_MEM_PINNED_HOST
        return K.Chunk(buf.data_ptr(), buf.numel(), n_tokens, codec, mem, base_pos)

    def op(self, table_dev: torch.Tensor, off: int, buf: torch.Tensor, n_tokens: int, codec: int):
        return self.K.XferOp(table_dev.data_ptr(), table_dev.numel(), off, self.chunk(buf, n_tokens, codec))

    def sync(self) -> int:
        st = self.K.kdn_status_sync(self.ctx, self.stream.cuda_stream)
        torch.cuda.synchronize()
        return st

    def store(self, ops):
        self.K.kdn_store(self.ctx, self.pool_id, ops, self.stream.cuda_stream)

    def retrieve(self, ops):
        self.K.kdn_retrieve(self.ctx, self.pool_id, ops, self.stream.cuda_stream)

    def compose(self, reqs):
        self.K.kdn_compose(self.ctx, self.pool_id, reqs, self.stream.cuda_stream)

    def pool_np(self, blocks=None, layers=None) -> np.ndarray:
        torch.cuda.synchronize()
        return synth.pool_to_numpy(self.k, self.v, blocks, layers)


def to_np(buf: torch.Tensor) -> np.ndarray:
    return buf.detach().cpu().numpy().copy()


def bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in bf16 steps between two bit patterns (finite values), across zero."""
    def key(x):
        x = x.astype(np.int32)
        return np.where(x & 0x8000, -(x & 0x7fff), x & 0x7fff)
    return np.abs(key(a_bits) - key(b_bits))


def check_rotated_keys(got_bits: np.ndarray, kref: np.ndarray, kmag: np.ndarray, oracle_bits: np.ndarray, min_equal=0.995):
    """Tolerance for re-rotated keys.

    |got - ref64| <= 2^-8 |ref64| + 2^-21 (|u| + |w|): one bf16 ulp relative to the fp64 result, plus a
    floor for results that cancel to almost nothing, where the fp32 rounding of the table and of the
    products (each <= 2^-24 relative to |u| or |w|) is all that is left.  Also: at most one bf16 step
    from the oracle's own rounding wherever the result did not cancel, and almost always equal to it.
    """
    got = bits_to_f64(got_bits)
    err = np.abs(got - kref)
    tol = 2.0 ** -8 * np.abs(kref) + 2.0 ** -21 * kmag
    bad = err > tol
    assert not bad.any(), "%d rotated key elements out of tolerance, worst %.3g vs %.3g" % (
        int(bad.sum()), float(err[bad].max()), float(tol[bad].max()))
    d = bf16_ulp_distance(got_bits, oracle_bits)
    # where the result did not cancel (|ref| >= 2^-12 (|u|+|w|)) the fp32 error is far below a bf16 step, so the
    # kernel may differ from the oracle's rounding by one step at most (a near-tie); cancelled results are
    # covered by the absolute floor above only
    solid = np.abs(kref) >= 2.0 ** -12 * kmag
    assert d[solid].max(initial=0) <= 1, "rotated key differs from the rounded fp64 result by %d bf16 steps" % int(d[solid].max())
    frac_equal = float((d == 0).mean())
    assert frac_equal > min_equal, "only %.4f of rotated keys equal the rounded fp64 result" % frac_equal
    return frac_equal
