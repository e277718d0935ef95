"""Seeded synthetic inputs: KV pools, block tables, chunk-to-request assignments.

This module serves both the CUDA library's callers and the CPU oracle's tests.
It holds no part of the store / retrieve / compose arithmetic: it only draws
random values, lays them out as a paged pool, and draws block placements.

The paper evaluates on a retrieval-augmented workload of a 70B model (Sec. 3.2
"Early promise": 8K knowledge tokens plus 2K history tokens per request); no
dataset is needed for the data-movement path, so the inputs here reproduce its
shape only: bf16 K/V ~ N(0, 1) with a few large-magnitude channels per head (the
structure real key/value activations show), in the paged layout of a serving
engine, with block tables from fully contiguous to fully fragmented.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

SEED_VALUES = 1234
SEED_OUTLIERS = 1235
SEED_TABLES = 1236
SEED_ASSIGN = 1237

OUTLIERS_PER_HEAD = 4
OUTLIER_GAIN = 20.0


@dataclass(frozen=True)
class KVShape:
    name: str
    n_layers: int
    n_kv_heads: int
    head_dim: int
    block_size: int
    n_blocks: int
    rope_theta: float

    @property
    def row_elems(self) -> int:            # elements of one token in one (layer, K|V) plane
        return self.n_kv_heads * self.head_dim

    @property
    def elems_per_token(self) -> int:      # all layers, K and V
        return self.n_layers * 2 * self.row_elems

    def with_(self, **kw) -> "KVShape":
        d = dict(self.__dict__)
        d.update(kw)
        return KVShape(**d)


TOY = KVShape("toy", 2, 2, 64, 16, 64, 10000.0)
LLAMA3_8B = KVShape("llama3-8b", 32, 8, 128, 16, 16384, 500000.0)
LLAMA3_70B = KVShape("llama3-70b", 80, 8, 128, 16, 16384, 500000.0)


def outlier_gain(shape: KVShape, seed: int = SEED_OUTLIERS) -> torch.Tensor:
    """fp32 [L][2][H][D]: 20 on four distinct seeded channels of every (layer, K|V, head), else 1."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    gain = torch.ones(L, 2, H, D, dtype=torch.float32)
    k = min(OUTLIERS_PER_HEAD, D)
    # argsort of iid uniforms = a uniform random permutation per row; its first k entries are distinct
    picks = torch.rand(L, 2, H, D, generator=g).argsort(dim=-1)[..., :k]
    gain.scatter_(-1, picks, OUTLIER_GAIN)
    return gain


def make_pool(shape: KVShape, device="cpu", seed: int = SEED_VALUES, outliers: bool = True,
              outlier_seed: int = SEED_OUTLIERS) -> Tuple[List[torch.Tensor], List[torch.Tensor]]:
    """Per-layer K and V pools, each bf16 [n_blocks][block_size][H][D], values N(0,1) x channel gain."""
    dev = torch.device(device)
    g = torch.Generator(device=dev).manual_seed(seed)
    gain = outlier_gain(shape, outlier_seed).to(dev) if outliers else None
    dims = (shape.n_blocks, shape.block_size, shape.n_kv_heads, shape.head_dim)
    slab = max(1, min(shape.n_blocks, (1 << 27) // max(1, shape.block_size * shape.row_elems)))
    k_layers, v_layers = [], []
    for l in range(shape.n_layers):
        for kv, dst in ((0, k_layers), (1, v_layers)):
            t = torch.empty(dims, dtype=torch.bfloat16, device=dev)
            for b0 in range(0, shape.n_blocks, slab):
                b1 = min(shape.n_blocks, b0 + slab)
                x = torch.randn((b1 - b0,) + dims[1:], generator=g, device=dev, dtype=torch.float32)
                if gain is not None:
                    x *= gain[l, kv]
                t[b0:b1] = x.to(torch.bfloat16)
            dst.append(t)
    return k_layers, v_layers


def make_table(n: int, pool_blocks: int, run_length: Optional[int], seed: int = SEED_TABLES,
               exclude: Optional[Sequence[int]] = None) -> np.ndarray:
    """int32 [n] physical block ids, pairwise distinct and disjoint from ``exclude``.

    The table is a sequence of runs of ``run_length`` consecutive physical blocks, the runs placed at
    seeded random aligned slots: ``run_length=None`` (or >= n) is one contiguous run, 1 is a uniformly
    random placement of every block.
    """
    if n == 0:
        return np.zeros(0, dtype=np.int32)
    r = n if (run_length is None or run_length >= n) else max(1, int(run_length))
    rng = np.random.default_rng(seed)
    taken = np.zeros(pool_blocks, dtype=bool)
    if exclude is not None and len(exclude):
        taken[np.asarray(exclude, dtype=np.int64)] = True
    n_runs = -(-n // r)
    if r == 1:
        free = np.flatnonzero(~taken)
        if len(free) < n:
            raise ValueError("not enough free blocks")
        return rng.permutation(free)[:n].astype(np.int32)
    # all start positions whose r blocks are free; greedily take a random non-overlapping subset
    c = np.concatenate(([0], np.cumsum(taken)))
    starts = np.flatnonzero((c[r:] - c[:-r]) == 0)
    rng.shuffle(starts)
    out: List[np.ndarray] = []
    for s in starts:
        if len(out) == n_runs:
            break
        if not taken[s:s + r].any():
            taken[s:s + r] = True
            out.append(np.arange(s, s + r))
    if len(out) < n_runs:
        raise ValueError("not enough free runs of %d blocks" % r)
    return np.concatenate(out)[:n].astype(np.int32)


def assign_chunks(n_requests: int, chunks_per_request: int, n_library: int,
                  seed: int = SEED_ASSIGN) -> np.ndarray:
    """int64 [n_requests][chunks_per_request]: which library chunk each request slot reuses."""
    rng = np.random.default_rng(seed)
    return rng.integers(0, n_library, size=(n_requests, chunks_per_request))


def pool_to_numpy(k_layers: Sequence[torch.Tensor], v_layers: Sequence[torch.Tensor],
                  blocks: Optional[Sequence[int]] = None,
                  layers: Optional[Sequence[int]] = None) -> np.ndarray:
    """Host copy uint16 [L'][2][nb'][bs][H][D] of the given blocks (all if None) of the given layers."""
    ls = list(range(len(k_layers))) if layers is None else list(layers)
    idx = None
    if blocks is not None:
        idx = torch.as_tensor(np.asarray(blocks, dtype=np.int64), device=k_layers[0].device)
    planes = []
    for l in ls:
        pair = []
        for t in (k_layers[l], v_layers[l]):
            sel = t if idx is None else t.index_select(0, idx)
            pair.append(sel.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))
        planes.append(np.stack(pair))
    return np.ascontiguousarray(np.stack(planes))


def numpy_to_layers(pool: np.ndarray, device="cpu") -> Tuple[List[torch.Tensor], List[torch.Tensor]]:
    """Inverse of ``pool_to_numpy`` for a whole pool: per-layer bf16 tensors on ``device``."""
    k_layers, v_layers = [], []
    for l in range(pool.shape[0]):
        for kv, dst in ((0, k_layers), (1, v_layers)):
            t = torch.from_numpy(pool[l, kv].view(np.int16).copy()).view(torch.bfloat16).to(device)
            dst.append(t.contiguous())
    return k_layers, v_layers


def compact_table(table: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(unique physical blocks, table rewritten to index into them) for streaming a pool subset."""
    uniq, inv = np.unique(table, return_inverse=True)
    return uniq.astype(np.int64), inv.astype(np.int32)


def correlated_tokens(shape: KVShape, n_tokens: int, rho: float, seed: int, device="cpu", outliers: bool = True) -> torch.Tensor:
    """bf16 [L][2][n_tokens][H][D]: every channel a stationary first-order autoregressive sequence along tokens,
    x_t = rho x_{t-1} + sqrt(1 - rho^2) eps_t with eps ~ N(0, 1) (so x_t ~ N(0, 1) and neighbouring tokens correlate
    with coefficient rho; rho = 0 is the uncorrelated input of make_pool), times the channel gain of outlier_gain."""
    dev = torch.device(device)
    g = torch.Generator(device=dev).manual_seed(seed)
    L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
    eps = torch.randn((n_tokens, L * 2 * H * D), generator=g, device=dev, dtype=torch.float32)
    if rho != 0.0:
        # x = M eps with M[t][s] = rho^(t-s) sqrt(1 - rho^2) for 0 < s <= t and M[t][0] = rho^t
        t = torch.arange(n_tokens, device=dev, dtype=torch.float64)
        m = torch.tril(torch.pow(torch.tensor(float(rho), dtype=torch.float64, device=dev), (t[:, None] - t[None, :]).clamp(min=0)))
        m[:, 1:] *= float(np.sqrt(1.0 - rho * rho))
        eps = m.to(torch.float32) @ eps
    x = eps.reshape(n_tokens, L, 2, H, D).permute(1, 2, 0, 3, 4)
    if outliers:
        x = x * outlier_gain(shape).to(dev)[:, :, None]
    return x.to(torch.bfloat16).contiguous()


def place_tokens(k_layers: Sequence[torch.Tensor], v_layers: Sequence[torch.Tensor], table: np.ndarray, token_offset: int,
                 x: torch.Tensor) -> None:
    """Write x [L][2][T][H][D] into the pool at request positions token_offset + t of the request whose block table is
    ``table`` (input generation only: this is where a serving engine's prefill would have put the tokens)."""
    bs = k_layers[0].shape[1]
    pos = token_offset + np.arange(x.shape[2])
    blocks = torch.as_tensor(np.asarray(table, dtype=np.int64)[pos // bs], device=k_layers[0].device)
    slots = torch.as_tensor(pos % bs, device=k_layers[0].device)
    for l in range(len(k_layers)):
        k_layers[l][blocks, slots] = x[l, 0].to(k_layers[l].device)
        v_layers[l][blocks, slots] = x[l, 1].to(v_layers[l].device)
