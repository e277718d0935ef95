"""Multi-GPU plumbing: one process per GPU, no collective on the data path.

Store, retrieve and compose shard with no exchange step (every output element depends on its own token-head
row only), so ranks simply take disjoint chunks or requests and run the same kernels.  The only communication
is for measurement: a barrier and a max over ranks, through torch.distributed (NCCL on GPUs, gloo in tests).
"""
from __future__ import annotations

import os
from typing import Sequence, Tuple

import torch


def rank_env() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the launcher's environment; (0, 1, 0) when run alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def shard_range(n: int, rank: int, world: int) -> range:
    """Contiguous, balanced share of n independent units (chunks, requests) for one rank."""
    if world < 1 or not 0 <= rank < world or n < 0:
        raise ValueError("bad shard arguments")
    base, extra = divmod(n, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def head_range(n_kv_heads: int, rank: int, world: int) -> range:
    """The KV heads one rank of a tensor-parallel group holds: a contiguous, equal share.

    Under tensor parallelism every rank's pool holds ``n_kv_heads / world`` heads of every block, and the rank stores,
    retrieves and composes its own slice of every chunk with an ordinary pool descriptor of that many heads: a coding
    group (64 elements along head_dim, or 64 tokens of one channel) never spans two heads, so the ranks' results are
    exactly the head slices of the unsharded result and nothing is exchanged."""
    if world < 1 or not 0 <= rank < world or n_kv_heads % world:
        raise ValueError("the KV heads must divide evenly over the ranks")
    per = n_kv_heads // world
    return range(rank * per, (rank + 1) * per)


def max_over_ranks(values: Sequence[float], device="cpu", group=None) -> list:
    """Element-wise maximum of a list of floats over all ranks (identity when not initialised)."""
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return t.cpu().tolist()


def job_throughput(units_per_rank: float, world: int, seconds_max_over_ranks: float) -> float:
    """Whole-job rate: all ranks' units over the slowest rank's time."""
    return units_per_rank * world / seconds_max_over_ranks
