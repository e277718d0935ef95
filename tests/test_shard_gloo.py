"""The N > 1 host logic on CPU: two gloo ranks shard a batch of independent chunks, each runs the (oracle) path on
its share, and the timing reduction takes the maximum over ranks."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2409_13761_b200 import shard, synth


def test_shard_range_is_a_balanced_partition():
    for n in (0, 1, 7, 64, 65, 1000):
        for world in (1, 2, 3, 8):
            parts = [shard.shard_range(n, r, world) for r in range(world)]
            flat = [i for p in parts for i in p]
            assert flat == list(range(n))
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1
    with pytest.raises(ValueError):
        shard.shard_range(4, 2, 2)
    assert shard.job_throughput(10.0, 4, 2.0) == 20.0
    assert shard.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]       # no process group: identity


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert shard.rank_env() == (rank, world, rank)
        shape = synth.TOY.with_(n_blocks=64, block_size=4)
        k, v = synth.make_pool(shape, seed=9)                       # same pool on both ranks
        pool = synth.pool_to_numpy(k, v)
        n_chunks, T = 7, 8
        tables = [np.random.default_rng(100 + c).permutation(64)[:2].astype(np.int32) for c in range(n_chunks)]
        mine = shard.shard_range(n_chunks, rank, world)
        chunks = {c: oracle.store(pool, tables[c], 0, T, oracle.INT8_G64) for c in mine}
        np.savez(os.path.join(out_dir, "rank%d.npz" % rank), **{str(c): ch for c, ch in chunks.items()})
        # the slowest rank sets the time
        t = shard.max_over_ranks([1.0 + rank, 5.0 - rank])
        assert t == [float(world), 5.0]
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_chunks_without_any_exchange(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    shape = synth.TOY.with_(n_blocks=64, block_size=4)
    k, v = synth.make_pool(shape, seed=9)
    pool = synth.pool_to_numpy(k, v)
    got = {}
    for r in range(2):
        with np.load(os.path.join(str(tmp_path), "rank%d.npz" % r)) as z:
            for name in z.files:
                assert int(name) not in got                         # disjoint shares
                got[int(name)] = z[name]
    assert sorted(got) == list(range(7))                            # complete
    for c, ch in got.items():                                       # and identical to the single-process result
        tab = np.random.default_rng(100 + c).permutation(64)[:2].astype(np.int32)
        assert np.array_equal(ch, oracle.store(pool, tab, 0, 8, oracle.INT8_G64))


@pytest.mark.parametrize("codec", [oracle.RAW_BF16, oracle.INT8_G64, oracle.INT4_G64, oracle.INT8_KC64, oracle.INT4_KC64,
                                   oracle.INT8_TD64, oracle.INT4_TD64])
def test_head_sharded_ranks_reproduce_the_unsharded_result(codec):
    """Tensor-parallel sharding: each rank stores and retrieves its own heads with an ordinary descriptor; put side by
    side along the head axis, the ranks' pools equal the pool of the unsharded retrieve (no exchange step)."""
    shape = synth.TOY.with_(n_kv_heads=4, n_blocks=24, block_size=16)
    k, v = synth.make_pool(shape, seed=17)
    pool = synth.pool_to_numpy(k, v)
    src, dst = np.arange(6, dtype=np.int32), np.arange(10, 16, dtype=np.int32)
    off, T = 16, 70
    full = np.zeros_like(pool)
    oracle.retrieve(full, dst, off, T, codec, oracle.store(pool, src, off, T, codec))
    world = 2
    parts = []
    for rank in range(world):
        hs = shard.head_range(shape.n_kv_heads, rank, world)
        mine = np.ascontiguousarray(pool[:, :, :, :, hs.start:hs.stop])
        out = np.zeros_like(mine)
        oracle.retrieve(out, dst, off, T, codec, oracle.store(mine, src, off, T, codec))
        parts.append(out)
    assert np.array_equal(np.concatenate(parts, axis=4), full)
    with pytest.raises(ValueError):
        shard.head_range(4, 0, 3)
