"""GPU parity at full workload sizes, in the batched launch configuration the benchmark times.

The pools are too large to replay on the CPU, so each test checks (a) sampled requests / layers element by element
against the oracle and (b) properties that hold at any size: raw store-then-retrieve is the identity, blocks that
are not a destination keep their bits, a composed request's suffix is untouched.
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
from paper_2409_13761_b200 import synth
from harness import Device, to_np, check_rotated_keys

pytestmark = pytest.mark.gpu
RAW, INT8, INT4 = oracle.RAW_BF16, oracle.INT8_G64, oracle.INT4_G64


def need_gib(gib):
    """Skip only on a device that is too small as built; on a B200 whose memory is merely occupied, fail: a silent
    skip there would void the full-size rows."""
    torch.cuda.empty_cache()
    free, total = torch.cuda.mem_get_info()
    if total < gib * (1 << 30):
        pytest.skip("needs a device with %d GiB of memory" % gib)
    assert free >= gib * (1 << 30), "needs %d GiB of free device memory, %.1f GiB are free of %.1f" % (
        gib, free / 2 ** 30, total / 2 ** 30)


def sub_chunk(chunk: np.ndarray, L: int, T: int, H: int, D: int, codec: int, layers) -> np.ndarray:
    """The chunk restricted to some layers, in the same layout (a chunk of len(layers) layers)."""
    n = L * 2 * T * H * D
    if codec == RAW:
        return np.ascontiguousarray(chunk.view(np.uint16).reshape(L, -1)[layers]).view(np.uint8).reshape(-1)
    nc = n // 2 if codec == INT4 else n
    codes = np.ascontiguousarray(chunk[:nc].reshape(L, -1)[layers]).reshape(-1)
    scales = np.ascontiguousarray(chunk[nc:].reshape(L, -1)[layers]).reshape(-1)
    return np.concatenate([codes, scales])


def block_sums(dev):
    """Per (plane, block) 64-bit checksum of the whole pool, computed on the device."""
    out = []
    for t in dev.k + dev.v:
        out.append(t.view(torch.int32).reshape(t.shape[0], -1).to(torch.int64).sum(dim=1))
    return torch.stack(out)


def test_8b_store_then_retrieve_64_chunks_of_512_tokens():
    need_gib(60)
    shape = synth.LLAMA3_8B
    dev = Device(shape)
    try:
        n_req, T, bs = 64, 512, shape.block_size
        nb = T // bs
        src = synth.make_table(n_req * nb, shape.n_blocks, 1, synth.SEED_TABLES).reshape(n_req, nb)
        dst = synth.make_table(n_req * nb, shape.n_blocks, 1, synth.SEED_TABLES + 1, exclude=src.reshape(-1)).reshape(n_req, nb)
        d_src, d_dst = dev.table(src.reshape(-1)), dev.table(dst.reshape(-1))
        sample = [0, 29, 63]
        layers = list(range(shape.n_layers))
        for codec in (RAW, INT8, INT4, oracle.INT4_KC64):
            cb = dev.K.kdn_chunk_bytes(dev.desc, T, codec)
            big = torch.empty(n_req * cb, dtype=torch.uint8, device=dev.dev)
            K = dev.K
            st = [K.XferOp(d_src.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
            rt = [K.XferOp(d_dst.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
            before = block_sums(dev)
            dev.store(st)
            assert dev.sync() == 0
            assert torch.equal(block_sums(dev), before)                      # store writes no pool block
            dev.retrieve(rt)
            assert dev.sync() == 0
            after = block_sums(dev)
            keep = torch.ones(shape.n_blocks, dtype=torch.bool, device=dev.dev)
            keep[torch.from_numpy(dst.reshape(-1).astype(np.int64)).to(dev.dev)] = False
            assert torch.equal(after[:, keep], before[:, keep])              # only destination blocks changed
            if codec == RAW:                                                 # identity on every chunk, on the device
                si = torch.from_numpy(src.reshape(-1).astype(np.int64)).to(dev.dev)
                di = torch.from_numpy(dst.reshape(-1).astype(np.int64)).to(dev.dev)
                for t in dev.k + dev.v:
                    assert torch.equal(t.index_select(0, si), t.index_select(0, di))
            def check(i):                                                    # element by element against the oracle
                sp = dev.pool_np(src[i], layers)
                got = to_np(big[i * cb:(i + 1) * cb])
                got_dst = dev.pool_np(dst[i], layers)

                def cpu_side():
                    want = oracle.store(sp, np.arange(nb, dtype=np.int32), 0, T, codec)
                    assert np.array_equal(got, want), (codec, i)
                    ref = np.zeros_like(sp)
                    oracle.retrieve(ref, np.arange(nb, dtype=np.int32), 0, T, codec, want)
                    assert np.array_equal(got_dst, ref), (codec, i)
                return cpu_side
            # int8 (the codec of the benchmark step): every one of the 64 chunks; the others: three of them
            todo = list(range(n_req)) if codec == INT8 else sample
            with ThreadPoolExecutor(max_workers=max(1, min(16, len(os.sched_getaffinity(0))))) as ex:
                for first in range(0, len(todo), 16):                        # 16 chunks of host copies at a time
                    for f in [ex.submit(check(i)) for i in todo[first:first + 16]]:
                        f.result()
            del big
            torch.cuda.empty_cache()
    finally:
        dev.close()
        del dev
        torch.cuda.empty_cache()


def test_8b_rag_compose_10_chunks_of_1024_tokens_with_suffix():
    need_gib(50)
    shape = synth.LLAMA3_8B
    dev = Device(shape)
    try:
        K = dev.K
        n_parts, T, bs = 10, 1024, shape.block_size
        nb = T // bs
        suffix_blocks = 256 // bs
        src = synth.make_table(n_parts * nb, shape.n_blocks, 1, synth.SEED_TABLES + 2).reshape(n_parts, nb)
        req = synth.make_table(n_parts * nb + suffix_blocks, shape.n_blocks, 1, synth.SEED_TABLES + 3, exclude=src.reshape(-1))
        d_src, d_req = dev.table(src.reshape(-1)), dev.table(req)
        layers = [0, 13, 31]
        L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
        for codec in (RAW, INT8, INT4):
            pb = K.kdn_chunk_bytes(dev.desc, T, codec)
            parts = torch.empty(n_parts * pb, dtype=torch.uint8, device=dev.dev)
            dev.store([K.XferOp(d_src.data_ptr() + j * nb * 4, nb, 0, K.Chunk(parts.data_ptr() + j * pb, pb, T, codec)) for j in range(n_parts)])
            assert dev.sync() == 0
            before = block_sums(dev)
            pre = dev.pool_np(req, layers)                                   # the request's blocks before composing
            dev.compose([K.ComposeReq(d_req.data_ptr(), len(req), [K.Chunk(parts.data_ptr() + j * pb, pb, T, codec, K.KDN_MEM_DEVICE, 0)
                                                                  for j in range(n_parts)], [j * T for j in range(n_parts)], shape.rope_theta)])
            assert dev.sync() == 0
            after = block_sums(dev)
            keep = torch.ones(shape.n_blocks, dtype=torch.bool, device=dev.dev)
            keep[torch.from_numpy(req[:n_parts * nb].astype(np.int64)).to(dev.dev)] = False
            assert torch.equal(after[:, keep], before[:, keep])              # suffix blocks and the rest of the pool untouched
            # sampled layers, all parts, against the oracle
            ref = pre.copy()
            ident = np.arange(len(req), dtype=np.int32)
            oparts = []
            for j in range(n_parts):
                ch = sub_chunk(to_np(parts[j * pb:(j + 1) * pb]), L, T, H, D, codec, layers)
                sp = dev.pool_np(src[j], layers)
                assert np.array_equal(ch, oracle.store(sp, np.arange(nb, dtype=np.int32), 0, T, codec))
                oparts.append((ch, T, codec, 0, j * T))
            kref, kmag = oracle.compose(ref, ident, oparts, shape.rope_theta, want_ref=True)
            got = dev.pool_np(req, layers)
            assert np.array_equal(got[:, 1], ref[:, 1])                      # values
            assert np.array_equal(got[:, 0, :nb], ref[:, 0, :nb])            # part 0: delta 0, a plain retrieve
            assert np.array_equal(got[:, :, n_parts * nb:], pre[:, :, n_parts * nb:])   # suffix
            gk = got[:, 0, nb:n_parts * nb].reshape(len(layers), -1, H, D)
            rk = ref[:, 0, nb:n_parts * nb].reshape(len(layers), -1, H, D)
            frac = check_rotated_keys(gk, kref[:, T:n_parts * T], kmag[:, T:n_parts * T], rk)
            assert frac > 0.999
            del parts
            torch.cuda.empty_cache()
    finally:
        dev.close()
        del dev
        torch.cuda.empty_cache()


def test_70b_batch_of_32_requests_each_retrieving_4_chunks_of_2048_tokens():
    need_gib(120)
    shape = synth.LLAMA3_70B
    dev = Device(shape)
    try:
        K = dev.K
        n_lib, T, bs = 16, 2048, shape.block_size
        nb = T // bs
        L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
        assign = synth.assign_chunks(32, 4, n_lib).reshape(-1)               # 128 retrievals
        lib_src = synth.make_table(n_lib * nb, shape.n_blocks, 1, synth.SEED_TABLES).reshape(n_lib, nb)
        dst = synth.make_table(len(assign) * nb, shape.n_blocks, 1, synth.SEED_TABLES + 1).reshape(len(assign), nb)   # the whole pool
        d_src, d_dst = dev.table(lib_src.reshape(-1)), dev.table(dst.reshape(-1))
        layers = [0, 41, 79]
        sample = [0, 77, 127]
        for codec in (INT8, RAW):
            cb = K.kdn_chunk_bytes(dev.desc, T, codec)
            lib = torch.empty(n_lib * cb, dtype=torch.uint8, device=dev.dev)
            dev.store([K.XferOp(d_src.data_ptr() + c * nb * 4, nb, 0, K.Chunk(lib.data_ptr() + c * cb, cb, T, codec)) for c in range(n_lib)])
            assert dev.sync() == 0
            # four of the retrievals read their chunk from page-locked host memory through the side stream
            host_ids = sorted(set(int(assign[r]) for r in (5, 50, 90, 120)))
            pinned = {c: lib[c * cb:(c + 1) * cb].cpu().pin_memory() for c in host_ids}
            ops = []
            for r, c in enumerate(assign):
                c = int(c)
                if r in (5, 50, 90, 120):
                    ch = K.Chunk(pinned[c].data_ptr(), cb, T, codec, K.KDN_MEM_PINNED_HOST)
                else:
                    ch = K.Chunk(lib.data_ptr() + c * cb, cb, T, codec)
                ops.append(K.XferOp(d_dst.data_ptr() + r * nb * 4, nb, 0, ch))
            dev.retrieve(ops)
            assert dev.sync() == 0
            for r in sample + [5, 120]:
                c = int(assign[r])
                ch = sub_chunk(to_np(lib[c * cb:(c + 1) * cb]), L, T, H, D, codec, layers)
                ref = np.zeros((len(layers), 2, nb, bs, H, D), dtype=np.uint16)
                oracle.retrieve(ref, np.arange(nb, dtype=np.int32), 0, T, codec, ch)
                assert np.array_equal(dev.pool_np(dst[r], layers), ref), (codec, r)
            del lib, pinned
            torch.cuda.empty_cache()
    finally:
        dev.close()
        del dev
        torch.cuda.empty_cache()


@pytest.mark.parametrize("run_blocks", [None, 8, 1], ids=["contiguous", "runs_of_8", "fragmented"])
def test_8b_sweep_points_block_size_32_longest_and_shortest_chunks(run_blocks):
    """Two ends of the chunk-length sweep on the 8B shape with block_size 32: one 8192-token chunk and a batch of forty
    128-token chunks, at three block-table fragmentations, stored and retrieved in the batched calls the sweep times."""
    need_gib(20)
    shape = synth.LLAMA3_8B.with_(block_size=32, n_blocks=2048)
    dev = Device(shape)
    try:
        K, bs = dev.K, shape.block_size
        layers = [0, 13, shape.n_layers - 1]
        for T, n_req in ((8192, 1), (128, 40)):
            nb = T // bs
            r = nb if run_blocks is None else run_blocks
            src = synth.make_table(n_req * nb, shape.n_blocks, r, synth.SEED_TABLES).reshape(n_req, nb)
            dst = synth.make_table(n_req * nb, shape.n_blocks, r, synth.SEED_TABLES + 1, exclude=src.reshape(-1)).reshape(n_req, nb)
            d_src, d_dst = dev.table(src.reshape(-1)), dev.table(dst.reshape(-1))
            for codec in (RAW, INT8):
                cb = K.kdn_chunk_bytes(dev.desc, T, codec)
                big = torch.empty(n_req * cb, dtype=torch.uint8, device=dev.dev)
                st = [K.XferOp(d_src.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
                rt = [K.XferOp(d_dst.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
                before = block_sums(dev)
                dev.store(st)
                dev.retrieve(rt)
                assert dev.sync() == 0
                after = block_sums(dev)
                keep = torch.ones(shape.n_blocks, dtype=torch.bool, device=dev.dev)
                keep[torch.from_numpy(dst.reshape(-1).astype(np.int64)).to(dev.dev)] = False
                assert torch.equal(after[:, keep], before[:, keep])          # only destination blocks changed
                for i in (0, n_req - 1):
                    sp = dev.pool_np(src[i], layers)
                    want = oracle.store(sp, np.arange(nb, dtype=np.int32), 0, T, codec)
                    got = sub_chunk(to_np(big[i * cb:(i + 1) * cb]), shape.n_layers, T, shape.n_kv_heads, shape.head_dim, codec, layers)
                    assert np.array_equal(got, want), (T, codec, i)
                    ref = np.zeros_like(sp)
                    oracle.retrieve(ref, np.arange(nb, dtype=np.int32), 0, T, codec, want)
                    assert np.array_equal(dev.pool_np(dst[i], layers), ref), (T, codec, i)
                del big
    finally:
        dev.close()
        del dev
        torch.cuda.empty_cache()


@pytest.mark.parametrize("codec", [oracle.INT8_TD64, oracle.INT4_TD64], ids=["int8td", "int4td"])
def test_8b_token_delta_store_and_retrieve_16_chunks_of_512_tokens(codec):
    """The token-delta Rice codecs at the 8B shape, in the batched calls the benchmark times, on token-correlated input:
    the bytes in use of every chunk are consistent (offset table monotone, 16-byte aligned, equal to the lengths' sums),
    sampled chunks and layers equal the oracle's segment for segment (scales, lengths, parameters, streams), and the
    retrieved blocks equal the oracle's; blocks that are no destination keep their bits."""
    need_gib(50)
    shape = synth.LLAMA3_8B
    dev = Device(shape)
    try:
        K = dev.K
        n_req, T, bs = 16, 512, shape.block_size
        nb = T // bs
        L, H, D = shape.n_layers, shape.n_kv_heads, shape.head_dim
        R, G = H * D, T // 64
        src = synth.make_table(n_req * nb, shape.n_blocks, 1, synth.SEED_TABLES).reshape(n_req, nb)
        dst = synth.make_table(n_req * nb, shape.n_blocks, 1, synth.SEED_TABLES + 1, exclude=src.reshape(-1)).reshape(n_req, nb)
        for i in range(n_req):                                               # neighbouring tokens correlate (rho 0.9 / 0.99)
            synth.place_tokens(dev.k, dev.v, src[i], 0, synth.correlated_tokens(shape, T, 0.9 if i % 2 else 0.99, 500 + i, dev.dev))
        d_src, d_dst = dev.table(src.reshape(-1)), dev.table(dst.reshape(-1))
        cb = K.kdn_chunk_bytes(dev.desc, T, codec)
        lay = K.kdn_td_layout(dev.desc, T, codec)
        S = lay["segments"]
        big = torch.full((n_req * cb,), 0xA5, dtype=torch.uint8, device=dev.dev)
        st = [K.XferOp(d_src.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
        rt = [K.XferOp(d_dst.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
        before = block_sums(dev)
        dev.store(st)
        assert dev.sync() == 0
        assert torch.equal(block_sums(dev), before)
        dev.retrieve(rt)
        assert dev.sync() == 0
        after = block_sums(dev)
        keep = torch.ones(shape.n_blocks, dtype=torch.bool, device=dev.dev)
        keep[torch.from_numpy(dst.reshape(-1).astype(np.int64)).to(dev.dev)] = False
        assert torch.equal(after[:, keep], before[:, keep])
        layers = [0, 17, 31]
        total_used = 0
        for i in range(n_req):
            head = to_np(big[i * cb:i * cb + lay["streams_offset"]])
            seg_off = head[:8 * (S + 1)].view(np.uint64).astype(np.int64)
            lens = head[lay["lens_offset"]:lay["params_offset"]].reshape(S, R)
            sizes = (lens.astype(np.int64).sum(axis=1) + 15) // 16 * 16
            assert seg_off[0] == lay["streams_offset"] and np.array_equal(np.diff(seg_off), sizes)
            assert lens.max() <= (72 if codec == oracle.INT8_TD64 else 40)
            total_used += int(seg_off[S])
            assert torch.all(big[i * cb + int(seg_off[S]):(i + 1) * cb] == 0xA5)       # nothing past the bytes in use
            if i not in (0, 7, 15):
                continue
            sp = dev.pool_np(src[i], layers)
            want = oracle.store(sp, np.arange(nb, dtype=np.int32), 0, T, codec)
            wl = oracle.td_layout(len(layers), H, D, T, codec)
            w_off = want[:8 * (wl["segments"] + 1)].view(np.uint64).astype(np.int64)
            got = to_np(big[i * cb:i * cb + int(seg_off[S])])
            for j, l in enumerate(layers):
                for kv in range(2):
                    for g in range(G):
                        s_full, s_sub = (2 * l + kv) * G + g, (2 * j + kv) * G + g
                        for region, width in (("scales", 4), ("lens", 1), ("params", 1)):
                            a = got[lay[region + "_offset"] + s_full * R * width:lay[region + "_offset"] + (s_full + 1) * R * width]
                            b = want[wl[region] + s_sub * R * width:wl[region] + (s_sub + 1) * R * width]
                            assert np.array_equal(a, b), (i, l, kv, g, region)
                        n = int(w_off[s_sub + 1] - w_off[s_sub])
                        assert n == int(seg_off[s_full + 1] - seg_off[s_full])
                        assert np.array_equal(got[seg_off[s_full]:seg_off[s_full] + n], want[w_off[s_sub]:w_off[s_sub] + n]), (i, l, kv, g)
            ref = np.zeros_like(sp)
            oracle.retrieve(ref, np.arange(nb, dtype=np.int32), 0, T, codec, want)
            assert np.array_equal(dev.pool_np(dst[i], layers), ref), (codec, i)
        bits = 8.0 * total_used / (n_req * T * shape.elems_per_token)
        assert bits < (8.0 if codec == oracle.INT8_TD64 else 3.8)              # correlated input: smaller than the fixed-rate code
    finally:
        dev.close()
        del dev
        torch.cuda.empty_cache()


@pytest.mark.parametrize("heads", [1, 2])
def test_8b_pool_of_one_rank_of_a_head_sharded_engine(heads):
    """What one rank of a tensor-parallel engine holds of the 8B shape: `heads` of the 8 KV heads, i.e. pool blocks of
    4 or 8 KiB, in the launch configuration the benchmark's head-sharded leg times (512-token chunks, 2 GiB per launch,
    fully fragmented tables).  Store then retrieve, raw and int8: pool blocks other than the destinations keep their
    bits, raw is the identity, sampled chunks are checked element by element against the oracle."""
    need_gib(24)
    shape = synth.LLAMA3_8B.with_(n_kv_heads=heads, n_blocks=32768)
    dev = Device(shape)
    try:
        K = dev.K
        T, bs = 512, shape.block_size
        nb = T // bs
        n_req = (2 << 30) // (T * shape.elems_per_token * 2)
        src = synth.make_table(n_req * nb, shape.n_blocks, 1, synth.SEED_TABLES).reshape(n_req, nb)
        dst = synth.make_table(n_req * nb, shape.n_blocks, 1, synth.SEED_TABLES + 1, exclude=src.reshape(-1)).reshape(n_req, nb)
        d_src, d_dst = dev.table(src.reshape(-1)), dev.table(dst.reshape(-1))
        layers = list(range(shape.n_layers))
        for codec in (RAW, INT8):
            cb = K.kdn_chunk_bytes(dev.desc, T, codec)
            big = torch.empty(n_req * cb, dtype=torch.uint8, device=dev.dev)
            st = [K.XferOp(d_src.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
            rt = [K.XferOp(d_dst.data_ptr() + i * nb * 4, nb, 0, K.Chunk(big.data_ptr() + i * cb, cb, T, codec)) for i in range(n_req)]
            before = block_sums(dev)
            dev.store(st)
            assert dev.sync() == 0
            info = K.kdn_last_launch(dev.ctx)
            assert info["tile_bytes"] == bs * heads * shape.head_dim * 2            # a tile is one pool block
            assert codec != RAW or info["ctas_per_sm"] >= 4                          # ... and in the copy form more CTAs keep the bytes in flight
            assert torch.equal(block_sums(dev), before)
            dev.retrieve(rt)
            assert dev.sync() == 0
            after = block_sums(dev)
            keep = torch.ones(shape.n_blocks, dtype=torch.bool, device=dev.dev)
            keep[torch.from_numpy(dst.reshape(-1).astype(np.int64)).to(dev.dev)] = False
            assert torch.equal(after[:, keep], before[:, keep])
            if codec == RAW:
                si = torch.from_numpy(src.reshape(-1).astype(np.int64)).to(dev.dev)
                di = torch.from_numpy(dst.reshape(-1).astype(np.int64)).to(dev.dev)
                for t in dev.k + dev.v:
                    assert torch.equal(t.index_select(0, si), t.index_select(0, di))
            for i in (0, n_req // 3, n_req - 1):
                sp = dev.pool_np(src[i], layers)
                want = oracle.store(sp, np.arange(nb, dtype=np.int32), 0, T, codec)
                assert np.array_equal(to_np(big[i * cb:(i + 1) * cb]), want), (codec, i)
                ref = np.zeros_like(sp)
                oracle.retrieve(ref, np.arange(nb, dtype=np.int32), 0, T, codec, want)
                assert np.array_equal(dev.pool_np(dst[i], layers), ref), (codec, i)
            del big
            torch.cuda.empty_cache()
    finally:
        dev.close()
        del dev
        torch.cuda.empty_cache()
